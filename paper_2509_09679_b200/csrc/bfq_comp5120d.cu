// Composite transform for d = 5120 = 40 x 128 with BOTH factors on the tensor cores (paper Sec. 3.3).
//
// The seven stages of the 128-point butterfly Q2 are merged into one dense 128 x 128 block, which the
// paper's O(n log n) argument does not need but the hardware rewards: on CUDA cores the 128-point butterfly of
// 40 runs costs about 730 issue slots per token per scheduler (bfq_comp5120.cu), several times the time the row
// spends on the HBM bus, whereas the dense block is 2.6 MFLOP per token on a unit that does 7800 per clock.
// Per token, with X the 40 x 128 bf16 row (run k, position j'):
//
//   MMA 1  T^T[j][k]  = sum_j' Q2[j][j'] X[k][j']      A = Q2 (shared memory, resident), B = X (the TMA tile itself)
//   MMA 2  Y^T[j][i]  = sum_k  T^T[j][k] Q1[i][k]      A = T^T read straight from tensor memory, B = Q1 (shared memory)
//
// so no element passes through a CUDA core before the epilogue.  Accuracy: X is exact in bf16; Q2 is split into two
// bf16 terms (hi + lo, 16 mantissa bits) and MMA 1 runs once per term (kind::f16, fp32 accumulation); MMA 2 is
// kind::tf32: the tensor core reads the fp32 accumulators of MMA 1 as TF32 (the 13 low mantissa bits are dropped)
// and Q1 is rounded to TF32 once.
//
// Shapes.  A group is 4 tokens.  MMA 1: M = 128 (output position j = tensor-memory lane), N = 160 (4 tokens x 40
// runs = the rows of the TMA tile), K = 16 x 8 steps x 2 terms -> D1 (160 columns, two buffers).  MMA 2, per token:
// M = 128, N = 48 (40 output runs + 8 zero rows of Q1), K = 8 x 5 steps, A = 40 columns of D1 -> D2 (4 x 48 columns).
// Both operands of MMA 1 are K-major with the 128-byte swizzle (the layout TMA writes); Q1 is K-major without swizzle.
//
// Warps: 0..15 epilogue (warp w reads lanes 32 (w mod 4) .. + 31 of token w / 4 of the group: one position j, forty
// runs i per thread; the row absmax is combined across the four lane quarters through shared memory; INT4 codes of
// 8 positions x 8 runs are transposed between 8 lanes by three shuffles so that every lane stores whole 32-bit
// words); warp 16 lane 0 issues the MMAs; warp 17 lane 0 the TMA loads (three stages).  Every wait is bounded.
#include <cuda.h>
#include <cuda_bf16.h>
#include <cuda_runtime.h>

#include "bfq_fast.h"
#include "bfq_generic.cuh"
#include "bfq_n4096.cuh"
#include "bfq_ptx.cuh"

namespace bfq {
namespace c5d {

using namespace ptx;

constexpr int kN1 = 40, kN2 = 128, kD = kN1 * kN2;
constexpr int kTok = 4;                 // tokens per group
constexpr int kRuns = kTok * kN1;       // 160 = N of MMA 1
constexpr int kEpiWarps = 16;
constexpr int kMmaWarp = 16, kTmaWarp = 17;
constexpr int kThreads = 32 * 18;
constexpr int kNPad = 48, kKSteps2 = kN1 / 8;
constexpr int kStagesX = 3;

// shared memory map (bytes from a 1024-aligned base)
constexpr int kHalfBytes = kRuns * 128;             // 20480: 64 positions of every run of a group
constexpr int kStageBytes = 2 * kHalfBytes;         // 40960
constexpr int kXOff = 0;                            // [3 stages][2 halves][160 rows][128 B], 128-byte swizzle
constexpr int kQ2Half = kN2 * 128;                  // 16384: 128 rows x 64 positions, bf16
constexpr int kQ2Off = kXOff + kStagesX * kStageBytes;  // [2 terms][2 halves][128 rows][128 B], 128-byte swizzle
constexpr int kQ2Bytes = 4 * kQ2Half;               // 65536
constexpr int kBBlock = kNPad * 8 * 4;              // 1536: one k-step block of Q1 (TF32)
constexpr int kQ1Off = kQ2Off + kQ2Bytes;
constexpr int kBarOff = kQ1Off + kKSteps2 * kBBlock;
constexpr int kAmaxOff = kBarOff + 128;             // float [2 group parities][4 tokens][4 quarters]
constexpr int kMiscOff = kAmaxOff + 128;            // tensor-memory base address
constexpr int kSmemBytes = kMiscOff + 16 + 1024;

// tensor memory columns
constexpr int kD1Col = 0;                 // two buffers of 160
constexpr int kD2Col = 2 * kRuns;         // 320: four tokens x 48

enum : int { kBarXFull = 0, kBarXEmpty = 3, kBarMmaDone = 6, kBarD2Empty = 7, kNumBars = 8 };

struct Params {
    const uint4* q2img;   // device: the shared-memory image of Q2 (hi, lo) built by k_build_dense128
    const float* q1;      // device, [40][40] row-major
    uint8_t* codes;       // [rows][2560] or null
    uint16_t* scales;     // [rows]
    __nv_bfloat16* y;     // [rows][ldy] or null
    int64_t ldy;
    int64_t rows;
    int* status;
    int transpose_q1;     // 1: apply Q1^T (the inverse transform; q2img then holds Q2^T)
    int bits;             // 4 or 8 (codes != null)
};

__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void fence_proxy_async() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }

// Bounded wait.  Between attempts the warp sleeps SLEEP_NS: a poll costs about ten issue slots, and sixteen epilogue
// warps polling at full rate took a third of all instructions.
template <uint32_t SLEEP_NS>
__device__ __forceinline__ bool wait_or_fail(uint32_t bar, uint32_t parity, int* status) {
    for (int i = 0; i < (1 << 22); ++i) {
        if (mbar_try_wait(bar, parity)) return true;
        __nanosleep(SLEEP_NS);
        if ((i & 255) == 255 && *reinterpret_cast<volatile int*>(status) != 0) break;
    }
    atomicExch(status, 1);
    return false;
}

// Shared-memory matrix descriptors (version 1).  K-major with the 128-byte swizzle: rows of 128 bytes, 8-row groups
// 1024 bytes apart (stride byte offset), leading byte offset unused (encoded as 1); the start address advances by
// 32 bytes per 16-element K step inside the swizzle atom.  K-major without swizzle: 8 x 16-byte core matrices.
__device__ __forceinline__ uint64_t desc_sw128(uint32_t addr) {
    return static_cast<uint64_t>((addr & 0x3FFFFu) >> 4) | (static_cast<uint64_t>(1) << 16) |
           (static_cast<uint64_t>(1024 >> 4) << 32) | (static_cast<uint64_t>(1) << 46) | (static_cast<uint64_t>(2) << 61);
}
__device__ __forceinline__ uint64_t desc_plain(uint32_t addr, uint32_t lbo_bytes, uint32_t sbo_bytes) {
    return static_cast<uint64_t>((addr & 0x3FFFFu) >> 4) | (static_cast<uint64_t>(lbo_bytes >> 4) << 16) |
           (static_cast<uint64_t>(sbo_bytes >> 4) << 32) | (static_cast<uint64_t>(1) << 46);
}
// Instruction descriptors: fp32 accumulate, both operands K-major, M = 128.
constexpr uint32_t kIdesc1 = (1u << 4) | (1u << 7) | (1u << 10) | (uint32_t(kRuns >> 3) << 17) | (uint32_t(128 >> 4) << 24);  // bf16 x bf16, N = 160
constexpr uint32_t kIdesc2 = (1u << 4) | (2u << 7) | (2u << 10) | (uint32_t(kNPad >> 3) << 17) | (uint32_t(128 >> 4) << 24);  // tf32 x tf32, N = 48

__device__ __forceinline__ void mma_bf16_ss(uint32_t d_tmem, uint64_t adesc, uint64_t bdesc, uint32_t accumulate) {
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
        ::"r"(d_tmem), "l"(adesc), "l"(bdesc), "r"(kIdesc1), "r"(accumulate)
        : "memory");
}
// A operand from tensor memory (lanes = rows, 8 consecutive 32-bit columns = one K step)
__device__ __forceinline__ void mma_tf32_ts(uint32_t d_tmem, uint32_t a_tmem, uint64_t bdesc, uint32_t accumulate) {
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::tf32 [%0], [%1], %2, %3, p;\n\t}"
        ::"r"(d_tmem), "r"(a_tmem), "l"(bdesc), "r"(kIdesc2), "r"(accumulate)
        : "memory");
}
__device__ __forceinline__ void mma_commit(uint32_t bar) {
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}

__device__ __forceinline__ void tmem_wait_ld8(uint32_t (&v)[8]) {
    asm volatile("tcgen05.wait::ld.sync.aligned;"
                 : "+r"(v[0]), "+r"(v[1]), "+r"(v[2]), "+r"(v[3]), "+r"(v[4]), "+r"(v[5]), "+r"(v[6]), "+r"(v[7])
                 :
                 : "memory");
}

// ---- TMA thread: three stages of 4 tokens ---------------------------------------------------------------------------
__device__ __forceinline__ void issue_load(const CUtensorMap* tmap, uint32_t smem, uint32_t bars, int g) {
    const int64_t token0 = int64_t(kTok) * (blockIdx.x + int64_t(g) * gridDim.x);
    const int stage = g % kStagesX;
    const uint32_t bar = bars + 8 * (kBarXFull + stage), dst = smem + kXOff + stage * kStageBytes;
    mbar_expect_tx(bar, kStageBytes);
    tma_load_3d(dst, tmap, 0, 0, static_cast<int>(token0), bar);
    tma_load_3d(dst + kHalfBytes, tmap, 64, 0, static_cast<int>(token0), bar);
}

// the first loads (every stage is free) go out before the CTA stages its resident operands
__device__ __forceinline__ void tma_prologue(const CUtensorMap* tmap, uint32_t smem, uint32_t bars, int n_groups) {
    for (int g = 0; g < kStagesX && g < n_groups; ++g) issue_load(tmap, smem, bars, g);
}

__device__ __forceinline__ void tma_role(const Params& P, const CUtensorMap* tmap, uint32_t smem, uint32_t bars,
                                         int n_groups) {
    int issued = n_groups < kStagesX ? n_groups : kStagesX;
    for (int g = kStagesX; g < n_groups; ++g) {
        const int stage = g % kStagesX;
        // the stage is free once the MMAs that read it have completed (their commit arrives on x_empty)
        if (!wait_or_fail<40>(bars + 8 * (kBarXEmpty + stage), ((g / kStagesX) - 1) & 1, P.status)) break;
        issue_load(tmap, smem, bars, g);
        issued = g + 1;
    }
    // no copy of this CTA may be in flight when it leaves (returns at once on the normal path)
    for (int g = issued - kStagesX; g < issued; ++g)
        if (g >= 0) wait_or_fail<500>(bars + 8 * (kBarXFull + g % kStagesX), (g / kStagesX) & 1, P.status);
}

// ---- MMA thread -------------------------------------------------------------------------------------------------------
__device__ __forceinline__ bool issue_mma1(const Params& P, uint32_t smem, uint32_t bars, uint32_t tmem_base, int g) {
    const int stage = g % kStagesX;
    if (!wait_or_fail<100>(bars + 8 * (kBarXFull + stage), (g / kStagesX) & 1, P.status)) return false;
    tmem_fence_after();
    const uint32_t d1 = tmem_base + kD1Col + (g & 1) * kRuns;
#pragma unroll
    for (int ks = 0; ks < kN2 / 16; ++ks) {
        const uint64_t b = desc_sw128(smem + kXOff + stage * kStageBytes + (ks >> 2) * kHalfBytes + (ks & 3) * 32);
#pragma unroll
        for (int term = 0; term < 2; ++term) {
            const uint64_t a = desc_sw128(smem + kQ2Off + term * (2 * kQ2Half) + (ks >> 2) * kQ2Half + (ks & 3) * 32);
            mma_bf16_ss(d1, a, b, (ks | term) != 0 ? 1u : 0u);
        }
    }
    mma_commit(bars + 8 * (kBarXEmpty + stage));
    return true;
}

__device__ __forceinline__ void mma_role(const Params& P, uint32_t smem, uint32_t bars, uint32_t tmem_base, int n_groups) {
    int committed = -1;
    bool ok = n_groups == 0 || issue_mma1(P, smem, bars, tmem_base, 0);
    for (int g = 0; ok && g < n_groups; ++g) {
        // keep the tensor pipe fed: the first factor of the next group goes to the other D1 buffer
        if (g + 1 < n_groups && !issue_mma1(P, smem, bars, tmem_base, g + 1)) break;
        // D2 is single-buffered: the epilogue of the previous group must have read it
        if (g >= 1 && !wait_or_fail<32>(bars + 8 * kBarD2Empty, (g - 1) & 1, P.status)) break;
        tmem_fence_after();
        const uint32_t d1 = tmem_base + kD1Col + (g & 1) * kRuns;
#pragma unroll
        for (int tau = 0; tau < kTok; ++tau) {
#pragma unroll
            for (int s = 0; s < kKSteps2; ++s) {
                const uint64_t b = desc_plain(smem + kQ1Off + s * kBBlock, 128, 256);
                mma_tf32_ts(tmem_base + kD2Col + tau * kNPad, d1 + tau * kN1 + 8 * s, b, s > 0 ? 1u : 0u);
            }
        }
        mma_commit(bars + 8 * kBarMmaDone);
        committed = g;
    }
    if (committed >= 0) wait_or_fail<500>(bars + 8 * kBarMmaDone, committed & 1, P.status);
}

// ---- epilogue warps ---------------------------------------------------------------------------------------------------
// 8 x 8 blocks of 4-bit codes held as one word per lane (lane a of 8: position j0 + a, nibble b: run i0 + b) are
// transposed so that lane a holds run i0 + a with nibble p = position j0 + p: three exchanges at lane distance 1, 2, 4
// swap the off-diagonal nibbles, bytes and half-words.  Five independent blocks go through each exchange together.
// Per round a lane keeps the nibbles selected by its mask and takes the others from its partner's word rotated left by
// 4 d or right by 4 d bits (rotl by 32 - 4 d), depending on which side of the exchange it is: keep[] and rot[] are the
// lane's three masks and rotation counts.
__device__ __forceinline__ void transpose8x8_nibbles(uint32_t (&w)[5], const uint32_t (&keep)[3], const uint32_t (&rot)[3]) {
#pragma unroll
    for (int r = 0; r < 3; ++r) {
        uint32_t p[5];
#pragma unroll
        for (int k = 0; k < 5; ++k) p[k] = __shfl_xor_sync(0xffffffffu, w[k], 1 << r);
#pragma unroll
        for (int k = 0; k < 5; ++k) {
            const uint32_t ps = __funnelshift_l(p[k], p[k], rot[r]);
            w[k] = (w[k] & keep[r]) | (ps & ~keep[r]);
        }
    }
}

__device__ __forceinline__ void epilogue_role(const Params& P, uint8_t* sm, uint32_t bars, uint32_t tmem_base, int n_groups,
                                              int w, int lane) {
    const int qd = w & 3, tau = w >> 2, j = 32 * qd + lane, a = lane & 7;
    float* const amax_slots = reinterpret_cast<float*>(sm + kAmaxOff);
    const uint32_t taddr = tmem_base + (static_cast<uint32_t>(32 * qd) << 16) + kD2Col + tau * kNPad;
    const uint32_t keep[3] = {(a & 1) ? 0xF0F0F0F0u : 0x0F0F0F0Fu, (a & 2) ? 0xFF00FF00u : 0x00FF00FFu,
                              (a & 4) ? 0xFFFF0000u : 0x0000FFFFu};
    const uint32_t rot[3] = {(a & 1) ? 28u : 4u, (a & 2) ? 24u : 8u, 16u};
    // A warp whose wait gave up stays in the loop without waiting or loading (dead), so that the four warps of a token
    // always meet at the named barrier of the absmax exchange the same number of times.
    bool dead = false;
    for (int g = 0; g < n_groups; ++g) {
        if (!dead) {
            const bool ok = wait_or_fail<40>(bars + 8 * kBarMmaDone, g & 1, P.status);
            dead = !__all_sync(0xffffffffu, ok);
        }
        if (dead) {  // keep the barrier count of the absmax exchange, do nothing else
            if (P.codes != nullptr) bar_sync(1 + tau, 128);
            continue;
        }
        tmem_fence_after();
        // this thread's position j of its token: 40 output runs
        uint32_t v[kN1];
        tmem_ld32(taddr, reinterpret_cast<uint32_t(&)[32]>(v[0]));
        tmem_ld8(taddr + 32, reinterpret_cast<uint32_t(&)[8]>(v[32]));
        tmem_wait_ld32(reinterpret_cast<uint32_t(&)[32]>(v[0]));
        tmem_wait_ld8(reinterpret_cast<uint32_t(&)[8]>(v[32]));
        tmem_fence_before();
        mbar_arrive(bars + 8 * kBarD2Empty);  // D2 is in registers: the next group's second factor may overwrite it

        const int64_t token = int64_t(kTok) * (blockIdx.x + int64_t(g) * gridDim.x) + tau;
        const bool valid = token < P.rows;
        if (P.y != nullptr) {
            // runs i and i + 1: the even lane stores positions (j, j + 1) of run i, the odd lane those of run i + 1
            const bool odd = lane & 1;
#pragma unroll
            for (int i = 0; i < kN1; i += 2) {
                const float mine = __uint_as_float(odd ? v[i + 1] : v[i]);
                const float other = __shfl_xor_sync(0xffffffffu, __uint_as_float(odd ? v[i] : v[i + 1]), 1);
                const uint32_t word = odd ? pack_bf16x2(other, mine) : pack_bf16x2(mine, other);
                if (valid) *reinterpret_cast<uint32_t*>(P.y + token * P.ldy + (i + (odd ? 1 : 0)) * kN2 + (j & ~1)) = word;
            }
        }
        if (P.codes != nullptr) {
            // row absmax: thread (four partial maxima) -> warp -> the four lane quarters (through shared memory)
            float m4[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
            for (int i = 0; i < kN1; ++i) m4[i & 3] = fmaxf(m4[i & 3], fabsf(__uint_as_float(v[i])));
            float m = fmaxf(fmaxf(m4[0], m4[1]), fmaxf(m4[2], m4[3]));
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, o));
            if (lane == 0) amax_slots[(g & 1) * 16 + tau * 4 + qd] = m;
            __syncwarp();
            bar_sync(1 + tau, 128);  // the four warps of this token (slots alternate between groups: one barrier is enough)
            const float4 q4 = *reinterpret_cast<const float4*>(amax_slots + (g & 1) * 16 + tau * 4);
            const float amax = fmaxf(fmaxf(q4.x, q4.y), fmaxf(q4.z, q4.w));
            float inv;
            const uint16_t sb = row_scale(amax, P.bits == 8 ? 127 : 7, &inv);
            const bool saturated = sb == 0x7BFFu || sb < 0x0400u || !(amax < 3.0e38f);
            if (qd == 0 && lane == 0 && valid) P.scales[token] = sb;
            if (P.bits == 8) {
                // one byte per element: |y / s| < 127.5 for a normal scale, y * inv + 1.5 * 2^23 has the two's complement
                // code in its low byte.  A thread packs four runs into a word; 4 x 4 byte blocks are transposed between
                // four lanes (two byte-permute exchanges) so that lane a stores run 4 blk + a, positions j0 .. j0 + 3.
                const int a4 = lane & 3;
                const uint32_t sel1 = (a4 & 1) ? 0x3715u : 0x6240u, sel2 = (a4 & 2) ? 0x3276u : 0x5410u;
                uint32_t wb[kN1 / 4];
#pragma unroll
                for (int blk = 0; blk < kN1 / 4; ++blk) {
                    uint32_t c[4];
#pragma unroll
                    for (int b = 0; b < 4; ++b) {
                        const float y = __uint_as_float(v[4 * blk + b]);
                        c[b] = saturated ? static_cast<uint32_t>(quant1(y, inv, -128, 127)) : __float_as_uint(fmaf(y, inv, 12582912.0f));
                    }
                    wb[blk] = __byte_perm(__byte_perm(c[0], c[1], 0x0040u), __byte_perm(c[2], c[3], 0x0040u), 0x5410u);
                }
#pragma unroll
                for (int blk = 0; blk < kN1 / 4; ++blk) wb[blk] = __byte_perm(wb[blk], __shfl_xor_sync(0xffffffffu, wb[blk], 1), sel1);
#pragma unroll
                for (int blk = 0; blk < kN1 / 4; ++blk) wb[blk] = __byte_perm(wb[blk], __shfl_xor_sync(0xffffffffu, wb[blk], 2), sel2);
                if (valid) {
#pragma unroll
                    for (int blk = 0; blk < kN1 / 4; ++blk)
                        *reinterpret_cast<uint32_t*>(P.codes + token * kD + (4 * blk + a4) * kN2 + (j & ~3)) = wb[blk];
                }
                continue;
            }
            uint32_t word[5];
            if (!saturated) {
                // |y / s| < 7.5 for a normal, unsaturated fp16 scale: y * inv + (1.5 * 2^23 + 8) has r + 8 in [1, 15] in
                // its low mantissa bits (r = y / s rounded to nearest even); eight of them are summed with weights
                // 16^b, the exponent bits are removed and bit 3 of every nibble is flipped
                constexpr float kMagic = 12582920.0f;
                constexpr uint32_t kUnbias = 0u - 0x4B400000u * 0x11111111u;
#pragma unroll
                for (int blk = 0; blk < 5; ++blk) {
                    uint32_t c[8];
#pragma unroll
                    for (int b = 0; b < 8; ++b) c[b] = __float_as_uint(fmaf(__uint_as_float(v[8 * blk + b]), inv, kMagic));
                    // shift-and-add pairs, then pairs of pairs (three levels instead of a chain of seven)
                    const uint32_t s01 = c[1] * 16u + c[0], s23 = c[3] * 16u + c[2];
                    const uint32_t s45 = c[5] * 16u + c[4], s67 = c[7] * 16u + c[6];
                    const uint32_t lo = s23 * 256u + s01, hi = s67 * 256u + s45;
                    word[blk] = ((hi * 65536u + lo) + kUnbias) ^ 0x88888888u;
                }
            } else {
#pragma unroll
                for (int blk = 0; blk < 5; ++blk) {
                    word[blk] = 0u;
#pragma unroll
                    for (int b = 0; b < 8; ++b)
                        word[blk] |= (static_cast<uint32_t>(quant1(__uint_as_float(v[8 * blk + b]), inv, -8, 7)) & 0xFu) << (4 * b);
                }
            }
            transpose8x8_nibbles(word, keep, rot);
            if (valid) {
#pragma unroll
                for (int blk = 0; blk < 5; ++blk)
                    *reinterpret_cast<uint32_t*>(P.codes + token * (kD / 2) + (8 * blk + a) * (kN2 / 2) + (j >> 3) * 4) = word[blk];
            }
        }
    }
}

__global__ void __launch_bounds__(kThreads, 1)
k_comp5120d(const __grid_constant__ Params P, const __grid_constant__ CUtensorMap tmap, int64_t total_groups) {
    extern __shared__ uint8_t smem_raw[];
    const uint32_t smem = (smem_u32(smem_raw) + 1023u) & ~1023u;
    uint8_t* const sm = smem_raw + (smem - smem_u32(smem_raw));
    const uint32_t bars = smem + kBarOff;
    uint32_t* const tmem_slot = reinterpret_cast<uint32_t*>(sm + kMiscOff);
    const int t = threadIdx.x, warp = t >> 5, lane = t & 31;
    const int n_groups =
        blockIdx.x < total_groups ? static_cast<int>((total_groups - blockIdx.x + gridDim.x - 1) / gridDim.x) : 0;

    if (t == 0) {
        for (int s = 0; s < kStagesX; ++s) {
            mbar_init(bars + 8 * (kBarXFull + s), 1);
            mbar_init(bars + 8 * (kBarXEmpty + s), 1);
        }
        mbar_init(bars + 8 * kBarMmaDone, 1);
        mbar_init(bars + 8 * kBarD2Empty, 32 * kEpiWarps);
        mbar_init_fence();
    }
    __syncwarp();
    if (warp == 0) tmem_alloc512(smem_u32(tmem_slot));
    __syncthreads();  // barriers are initialised: the first loads can go out while the operands are being staged
    if (warp == kTmaWarp && lane == 0) tma_prologue(&tmap, smem, bars, n_groups);
    // Q2 (two bf16 terms, already in the swizzled operand layout) and Q1 (TF32, K-major without swizzle: row i and
    // contraction index kq = k mod 8 of k-step k / 8 at 256 (i / 8) + 16 (i mod 8) + 128 (kq / 4) + 4 (kq mod 4))
    for (int e = t; e < kQ2Bytes / 16; e += kThreads) reinterpret_cast<uint4*>(sm + kQ2Off)[e] = __ldg(P.q2img + e);
    for (int e = t; e < kNPad * kN1; e += kThreads) {
        const int i = e / kN1, k = e - i * kN1, kq = k & 7;
        const float val = i < kN1 ? (P.transpose_q1 ? P.q1[k * kN1 + i] : P.q1[i * kN1 + k]) : 0.f;
        *reinterpret_cast<uint32_t*>(sm + kQ1Off + (k >> 3) * kBBlock + 256 * (i >> 3) + 16 * (i & 7) + 128 * (kq >> 2) +
                                     4 * (kq & 3)) = (__float_as_uint(val) + 0x1000u) & 0xFFFFE000u;
    }
    fence_proxy_async();
    tmem_fence_before();
    __syncthreads();
    tmem_fence_after();
    const uint32_t tmem_base = *tmem_slot;

    if (warp < kEpiWarps) {
        epilogue_role(P, sm, bars, tmem_base, n_groups, warp, lane);
    } else if (warp == kMmaWarp) {
        if (lane == 0) mma_role(P, smem, bars, tmem_base, n_groups);
    } else if (warp == kTmaWarp) {
        if (lane == 0) tma_role(P, &tmap, smem, bars, n_groups);
    }
    tmem_fence_before();
    __syncthreads();
    if (warp == 0) {
        tmem_fence_after();
        tmem_dealloc512(tmem_base);
    }
}

// Dense Q2 from the plan's (cos, sin) table: thread c pushes the unit vector e_c through the 7 stages in float64 and
// writes column c, split into two bf16 terms, at its place in the swizzled K-major operand image:
// [term][half = c / 64][row j][16-byte chunk ((c mod 64) / 8) xor (j mod 8)][c mod 8].
// The second image (offset kQ2Bytes) holds Q2^T in the same layout, for the inverse transform.
__global__ void __launch_bounds__(kN2) k_build_dense128(const float2* __restrict__ tw, __nv_bfloat16* __restrict__ img) {
    const int c = threadIdx.x;
    double col[kN2];
    for (int jj = 0; jj < kN2; ++jj) col[jj] = jj == c ? 1.0 : 0.0;
    for (int s = 0; s < 7; ++s) {
        for (int q = 0; q < kN2 / 2; ++q) {
            const int lo = ((q >> s) << (s + 1)) | (q & ((1 << s) - 1)), hi = lo + (1 << s);
            const float2 cs = tw[s * (kN2 / 2) + q];
            const double x0 = col[lo], x1 = col[hi];
            col[lo] = double(cs.x) * x0 - double(cs.y) * x1;
            col[hi] = double(cs.y) * x0 + double(cs.x) * x1;
        }
    }
    for (int jj = 0; jj < kN2; ++jj) {
        const float f = static_cast<float>(col[jj]);
        const __nv_bfloat16 hi = __float2bfloat16_rn(f);
        const __nv_bfloat16 lo = __float2bfloat16_rn(f - __bfloat162float(hi));
        const int idx = (c >> 6) * (kQ2Half / 2) + jj * 64 + ((((c & 63) >> 3) ^ (jj & 7)) << 3) + (c & 7);
        img[idx] = hi;
        img[2 * (kQ2Half / 2) + idx] = lo;
        // transposed: row c, contraction index jj
        const int idt = (jj >> 6) * (kQ2Half / 2) + c * 64 + ((((jj & 63) >> 3) ^ (c & 7)) << 3) + (jj & 7);
        img[kQ2Bytes / 2 + idt] = hi;
        img[kQ2Bytes / 2 + 2 * (kQ2Half / 2) + idt] = lo;
    }
}

}  // namespace c5d

// ---- host side -----------------------------------------------------------------------------------------------------
size_t comp5120d_image_bytes() { return 2 * c5d::kQ2Bytes; }  // Q2 and Q2^T

bool comp5120d_available(const bfq_plan* plan) {
    return plan->n == c5d::kN2 && plan->cc_major == 10 && plan->dense128 != nullptr && encode_tiled() != nullptr;
}

cudaError_t comp5120d_set_angles(const bfq_plan* plan, cudaStream_t st) {
    c5d::k_build_dense128<<<1, c5d::kN2, 0, st>>>(plan->tw, static_cast<__nv_bfloat16*>(plan->dense128));
    return cudaGetLastError();
}

cudaError_t comp5120d_launch(bfq_plan* plan, const float* q1, const void* x, int64_t rows, int64_t ldx, int bits,
                             uint8_t* codes, uint16_t* scales, void* y_bf16, int64_t ldy, bool inverse, cudaStream_t st) {
    using namespace c5d;
    Params P{};
    P.bits = bits;
    P.q2img = static_cast<const uint4*>(plan->dense128) + (inverse ? kQ2Bytes / 16 : 0);
    P.transpose_q1 = inverse ? 1 : 0;
    P.q1 = q1, P.codes = codes, P.scales = scales, P.y = static_cast<__nv_bfloat16*>(y_bf16), P.ldy = ldy;
    P.rows = rows, P.status = plan->status_word;
    // x: [rows][ldx] bf16 seen as {128 positions of a run, 40 runs, rows tokens}; a box is 64 positions of every run of
    // four tokens, 128-byte swizzled: row 40 token + run of the B operand
    CUtensorMap tmap;
    const cuuint64_t dims[3] = {kN2, kN1, static_cast<cuuint64_t>(rows)};
    const cuuint64_t strides[2] = {kN2 * 2, static_cast<cuuint64_t>(ldx) * 2};
    const cuuint32_t box[3] = {64, kN1, kTok};
    const cuuint32_t estr[3] = {1, 1, 1};
    if (encode_tiled()(&tmap, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void*>(x), dims, strides, box, estr,
                       CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
                       CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
        return cudaErrorInvalidValue;
    static bool attr_set[kMaxDevices] = {};
    if (!attr_set[plan->device]) {
        cudaError_t e = cudaFuncSetAttribute(k_comp5120d, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBytes);
        if (e != cudaSuccess) return e;
        attr_set[plan->device] = true;
    }
    const int64_t total_groups = (rows + kTok - 1) / kTok;
    const int grid = static_cast<int>(total_groups < plan->sm_count ? total_groups : plan->sm_count);
    k_comp5120d<<<grid, kThreads, kSmemBytes, st>>>(P, tmap, total_groups);
    return cudaGetLastError();
}

}  // namespace bfq
