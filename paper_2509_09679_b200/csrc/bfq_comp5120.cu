// Composite transform for d = 5120 = 40 x 128 (paper Sec. 3.3, "Concrete Example for d = 5120"): bf16 token rows,
// Y = Q1 (X Q2^T) with Q2 the 128-point butterfly (7 stages, 448 angles) and Q1 the dense 40 x 40 factor, fused with
// the per-token INT4 quantizer (or written back as bf16 rows).
//
// Why this kernel looks unlike the n = 4096 one.  All 40 runs of all tokens share Q2's 448 angles, so the rotation
// constants can be warp-uniform: a THREAD owns a whole run (128 fp32 registers) and the 32 lanes of a warp hold 32
// different runs.  Every stage is then register-to-register with no exchange at all, and the constants are
// kernel parameters, i.e. constant-bank operands of the FFMAs instead of a third register read.  Each rotation is
// three FMAs (lifting steps a += nt b; b += sn a; a += nt b with nt = -tan(phi/2), sn = sin(phi), |phi| <= pi/2;
// the +-pi reductions leave a sign per position that is applied when the row is written).
//
// The dense factor is the one true contraction of the method and runs on the tensor cores: per token
// D[(j), i] = sum_k X'[k][j] Q1[i][k], a (128 x 40) x (40 x 40) product.  The butterfly threads write X' to shared
// memory as the A operand (rows = positions, the run index k is the contraction dimension), Q1 sits in shared memory
// as the B operand, both K-major in the canonical layout without swizzle; tcgen05.mma (kind::tf32, M = 128, N = 48,
// K = 8, five steps) accumulates into tensor memory, and four epilogue warps read their lanes back with tcgen05.ld,
// take the row absmax, quantize and store.
//
// One CTA per SM walks groups of 4 tokens:
//   warp 10      one thread: TMA loads of the next groups' rows (two stages), then the 20 MMAs of a group + commit
//   warps 4..9   butterfly: claim batches of 32 runs (5 per group), load them from the TMA stage, 7 stages in
//                registers, round to TF32 and store the A operand, arrive on a_full
//   warps 0..3   epilogue: warp w owns token w of the group = tensor-memory lanes 32 w .. 32 w + 31
// Row of the A tile: m = 32 tau + p for token tau and p = j / 4; tile t = j mod 4 (four tiles, 48 columns each), so
// an epilogue thread reads the four adjacent positions j = 4 p + t of every output run i from the four tiles.
// Every wait is bounded; a wait that gives up sets the plan's status word and the CTA drains and leaves.
#include <cuda.h>
#include <cuda_bf16.h>
#include <cuda_runtime.h>

#include <cmath>

#include "bfq_fast.h"
#include "bfq_generic.cuh"
#include "bfq_n4096.cuh"
#include "bfq_ptx.cuh"

namespace bfq {
namespace c5k {

using namespace ptx;

constexpr int kN1 = 40, kN2 = 128, kD = kN1 * kN2, kStages = 7;
constexpr int kTok = 4;                    // tokens per group
constexpr int kRuns = kTok * kN1;          // 160 runs per group
constexpr int kBatches = kRuns / 32;       // 5 batches of 32 runs
constexpr int kEpiWarps = 4, kBflyWarps = 7;
constexpr int kMmaWarp = kEpiWarps + kBflyWarps;
constexpr int kThreads = 32 * (kMmaWarp + 1);  // 384
constexpr int kNPad = 48;                  // MMA N: 40 output runs + 8 zero rows of Q1
constexpr int kKSteps = kN1 / 8;           // 5 MMA steps of K = 8

// shared memory map (bytes from a 1024-aligned base)
constexpr int kHalfBytes = kRuns * 128;            // 20480: one 64-element half of every run of a group
constexpr int kInStageBytes = 2 * kHalfBytes;      // 40960
constexpr int kInOff = 0;                          // [2 stages][2 halves][160 lines][128 B], 128-byte swizzle
// A: bytes between the core matrices of consecutive 4-k chunks.  144 rather than 128: the 32 lanes of a butterfly warp
// hold 32 consecutive k and store the same row, so their words sit at 4 (k mod 4) + 144 (k / 4): 32 distinct banks.
constexpr int kALbo = 144;
constexpr int kASbo = (kN1 / 4) * kALbo;           // A: bytes between consecutive 8-row groups
constexpr int kATile = 16 * kASbo;                 // one tile of A: 128 rows x 40 k, TF32
constexpr int kAOff = kInOff + 2 * kInStageBytes;  // 81920
constexpr int kABytes = 4 * kATile;
constexpr int kBBlock = kNPad * 8 * 4;             // 1536: one k-step block of B
constexpr int kBOff = kAOff + kABytes;             // 163840
constexpr int kBarOff = kBOff + kKSteps * kBBlock; // 171520
constexpr int kSmemBytes = kBarOff + 128 + 1024;   // barriers + alignment slack

enum : int { kBarInFull = 0, kBarAFull = 2, kBarMmaDone = 3, kBarDEmpty = 5, kNumBars = 7 };

struct Params {
    float nt[kStages][kN2 / 2];  // lifting constants of every pair of every stage: -tan(phi / 2) ...
    float sn[kStages][kN2 / 2];  // ... and sin(phi)
    uint32_t sign[4];                 // bit j set: position j of a run carries a pending factor -1
    const float* q1;                  // device, [40][40] row-major
    uint8_t* codes;                   // [rows][2560] or null
    uint16_t* scales;                 // [rows]
    __nv_bfloat16* y;                 // [rows][ldy] or null
    int64_t ldy;
    int64_t rows;
    int* status;
};

__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void fence_proxy_async() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }
// fp32 -> TF32 (10 mantissa bits), round to nearest with ties away from zero, for finite values: half an ulp is
// added to the magnitude; the tensor core reads the upper 19 bits and ignores the 13 low ones
__device__ __forceinline__ uint32_t to_tf32(float v) { return __float_as_uint(v) + 0x1000u; }
__device__ __forceinline__ void sts128(uint32_t addr, uint32_t a, uint32_t b, uint32_t c, uint32_t d) {
    asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(addr), "r"(a), "r"(b), "r"(c), "r"(d) : "memory");
}

// Bounded wait: the hardware suspends the thread for up to about 2 us per attempt (no issue slots are spent while
// it sleeps); gives up after 2^20 attempts, or early once any thread of the grid has reported a failure.
__device__ __forceinline__ bool wait_or_fail(uint32_t bar, uint32_t parity, int* status) {
    for (int i = 0; i < (1 << 20); ++i) {
        uint32_t ok;
        asm volatile(
            "{\n\t.reg .pred p;\n\t"
            "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2, %3;\n\t"
            "selp.u32 %0, 1, 0, p;\n\t}"
            : "=r"(ok)
            : "r"(bar), "r"(parity), "r"(2000u)
            : "memory");
        if (ok != 0) return true;
        if ((i & 63) == 63 && *reinterpret_cast<volatile int*>(status) != 0) break;
    }
    atomicExch(status, 1);
    return false;
}

// Shared-memory matrix descriptor without swizzle (canonical 8 x 16-byte core matrices): start address, leading and
// stride byte offsets in 16-byte units, descriptor version 1.
__device__ __forceinline__ uint64_t smem_desc(uint32_t addr, uint32_t lbo_bytes, uint32_t sbo_bytes) {
    return static_cast<uint64_t>((addr & 0x3FFFFu) >> 4) | (static_cast<uint64_t>(lbo_bytes >> 4) << 16) |
           (static_cast<uint64_t>(sbo_bytes >> 4) << 32) | (static_cast<uint64_t>(1) << 46);
}
// Instruction descriptor: fp32 accumulate, A and B TF32, both K-major, N = 48, M = 128.
constexpr uint32_t kIdesc = (1u << 4) | (2u << 7) | (2u << 10) | (0u << 15) | (0u << 16) | (uint32_t(kNPad >> 3) << 17) |
                            (uint32_t(128 >> 4) << 24);

__device__ __forceinline__ void mma_tf32(uint32_t d_tmem, uint64_t adesc, uint64_t bdesc, uint32_t accumulate) {
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::tf32 [%0], %1, %2, %3, p;\n\t}"
        ::"r"(d_tmem), "l"(adesc), "l"(bdesc), "r"(kIdesc), "r"(accumulate)
        : "memory");
}
__device__ __forceinline__ void mma_commit(uint32_t bar) {
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}

// ---- butterfly warps: a thread owns a whole run ------------------------------------------------------------------
__device__ __forceinline__ void load_run(uint32_t line, int u, float (&x)[kN2]) {
#pragma unroll
    for (int h = 0; h < 2; ++h) {
#pragma unroll
        for (int c = 0; c < 8; ++c) {
            const uint4 v = f4k::lds128(line + h * kHalfBytes + ((c ^ (u & 7)) << 4));
            const uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
            for (int k = 0; k < 4; ++k) {
                x[64 * h + 8 * c + 2 * k + 0] = __uint_as_float(w[k] << 16);
                x[64 * h + 8 * c + 2 * k + 1] = __uint_as_float(w[k] & 0xFFFF0000u);
            }
        }
    }
}

// Q2 on the run: stage s couples lo and lo + 2^s; every constant is a kernel parameter at a fixed offset.  Stage 0
// couples neighbours and runs on scalars; from stage 1 on positions (2 i, 2 i + 1) travel together in one 64-bit
// register and two pairs rotate per packed FMA, their constants being two consecutive floats of the parameter block.
__device__ __forceinline__ void butterfly128(const Params& P, float (&x)[kN2]) {
#pragma unroll
    for (int q = 0; q < kN2 / 2; ++q) {
        const float nt = P.nt[0][q], sn = P.sn[0][q];
        x[2 * q] = fmaf(nt, x[2 * q + 1], x[2 * q]);
        x[2 * q + 1] = fmaf(sn, x[2 * q], x[2 * q + 1]);
        x[2 * q] = fmaf(nt, x[2 * q + 1], x[2 * q]);
    }
    u64 X[kN2 / 2];
#pragma unroll
    for (int i = 0; i < kN2 / 2; ++i) X[i] = pack2(x[2 * i], x[2 * i + 1]);
#pragma unroll
    for (int s = 1; s < kStages; ++s) {
        const u64* nt2 = reinterpret_cast<const u64*>(&P.nt[s][0]);
        const u64* sn2 = reinterpret_cast<const u64*>(&P.sn[s][0]);
#pragma unroll
        for (int q2 = 0; q2 < kN2 / 4; ++q2) {
            const int q = 2 * q2, lo = ((q >> s) << (s + 1)) | (q & ((1 << s) - 1)), a = lo >> 1, b = a + (1 << (s - 1));
            const u64 nt = nt2[q2], sn = sn2[q2];
            X[a] = fma2(nt, X[b], X[a]);
            X[b] = fma2(sn, X[a], X[b]);
            X[a] = fma2(nt, X[b], X[a]);
        }
    }
#pragma unroll
    for (int i = 0; i < kN2 / 2; ++i) unpack2(X[i], x[2 * i], x[2 * i + 1]);
}

// A operand, K-major without swizzle: tile t holds rows m = 32 tau + p (position j = 4 p + t); element (m, k) sits at
// kASbo (m / 8) + 16 (m mod 8) + kALbo (k / 4) + 4 (k mod 4).
__device__ __forceinline__ void store_run(uint32_t a_base, int u, const float (&x)[kN2]) {
    const int tau = u / kN1, k = u - tau * kN1;
    const uint32_t base = a_base + (4 * tau) * kASbo + (k >> 2) * kALbo + (k & 3) * 4;
#pragma unroll
    for (int t = 0; t < 4; ++t) {
#pragma unroll
        for (int p = 0; p < 32; ++p)
            f4k::sts32(base + t * kATile + (p >> 3) * kASbo + (p & 7) * 16, to_tf32(x[4 * p + t]));
    }
}

__device__ __forceinline__ void butterfly_role(const Params& P, uint32_t smem, uint32_t bars, int* counter, int n_groups,
                                               int lane) {
    const int total = n_groups * kBatches;
    while (true) {
        int n = 0;
        if (lane == 0) n = atomicAdd(counter, 1);
        n = __shfl_sync(0xffffffffu, n, 0);
        if (n >= total) break;
        const int g = n / kBatches, u = 32 * (n - g * kBatches) + lane, stage = g & 1;
        bool ok = wait_or_fail(bars + 8 * (kBarInFull + stage), (g >> 1) & 1, P.status);
        if (!__all_sync(0xffffffffu, ok)) break;
        float x[kN2];
        load_run(smem + kInOff + stage * kInStageBytes + u * 128, u, x);
        butterfly128(P, x);
        if (g >= 1) {  // the tensor core must be done with the previous group's A operand
            ok = wait_or_fail(bars + 8 * (kBarMmaDone + ((g - 1) & 1)), ((g - 1) >> 1) & 1, P.status);
            if (!__all_sync(0xffffffffu, ok)) break;
        }
        store_run(smem + kAOff, u, x);
        fence_proxy_async();
        mbar_arrive(bars + 8 * kBarAFull);
    }
}

// ---- MMA + TMA thread ------------------------------------------------------------------------------------------
__device__ __forceinline__ void issue_load(const CUtensorMap* tmap, uint32_t smem, uint32_t bars, int g, int64_t token0) {
    const int stage = g & 1;
    const uint32_t bar = bars + 8 * (kBarInFull + stage), dst = smem + kInOff + stage * kInStageBytes;
    mbar_expect_tx(bar, kInStageBytes);
    tma_load_3d(dst, tmap, 0, 0, static_cast<int>(token0), bar);
    tma_load_3d(dst + kHalfBytes, tmap, 64, 0, static_cast<int>(token0), bar);
}

__device__ __forceinline__ void mma_role(const Params& P, const CUtensorMap* tmap, uint32_t smem, uint32_t bars,
                                         uint32_t tmem_base, int n_groups) {
    const int64_t stride = int64_t(kTok) * gridDim.x, first = int64_t(kTok) * blockIdx.x;
    if (n_groups > 0) issue_load(tmap, smem, bars, 0, first);
    if (n_groups > 1) issue_load(tmap, smem, bars, 1, first + stride);
    int committed = -1;
    for (int g = 0; g < n_groups; ++g) {
        if (!wait_or_fail(bars + 8 * kBarAFull, g & 1, P.status)) break;
        // every butterfly thread has read stage g & 1 (its loads precede its arrival): refill it
        if (g + 2 < n_groups) issue_load(tmap, smem, bars, g + 2, first + (g + 2) * stride);
        if (g >= 2 && !wait_or_fail(bars + 8 * (kBarDEmpty + (g & 1)), ((g >> 1) - 1) & 1, P.status)) break;
        tmem_fence_after();
#pragma unroll
        for (int t = 0; t < 4; ++t) {
#pragma unroll
            for (int s = 0; s < kKSteps; ++s) {
                const uint64_t adesc = smem_desc(smem + kAOff + t * kATile + 2 * s * kALbo, kALbo, kASbo);
                const uint64_t bdesc = smem_desc(smem + kBOff + s * kBBlock, 128, 256);
                mma_tf32(tmem_base + (g & 1) * (4 * kNPad) + t * kNPad, adesc, bdesc, s > 0 ? 1u : 0u);
            }
        }
        mma_commit(bars + 8 * (kBarMmaDone + (g & 1)));
        committed = g;
    }
    // drain: nothing of this CTA may be in flight when it leaves (both waits return at once on the normal path)
    if (committed >= 0) wait_or_fail(bars + 8 * (kBarMmaDone + (committed & 1)), (committed >> 1) & 1, P.status);
    for (int g = n_groups - 2; g < n_groups; ++g)
        if (g >= 0) wait_or_fail(bars + 8 * (kBarInFull + (g & 1)), (g >> 1) & 1, P.status);
}

// ---- epilogue warps: warp w = token w of the group = tensor-memory lanes 32 w .. 32 w + 31 -----------------------
// eight output runs i = 8 c .. 8 c + 7 of the four tiles: q[8 t + e] = Y~[i = 8 c + e][j = 4 p + t]
__device__ __forceinline__ void load_chunk(uint32_t taddr, int c, uint32_t (&q)[32]) {
#pragma unroll
    for (int t = 0; t < 4; ++t) tmem_ld8(taddr + t * kNPad + 8 * c, reinterpret_cast<uint32_t(&)[8]>(q[8 * t]));
    tmem_wait_ld32(q);
}

__device__ __forceinline__ void epilogue_role(const Params& P, uint32_t bars, uint32_t tmem_base, int n_groups, int w,
                                              int lane) {
    // pending signs of this thread's four positions j = 4 lane + t
    const uint32_t sbits = (P.sign[lane >> 3] >> (4 * (lane & 7))) & 0xFu;
    const uint32_t smask01 = ((sbits & 1u) ? 0x8000u : 0u) | ((sbits & 2u) ? 0x80000000u : 0u);
    const uint32_t smask23 = ((sbits & 4u) ? 0x8000u : 0u) | ((sbits & 8u) ? 0x80000000u : 0u);
    for (int g = 0; g < n_groups; ++g) {
        const int buf = g & 1;
        const bool ok = wait_or_fail(bars + 8 * (kBarMmaDone + buf), (g >> 1) & 1, P.status);
        if (!__all_sync(0xffffffffu, ok)) break;
        tmem_fence_after();
        const uint32_t taddr = tmem_base + (static_cast<uint32_t>(32 * w) << 16) + buf * (4 * kNPad);
        const int64_t token = int64_t(kTok) * (blockIdx.x + int64_t(g) * gridDim.x) + w;
        const bool valid = token < P.rows;
        uint32_t q[32];
        float inv = 0.f;
        bool saturated = false;
        if (P.codes != nullptr) {  // row absmax over all 5120 values, then the fp16 scale
            float amax = 0.f;
#pragma unroll 1
            for (int c = 0; c < kN1 / 8; ++c) {
                load_chunk(taddr, c, q);
#pragma unroll
                for (int e = 0; e < 32; ++e) amax = fmaxf(amax, fabsf(__uint_as_float(q[e])));
            }
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) amax = fmaxf(amax, __shfl_xor_sync(0xffffffffu, amax, o));
            const uint16_t sb = row_scale(amax, 7, &inv);
            // clamped or subnormal scale (its rounding error is not small), or an infinite / NaN row: keep the clamp
            saturated = sb == 0x7BFFu || sb < 0x0400u || !(amax < 3.0e38f);
            if (lane == 0 && valid) P.scales[token] = sb;
        }
        float inv_t[4];
#pragma unroll
        for (int t = 0; t < 4; ++t) inv_t[t] = ((sbits >> t) & 1u) ? -inv : inv;
#pragma unroll 1
        for (int c = 0; c < kN1 / 8; ++c) {
            load_chunk(taddr, c, q);
            if (c == kN1 / 8 - 1) {  // last read of this accumulator buffer: hand it back to the MMA thread
                tmem_fence_before();
                mbar_arrive(bars + 8 * (kBarDEmpty + buf));
            }
            if (P.y != nullptr && valid) {
#pragma unroll
                for (int e = 0; e < 8; ++e) {
                    uint2 o;
                    o.x = pack_bf16x2(__uint_as_float(q[e]), __uint_as_float(q[8 + e])) ^ smask01;
                    o.y = pack_bf16x2(__uint_as_float(q[16 + e]), __uint_as_float(q[24 + e])) ^ smask23;
                    *reinterpret_cast<uint2*>(P.y + token * P.ldy + (8 * c + e) * kN2 + 4 * lane) = o;
                }
            }
            if (P.codes != nullptr) {
                uint32_t hw[8];  // four 4-bit codes (j = 4 lane .. 4 lane + 3) of each of the eight runs
                if (!saturated) {
                    // |y / s| <= 7 (1 + 2^-10) < 7.5 when s is the row's own normal, unsaturated fp16 scale: no clamp needed;
                    // adding 1.5 * 2^23 + 8 rounds y * inv to the nearest integer r (ties to even, one rounding) and
                    // leaves r + 8 in [1, 15] in the low mantissa bits; the four biased codes are packed by
                    // multiply-adds and the bias is turned into two's complement by flipping bit 3 of every nibble
                    constexpr float kMagic = 12582920.0f;
                    constexpr uint32_t kUnbias = 0u - 0x4B400000u * 4369u;  // removes the bits of 1.5 * 2^23 from all four terms
#pragma unroll
                    for (int e = 0; e < 8; ++e) {
                        uint32_t acc = __float_as_uint(fmaf(__uint_as_float(q[e]), inv_t[0], kMagic));
                        acc += 16u * __float_as_uint(fmaf(__uint_as_float(q[8 + e]), inv_t[1], kMagic));
                        acc += 256u * __float_as_uint(fmaf(__uint_as_float(q[16 + e]), inv_t[2], kMagic));
                        acc += 4096u * __float_as_uint(fmaf(__uint_as_float(q[24 + e]), inv_t[3], kMagic));
                        hw[e] = ((acc + kUnbias) ^ 0x8888u) & 0xFFFFu;
                    }
                } else {
#pragma unroll
                    for (int e = 0; e < 8; ++e) {
                        hw[e] = 0u;
#pragma unroll
                        for (int t = 0; t < 4; ++t)
                            hw[e] |= (static_cast<uint32_t>(quant1(__uint_as_float(q[8 * t + e]), inv_t[t], -8, 7)) & 0xFu) << (4 * t);
                    }
                }
                // lanes 2 a and 2 a + 1 hold the two halves of one 32-bit word of every run: the even lane
                // assembles the word of run i, the odd lane that of run i + 1
                const bool odd = lane & 1;
#pragma unroll
                for (int e = 0; e < 8; e += 2) {
                    const uint32_t send = odd ? hw[e] : hw[e + 1];
                    const uint32_t recv = __shfl_xor_sync(0xffffffffu, send, 1);
                    const uint32_t word = odd ? (recv | (hw[e + 1] << 16)) : (hw[e] | (recv << 16));
                    const int i = 8 * c + e + (odd ? 1 : 0);
                    if (valid) *reinterpret_cast<uint32_t*>(P.codes + token * (kD / 2) + i * (kN2 / 2) + (lane >> 1) * 4) = word;
                }
            }
        }
    }
}

__global__ void __launch_bounds__(kThreads, 1)
k_comp5120(const __grid_constant__ Params P, const __grid_constant__ CUtensorMap tmap, int64_t total_groups) {
    extern __shared__ uint8_t smem_raw[];
    const uint32_t smem = (smem_u32(smem_raw) + 1023u) & ~1023u;
    uint8_t* const sm = smem_raw + (smem - smem_u32(smem_raw));
    const uint32_t bars = smem + kBarOff;
    uint32_t* const tmem_slot = reinterpret_cast<uint32_t*>(sm + kBarOff + 8 * kNumBars);
    int* const counter = reinterpret_cast<int*>(sm + kBarOff + 8 * kNumBars + 4);
    const int t = threadIdx.x, warp = t >> 5, lane = t & 31;
    const int n_groups =
        blockIdx.x < total_groups ? static_cast<int>((total_groups - blockIdx.x + gridDim.x - 1) / gridDim.x) : 0;

    if (t == 0) {
        mbar_init(bars + 8 * (kBarInFull + 0), 1);
        mbar_init(bars + 8 * (kBarInFull + 1), 1);
        mbar_init(bars + 8 * kBarAFull, kRuns);
        mbar_init(bars + 8 * (kBarMmaDone + 0), 1);
        mbar_init(bars + 8 * (kBarMmaDone + 1), 1);
        mbar_init(bars + 8 * (kBarDEmpty + 0), 32 * kEpiWarps);
        mbar_init(bars + 8 * (kBarDEmpty + 1), 32 * kEpiWarps);
        mbar_init_fence();
        *counter = 0;
    }
    __syncwarp();
    if (warp == 0) tmem_alloc512(smem_u32(tmem_slot));
    // B operand: Q1 rounded to TF32, K-major without swizzle, one block per k-step: row i (48 rows, the last eight
    // zero) and contraction index kq = k mod 8 sit at 256 (i / 8) + 16 (i mod 8) + 128 (kq / 4) + 4 (kq mod 4)
    for (int e = t; e < kNPad * kN1; e += kThreads) {
        const int i = e / kN1, k = e - i * kN1, kq = k & 7;
        const float v = i < kN1 ? P.q1[i * kN1 + k] : 0.f;
        *reinterpret_cast<uint32_t*>(sm + kBOff + (k >> 3) * kBBlock + 256 * (i >> 3) + 16 * (i & 7) + 128 * (kq >> 2) +
                                     4 * (kq & 3)) = to_tf32(v);
    }
    fence_proxy_async();
    tmem_fence_before();
    __syncthreads();
    tmem_fence_after();
    const uint32_t tmem_base = *tmem_slot;

    if (warp < kEpiWarps) {
        epilogue_role(P, bars, tmem_base, n_groups, warp, lane);
    } else if (warp < kMmaWarp) {
        butterfly_role(P, smem, bars, counter, n_groups, lane);
    } else if (lane == 0) {
        mma_role(P, &tmap, smem, bars, tmem_base, n_groups);
    }
    tmem_fence_before();
    __syncthreads();
    if (warp == 0) {
        tmem_fence_after();
        tmem_dealloc512(tmem_base);
    }
}

}  // namespace c5k

// ---- host side -----------------------------------------------------------------------------------------------------
// Lifting constants of Q2 from the angles (host, float64).  A rotation by psi with |psi| > pi/2 is minus a rotation by
// psi -+ pi; the minus signs are tracked per position (a pair whose two inputs carry opposite signs rotates by the
// negated angle and keeps its signs), and what is left after the last stage goes to Params::sign.
static void build_constants(const float* theta, c5k::Params* P) {
    using namespace c5k;
    const double pi = 3.14159265358979323846;
    int sign[kN2];
    for (int j = 0; j < kN2; ++j) sign[j] = 1;
    for (int s = 0; s < kStages; ++s) {
        for (int q = 0; q < kN2 / 2; ++q) {
            const int lo = ((q >> s) << (s + 1)) | (q & ((1 << s) - 1)), hi = lo + (1 << s);
            double psi = std::remainder(double(sign[lo] * sign[hi]) * double(theta[s * (kN2 / 2) + q]), 2.0 * pi);
            bool flip = false;
            if (psi > pi / 2) psi -= pi, flip = true;
            else if (psi < -pi / 2) psi += pi, flip = true;
            P->nt[s][q] = static_cast<float>(-std::tan(psi / 2));
            P->sn[s][q] = static_cast<float>(std::sin(psi));
            if (flip) sign[lo] = -sign[lo], sign[hi] = -sign[hi];
        }
    }
    for (int wd = 0; wd < 4; ++wd) P->sign[wd] = 0u;
    for (int j = 0; j < kN2; ++j)
        if (sign[j] < 0) P->sign[j >> 5] |= 1u << (j & 31);
}

bool comp5120_available(const bfq_plan* plan) {
    return plan->n == c5k::kN2 && plan->cc_major == 10 && plan->theta_host != nullptr && plan->comp5120 != nullptr &&
           encode_tiled() != nullptr;
}

size_t comp5120_param_bytes() { return sizeof(c5k::Params); }

// x: [rows][ldx] bf16 seen as {128 elements of a run, 40 runs, rows tokens}; a box is one 64-element half of every
// run of four tokens, 128-byte swizzled (line = 40 token + run)
static bool encode_token_map(CUtensorMap* tmap, const void* x, int64_t rows, int64_t ldx) {
    const cuuint64_t dims[3] = {c5k::kN2, c5k::kN1, static_cast<cuuint64_t>(rows)};
    const cuuint64_t strides[2] = {c5k::kN2 * 2, static_cast<cuuint64_t>(ldx) * 2};
    const cuuint32_t box[3] = {64, c5k::kN1, c5k::kTok};
    const cuuint32_t estr[3] = {1, 1, 1};
    return encode_tiled()(tmap, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void*>(x), dims, strides, box, estr,
                          CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
                          CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

cudaError_t comp5120_launch(bfq_plan* plan, const float* q1, const void* x, int64_t rows, int64_t ldx, uint8_t* codes,
                            uint16_t* scales, void* y_bf16, int64_t ldy, cudaStream_t st) {
    using namespace c5k;
    Params* P = static_cast<Params*>(plan->comp5120);
    if (!plan->comp5120_valid) {  // the angles' host copy was enqueued by bfq_set_angles: wait for it, once per angle set
        cudaError_t e = cudaEventSynchronize(plan->theta_event);
        if (e != cudaSuccess) return e;
        build_constants(plan->theta_host, P);
        plan->comp5120_valid = true;
    }
    P->q1 = q1, P->codes = codes, P->scales = scales, P->y = static_cast<__nv_bfloat16*>(y_bf16), P->ldy = ldy;
    P->rows = rows, P->status = plan->status_word;
    CUtensorMap tmap;
    if (!encode_token_map(&tmap, x, rows, ldx)) return cudaErrorInvalidValue;
    static bool attr_set[kMaxDevices] = {};
    if (!attr_set[plan->device]) {
        cudaError_t e = cudaFuncSetAttribute(k_comp5120, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBytes);
        if (e != cudaSuccess) return e;
        attr_set[plan->device] = true;
    }
    const int64_t total_groups = (rows + kTok - 1) / kTok;
    const int grid = static_cast<int>(total_groups < plan->sm_count ? total_groups : plan->sm_count);
    k_comp5120<<<grid, kThreads, kSmemBytes, st>>>(*P, tmap, total_groups);
    return cudaGetLastError();
}

}  // namespace bfq
