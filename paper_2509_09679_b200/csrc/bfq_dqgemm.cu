// Dense products of the layer-calibration step on the tensor cores, with the low-bit operands dequantized on the fly:
//     C[i][j] = alpha * sum_k A(i, k) * B(j, k),   i < M, j < N, k < K
// where each operand is given as rows of fp32 / bf16 numbers or as packed two's-complement codes with one fp16 scale
// per stored row (the output format of bfq_forward_quant / bfq_fold_weights), stored either [rows][K] or transposed
// [K][rows].  This covers the three products of the reconstruction loss (paper Sec. 3.4):
//     Dequant(Quant(B x)) . Dequant(Quant(W B^T))^T,   err . Dequant(Quant(W B^T)),   err^T . Dequant(Quant(B x)).
//
// One CTA per 128 x 128 tile of C, K blocks of 64.  An operand tile in shared memory is 128 rows of 128 bytes (64 bf16)
// with the 128-byte swizzle, and every row is 64 elements that are CONTIGUOUS IN THE STORED OPERAND:
//   * stored [rows][K]: shared-memory row r = tile row r, 64 consecutive k (the K-major layout of the tensor core);
//   * stored [K][rows]: shared-memory row 64 h + k = stored row k0 + k, tile rows 64 h .. 64 h + 63 (the MN-major
//     layout: blocks of 64 tile rows 8192 bytes apart, groups of 8 k 1024 bytes apart).
// So one producer thread (eight producer warps: threads 0..127 for A, 128..255 for B) always turns 64 contiguous stored
// elements into one 128-byte row, with 16-byte loads and stores, whatever the orientation; the instruction descriptor
// tells the tensor core which layout each operand has.  Terms per operand:
//   * codes contracted along their stored row: the integer codes are exact in bf16 (one term); the row scale multiplies
//     the finished row / column of C;
//   * codes contracted across stored rows: the scale varies along k, so code x scale (at most 15 significant bits) is
//     stored as hi + lo, exactly;
//   * fp32 numbers: hi + lo = 16 significant bits (relative error 2^-17 per element); bf16 numbers: one term, exact.
// Codes become bf16 without integer-to-float conversions: a field u = code + 2^(b-1) OR-ed into the mantissa of 128.0
// is the bf16 number 128 + u, two fields per 32-bit word at a time, and one packed subtraction removes the offset.
// The global loads of the next K block are issued before the current one is converted.  One thread issues
// tcgen05.mma (kind::f16, M = N = 128, fp32 accumulators in tensor memory) for every pair of terms and commits to
// the stage's "empty" mbarrier; the ring has as many stages as fit 192 KB.  The producer warps then read the
// accumulators back (tcgen05.ld, a lane quarter and half of the columns each), apply alpha and the row / column
// scales and store fp32 rows of C.  Every wait is bounded and reports through the plan's status word.
#include "../../include/bfq.h"

#include <cuda_bf16.h>
#include <cuda_fp16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "bfq_plan.h"
#include "bfq_ptx.cuh"

namespace bfq {
namespace dqg {
using namespace ptx;

constexpr int kTile = 128;       // rows of A and of B per CTA
constexpr int kKB = 64;          // K block: one 128-byte swizzle atom of bf16
constexpr int kMaxStages = 6;
constexpr int kProducers = 256;  // threads 0..127 build A's tile, 128..255 B's; all run the epilogue; thread 256 issues the MMAs
constexpr uint32_t kTileBytes = kTile * kKB * 2;  // one bf16 term of one operand: 16 KB
constexpr uint32_t kRingBytes = 12 * kTileBytes;  // 192 KB of operand tiles
constexpr int kWaitLimit = 1 << 24;

struct Operand {
    const void* data;
    const uint16_t* scales;  // fp16 bits, one per stored row (codes only)
    int64_t ld;              // elements (numbers) or codes per stored row pitch
    int kind;                // BFQ_OP_*
    int transposed;          // 0: [rows][K], 1: [K][rows]
    int rows;                // M or N
};

__device__ __forceinline__ bool is_codes(int kind) { return kind >= BFQ_OP_CODES2; }
__host__ __device__ __forceinline__ int terms_of(int kind, int transposed) {
    if (kind == BFQ_OP_BF16) return 1;
    if (kind == BFQ_OP_F32) return 2;
    return transposed ? 2 : 1;
}
__host__ __device__ __forceinline__ int stages_of(int terms_a, int terms_b) {
    const int fit = 12 / (terms_a + terms_b);
    return fit < kMaxStages ? fit : kMaxStages;
}

__device__ __forceinline__ void fence_proxy_async() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ bool wait_bounded(uint32_t bar, uint32_t parity, int* status) {
    for (int i = 0; i < kWaitLimit; ++i) {
        if (mbar_try_wait(bar, parity)) return true;
    }
    atomicExch(status, 3);
    return false;
}
__device__ __forceinline__ void tmem_alloc128(uint32_t smem_dst) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], 128;" ::"r"(smem_dst) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_dealloc128(uint32_t taddr) {
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, 128;" ::"r"(taddr) : "memory");
}
// Shared-memory descriptor of a 128-byte-swizzled tile.  K-major operand: rows of 128 bytes, 8-row groups 1024 bytes
// apart (stride field), the leading field unused; one K step of 16 elements is 32 bytes further along the row.
// MN-major operand: rows of 128 bytes hold 64 tile rows for one k, groups of 8 k are 1024 bytes apart (stride field),
// blocks of 64 tile rows 8192 bytes apart (leading field); one K step of 16 is two groups = 2048 bytes further.
__device__ __forceinline__ uint64_t desc_sw128(uint32_t addr, uint32_t leading_bytes) {
    return static_cast<uint64_t>((addr & 0x3FFFFu) >> 4) | (static_cast<uint64_t>(leading_bytes >> 4) << 16) |
           (static_cast<uint64_t>(1024 >> 4) << 32) | (static_cast<uint64_t>(1) << 46) | (static_cast<uint64_t>(2) << 61);
}
// bf16 x bf16 -> fp32, M = 128, N = 128; bit 15 / 16: A / B is MN-major
__device__ __forceinline__ uint32_t make_idesc(int a_mn_major, int b_mn_major) {
    return (1u << 4) | (1u << 7) | (1u << 10) | (static_cast<uint32_t>(a_mn_major) << 15) |
           (static_cast<uint32_t>(b_mn_major) << 16) | (uint32_t(kTile >> 3) << 17) | (uint32_t(kTile >> 4) << 24);
}
__device__ __forceinline__ void mma_bf16(uint32_t d_tmem, uint64_t adesc, uint64_t bdesc, uint32_t idesc, uint32_t accumulate) {
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
        ::"r"(d_tmem), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate)
        : "memory");
}
__device__ __forceinline__ void mma_commit(uint32_t bar) {
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}

// ---- one shared-memory row: 64 elements that are contiguous in the stored operand -------------------------------
__device__ __forceinline__ void sts128(uint32_t at, uint32_t a, uint32_t b, uint32_t c, uint32_t d) {
    asm volatile("st.shared.v4.u32 [%0], {%1,%2,%3,%4};" ::"r"(at), "r"(a), "r"(b), "r"(c), "r"(d) : "memory");
}
__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi) {  // lo in bits 0..15
    const __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
    return *reinterpret_cast<const uint32_t*>(&v);
}
__device__ __forceinline__ uint32_t sub_bf16x2(uint32_t a, uint32_t b) {
    uint32_t d;
    asm("sub.bf16x2 %0, %1, %2;" : "=r"(d) : "r"(a), "r"(b));
    return d;
}
__device__ __forceinline__ uint32_t prmt(uint32_t a, uint32_t b, uint32_t sel) {
    uint32_t d;
    asm("prmt.b32 %0, %1, %2, %3;" : "=r"(d) : "r"(a), "r"(b), "r"(sel));
    return d;
}

// Where chunk j (16 bytes = 8 bf16) of shared-memory row `srow` of a tile goes
__device__ __forceinline__ uint32_t chunk_addr(uint32_t tile, int srow, int j) {
    return tile + static_cast<uint32_t>(srow) * 128u + static_cast<uint32_t>((j ^ (srow & 7)) << 4);
}

// two fp32 values -> their bf16 words (hi term, remainder term)
__device__ __forceinline__ void split2(float a, float b, uint32_t& hi, uint32_t& lo) {
    hi = pack_bf16(a, b);
    lo = pack_bf16(a - __uint_as_float(hi << 16), b - __uint_as_float(hi & 0xFFFF0000u));
}

// Raw 16-byte words of a row's 64 elements: fp32 16, bf16 8, 8-bit codes 4, 4-bit codes 2, 2-bit codes 1
template <int KIND>
struct RawWords {
    static constexpr int kCount = KIND == BFQ_OP_F32 ? 16 : (KIND == BFQ_OP_BF16 ? 8 : (KIND * 64) / 128);
};

// 8 codes of 4 bits (one word, element e in bits 4e..4e+3, two's complement) -> 4 words of bf16 pairs in element order
__device__ __forceinline__ void codes4_to_bf16(uint32_t w, uint32_t (&o)[4]) {
    const uint32_t x = w ^ 0x88888888u;  // u = code + 8
    // (128 + u_e, 128 + u_{e+4}) as a bf16 pair: the field sits in the low mantissa bits of 128.0 = 0x4300
    const uint32_t t0 = (x & 0x000F000Fu) | 0x43004300u, t1 = ((x >> 4) & 0x000F000Fu) | 0x43004300u;
    const uint32_t t2 = ((x >> 8) & 0x000F000Fu) | 0x43004300u, t3 = ((x >> 12) & 0x000F000Fu) | 0x43004300u;
    const uint32_t off = 0x43084308u;  // 136.0 twice
    const uint32_t c0 = sub_bf16x2(t0, off), c1 = sub_bf16x2(t1, off), c2 = sub_bf16x2(t2, off), c3 = sub_bf16x2(t3, off);
    o[0] = prmt(c0, c1, 0x5410u), o[1] = prmt(c2, c3, 0x5410u);  // elements (0,1), (2,3)
    o[2] = prmt(c0, c1, 0x7632u), o[3] = prmt(c2, c3, 0x7632u);  // elements (4,5), (6,7)
}
// 16 codes of 2 bits (one word) -> 8 words of bf16 pairs in element order
__device__ __forceinline__ void codes2_to_bf16(uint32_t w, uint32_t (&o)[8]) {
    const uint32_t x = w ^ 0xAAAAAAAAu;  // u = code + 2
    uint32_t c[8];                       // c[j] = (code_j, code_{j+8})
#pragma unroll
    for (int j = 0; j < 8; ++j) c[j] = sub_bf16x2(((x >> (2 * j)) & 0x00030003u) | 0x43004300u, 0x43024302u);
#pragma unroll
    for (int j = 0; j < 4; ++j) {
        o[j] = prmt(c[2 * j], c[2 * j + 1], 0x5410u);      // elements (2j, 2j+1)
        o[4 + j] = prmt(c[2 * j], c[2 * j + 1], 0x7632u);  // elements (8+2j, 9+2j)
    }
}
// 4 codes of 8 bits (one word) -> 2 words of bf16 pairs: byte u = code + 128 in the low mantissa bits of 2^23
__device__ __forceinline__ void codes8_to_bf16(uint32_t w, uint32_t (&o)[2]) {
    const uint32_t x = w ^ 0x80808080u;
    const float m = 8388736.0f;  // 2^23 + 128
    const float f0 = __uint_as_float(prmt(x, 0x4B000000u, 0x7440u)) - m, f1 = __uint_as_float(prmt(x, 0x4B000000u, 0x7441u)) - m;
    const float f2 = __uint_as_float(prmt(x, 0x4B000000u, 0x7442u)) - m, f3 = __uint_as_float(prmt(x, 0x4B000000u, 0x7443u)) - m;
    o[0] = pack_bf16(f0, f1), o[1] = pack_bf16(f2, f3);
}

struct Params {
    Operand a, b;
    float* c;
    int64_t ldc;
    int k;
    float alpha;
    int* status;
};

// zeroes the elements >= valid of the c-th chunk of a piece (its elements 8c .. 8c+7, two per word)
__device__ __forceinline__ void mask_chunk(uint32_t (&o)[4], int c, int valid) {
#pragma unroll
    for (int w = 0; w < 4; ++w) {
        const int e = 8 * c + 2 * w;
        o[w] = e >= valid ? 0u : (e + 1 >= valid ? (o[w] & 0xFFFFu) : o[w]);
    }
}

// One chunk (8 elements as 4 words of exact bf16 pairs) to chunk j of row `srow`: as it is, or times the scale in two
// terms.  c = which chunk of its piece this is (for the masking of a partial piece).
template <bool SCALED, bool PARTIAL>
__device__ __forceinline__ void store_bf16_chunk(uint32_t tile, int srow, int j, int c, uint32_t (&o)[4], float s, int valid) {
    if constexpr (PARTIAL) mask_chunk(o, c, valid);
    const uint32_t at = chunk_addr(tile, srow, j);
    if constexpr (!SCALED) {
        sts128(at, o[0], o[1], o[2], o[3]);
    } else {
        uint32_t hi[4], lo[4];
#pragma unroll
        for (int w = 0; w < 4; ++w) split2(__uint_as_float(o[w] << 16) * s, __uint_as_float(o[w] & 0xFFFF0000u) * s, hi[w], lo[w]);
        sts128(at, hi[0], hi[1], hi[2], hi[3]);
        sts128(at + kTileBytes, lo[0], lo[1], lo[2], lo[3]);
    }
}

// One raw 16-byte word = piece p of shared-memory row `srow` (the row's 64 elements are 128 / kPerWord pieces).
// SCALED (codes contracted across their stored rows): times `s`, two terms.  PARTIAL: only the first `valid` elements
// of the piece exist; the others are stored as zero.
template <int KIND, bool SCALED, bool PARTIAL>
__device__ __forceinline__ void convert_word(const uint4 raw, uint32_t tile, int srow, int p, float s, int valid) {
    if constexpr (KIND == BFQ_OP_F32) {
        // 4 numbers = half of chunk p / 2
        uint32_t hi[2], lo[2];
        split2(__uint_as_float(raw.x), __uint_as_float(raw.y), hi[0], lo[0]);
        split2(__uint_as_float(raw.z), __uint_as_float(raw.w), hi[1], lo[1]);
        if constexpr (PARTIAL) {
#pragma unroll
            for (int w = 0; w < 2; ++w) {
                const uint32_t m = 2 * w >= valid ? 0u : (2 * w + 1 >= valid ? 0xFFFFu : 0xFFFFFFFFu);
                hi[w] &= m, lo[w] &= m;
            }
        }
        const uint32_t at = chunk_addr(tile, srow, p >> 1) + 8u * (p & 1);
        asm volatile("st.shared.v2.u32 [%0], {%1,%2};" ::"r"(at), "r"(hi[0]), "r"(hi[1]) : "memory");
        asm volatile("st.shared.v2.u32 [%0], {%1,%2};" ::"r"(at + kTileBytes), "r"(lo[0]), "r"(lo[1]) : "memory");
    } else if constexpr (KIND == BFQ_OP_BF16) {
        uint32_t o[4] = {raw.x, raw.y, raw.z, raw.w};
        store_bf16_chunk<false, PARTIAL>(tile, srow, p, 0, o, 1.f, valid);
    } else if constexpr (KIND == BFQ_OP_CODES4) {
        const uint32_t ws[4] = {raw.x, raw.y, raw.z, raw.w};
#pragma unroll
        for (int w = 0; w < 4; ++w) {
            uint32_t o[4];
            codes4_to_bf16(ws[w], o);
            store_bf16_chunk<SCALED, PARTIAL>(tile, srow, 4 * p + w, w, o, s, valid);
        }
    } else if constexpr (KIND == BFQ_OP_CODES2) {
        const uint32_t ws[4] = {raw.x, raw.y, raw.z, raw.w};
#pragma unroll
        for (int w = 0; w < 4; ++w) {
            uint32_t o8[8];
            codes2_to_bf16(ws[w], o8);
            uint32_t oa[4] = {o8[0], o8[1], o8[2], o8[3]}, ob[4] = {o8[4], o8[5], o8[6], o8[7]};
            store_bf16_chunk<SCALED, PARTIAL>(tile, srow, 8 * p + 2 * w, 2 * w, oa, s, valid);
            store_bf16_chunk<SCALED, PARTIAL>(tile, srow, 8 * p + 2 * w + 1, 2 * w + 1, ob, s, valid);
        }
    } else {
        const uint32_t ws[4] = {raw.x, raw.y, raw.z, raw.w};
#pragma unroll
        for (int h = 0; h < 2; ++h) {
            uint32_t o2a[2], o2b[2];
            codes8_to_bf16(ws[2 * h], o2a);
            codes8_to_bf16(ws[2 * h + 1], o2b);
            uint32_t o[4] = {o2a[0], o2a[1], o2b[0], o2b[1]};
            store_bf16_chunk<SCALED, PARTIAL>(tile, srow, 2 * p + h, h, o, s, valid);
        }
    }
}

struct Ring {
    uint32_t sbase, stage_bytes, bar_full, bar_empty;
    int stages;
};

// Producer loop of one thread of the 128 that build one operand's tiles.  A K block of the operand is 128 shared-memory
// rows of kLpr 16-byte pieces; piece id = i * 128 + r (i = 0 .. kLpr - 1) is piece id % kLpr of row id / kLpr, so the
// lanes of a warp read consecutive pieces of the same stored row: global loads are coalesced as far as the stored row
// allows.  ACROSS: the operand is stored [K][rows]; shared-memory row 64 h + k is stored row k0 + k, tile rows
// 64 h .. 64 h + 63.
template <int KIND, bool ACROSS>
__device__ __forceinline__ bool produce(const Operand& op, int r, int tile_row0, uint32_t tile_off, const Ring& ring, int kblocks,
                                        int* status) {
    constexpr int kLpr = RawWords<KIND>::kCount;  // pieces per row = pieces per thread
    constexpr int kEbits = KIND == BFQ_OP_F32 ? 32 : (KIND == BFQ_OP_BF16 ? 16 : KIND);
    constexpr int kPerWord = 128 / kEbits;  // elements per piece
    constexpr bool kScaled = ACROSS && KIND >= BFQ_OP_CODES2;
    constexpr int kRowStep = kTile / kLpr;  // rows between a thread's consecutive pieces
    const int p = r % kLpr, row_first = r / kLpr;
    const uint8_t* const base = static_cast<const uint8_t*>(op.data);
    const int64_t pitch = op.ld * kEbits / 8;  // bytes of a stored row
    // per piece: how many of its elements exist (0: nothing is loaded) and where K block 0 of it starts
    auto srow_of = [&](int i) { return row_first + i * kRowStep; };
    auto valid_of = [&](int i) -> int {
        if constexpr (!ACROSS) {
            return tile_row0 + srow_of(i) < op.rows ? kPerWord : 0;
        } else {
            const int left = op.rows - (tile_row0 + 64 * (srow_of(i) >> 6) + p * kPerWord);
            return left < 0 ? 0 : (left > kPerWord ? kPerWord : left);
        }
    };
    auto src_of = [&](int i, int kb) -> const uint4* {
        if constexpr (!ACROSS) {
            return reinterpret_cast<const uint4*>(base + int64_t(tile_row0 + srow_of(i)) * pitch + int64_t(kb) * (kKB * kEbits / 8) + 16 * p);
        } else {
            const int sr = srow_of(i);
            return reinterpret_cast<const uint4*>(base + (int64_t(kb) * kKB + (sr & 63)) * pitch +
                                                  int64_t(tile_row0 + 64 * (sr >> 6)) * kEbits / 8 + 16 * p);
        }
    };
    auto load = [&](uint4 (&raw)[kLpr], float (&sc)[kLpr], int kb) {
#pragma unroll
        for (int i = 0; i < kLpr; ++i) {
            raw[i] = valid_of(i) > 0 ? __ldg(src_of(i, kb)) : make_uint4(0u, 0u, 0u, 0u);
            if constexpr (kScaled) sc[i] = __half2float(__ushort_as_half(__ldg(op.scales + kb * kKB + (srow_of(i) & 63))));
        }
    };
    // the raw words of the next kDepth K blocks are in flight while the current one is converted
    constexpr int kDepth = kLpr >= 16 ? 1 : (kLpr >= 8 ? 2 : 4);
    uint4 buf[kDepth + 1][kLpr];
    float sc[kDepth + 1][kScaled ? kLpr : 1];
    auto load_slot = [&](int d, int kb) {
        if constexpr (kScaled) {
            load(buf[d], sc[d], kb);
        } else {
            float none[kLpr];
            load(buf[d], none, kb);
        }
    };
#pragma unroll
    for (int d = 0; d < kDepth; ++d)
        if (d < kblocks) load_slot(d, d);
    int s = 0;
    uint32_t round = 0;  // how many times the ring has wrapped
    for (int kb = 0; kb < kblocks; ++kb) {
        if (kb + kDepth < kblocks) load_slot(kDepth, kb + kDepth);
        if (round > 0 && !wait_bounded(ring.bar_empty + 8 * s, (round - 1) & 1, status)) return false;
        const uint32_t tile = ring.sbase + s * ring.stage_bytes + tile_off;
#pragma unroll
        for (int i = 0; i < kLpr; ++i) {
            const int v = valid_of(i);
            const float si = kScaled ? sc[0][kScaled ? i : 0] : 1.f;
            if (v == kPerWord) {
                convert_word<KIND, kScaled, false>(buf[0][i], tile, srow_of(i), p, si, v);
            } else {
                convert_word<KIND, kScaled, true>(buf[0][i], tile, srow_of(i), p, si, v);
            }
        }
        fence_proxy_async();  // written through the generic proxy, read by the tensor core through the async one
        mbar_arrive(ring.bar_full + 8 * s);
#pragma unroll
        for (int d = 0; d < kDepth; ++d) {
#pragma unroll
            for (int i = 0; i < kLpr; ++i) {
                buf[d][i] = buf[d + 1][i];
                if constexpr (kScaled) sc[d][i] = sc[d + 1][i];
            }
        }
        if (++s == ring.stages) s = 0, ++round;
    }
    return true;
}

template <bool ACROSS>
__device__ __forceinline__ bool produce_kind(const Operand& op, int r, int tile_row0, uint32_t tile_off, const Ring& ring,
                                             int kblocks, int* status) {
    switch (op.kind) {
        case BFQ_OP_F32: return produce<BFQ_OP_F32, ACROSS>(op, r, tile_row0, tile_off, ring, kblocks, status);
        case BFQ_OP_BF16: return produce<BFQ_OP_BF16, ACROSS>(op, r, tile_row0, tile_off, ring, kblocks, status);
        case BFQ_OP_CODES2: return produce<BFQ_OP_CODES2, ACROSS>(op, r, tile_row0, tile_off, ring, kblocks, status);
        case BFQ_OP_CODES4: return produce<BFQ_OP_CODES4, ACROSS>(op, r, tile_row0, tile_off, ring, kblocks, status);
        default: return produce<BFQ_OP_CODES8, ACROSS>(op, r, tile_row0, tile_off, ring, kblocks, status);
    }
}

__global__ void __launch_bounds__(kProducers + 32, 1) k_dequant_gemm(const Params p) {
    extern __shared__ uint8_t smem_raw[];
    const uint32_t sbase = (smem_u32(smem_raw) + 1023u) & ~1023u;
    const int tid = threadIdx.x, warp = tid >> 5;
    const int ta = terms_of(p.a.kind, p.a.transposed), tb = terms_of(p.b.kind, p.b.transposed);
    Ring ring;
    ring.sbase = sbase;
    ring.stage_bytes = static_cast<uint32_t>(ta + tb) * kTileBytes;
    ring.stages = stages_of(ta, tb);
    const uint32_t bars = sbase + kRingBytes;  // full[6], empty[6], done, then the tensor-memory address
    ring.bar_full = bars, ring.bar_empty = bars + 8 * kMaxStages;
    const uint32_t bar_done = bars + 16 * kMaxStages, tmem_slot = bar_done + 8;

    if (warp == 0) tmem_alloc128(tmem_slot);
    if (tid == kProducers) {
        for (int s = 0; s < kMaxStages; ++s) {
            mbar_init(ring.bar_full + 8 * s, kProducers);
            mbar_init(ring.bar_empty + 8 * s, 1);
        }
        mbar_init(bar_done, 1);
        mbar_init_fence();
    }
    tmem_fence_before();
    __syncthreads();
    tmem_fence_after();
    uint32_t tmem_base;
    asm volatile("ld.shared.u32 %0, [%1];" : "=r"(tmem_base) : "r"(tmem_slot));

    const int m0 = blockIdx.x * kTile, n0 = blockIdx.y * kTile;
    const int kblocks = p.k / kKB;
    bool ok = true;

    if (tid < kProducers) {
        // ---- producers: threads 0..127 build A's tiles, 128..255 B's ----
        const bool for_a = tid < kTile;
        const int r = tid & (kTile - 1);
        const Operand& op = for_a ? p.a : p.b;
        const uint32_t tile_off = for_a ? 0u : static_cast<uint32_t>(ta) * kTileBytes;
        ok = op.transposed ? produce_kind<true>(op, r, for_a ? m0 : n0, tile_off, ring, kblocks, p.status)
                           : produce_kind<false>(op, r, for_a ? m0 : n0, tile_off, ring, kblocks, p.status);
        // ---- epilogue: accumulators -> alpha * row scale * column scale -> C ----
        if (ok) ok = wait_bounded(bar_done, 0, p.status);
        ok = __all_sync(0xFFFFFFFFu, ok);  // the tensor-memory loads below are warp-wide
        tmem_fence_after();
        if (ok) {
            // warp w reads lanes 32 (w & 3) .. +31 (rows of the tile) and columns 64 (w >> 2) .. +63
            const int ra = m0 + 32 * (warp & 3) + (tid & 31);
            const bool row_ok = ra < p.a.rows;
            float rs = p.alpha;
            if (row_ok && is_codes(p.a.kind) && !p.a.transposed) rs *= __half2float(__ushort_as_half(__ldg(p.a.scales + ra)));
            const bool col_scaled = is_codes(p.b.kind) && !p.b.transposed;
            float* crow = p.c + int64_t(row_ok ? ra : 0) * p.ldc + n0;
            const bool vec = (p.ldc & 3) == 0 && (reinterpret_cast<uintptr_t>(p.c) & 15u) == 0;
            const uint32_t tlane = tmem_base + (static_cast<uint32_t>((warp & 3) * 32) << 16);
            const int cbase = 64 * (warp >> 2);
            for (int c0 = cbase; c0 < cbase + 64; c0 += 32) {
                uint32_t acc[32];
                tmem_ld32(tlane + c0, acc);
                tmem_wait_ld32(acc);
                float out[32];
#pragma unroll
                for (int j = 0; j < 32; ++j) {
                    float cs = rs;
                    if (col_scaled && n0 + c0 + j < p.b.rows) cs *= __half2float(__ushort_as_half(__ldg(p.b.scales + n0 + c0 + j)));
                    out[j] = __uint_as_float(acc[j]) * cs;
                }
                if (!row_ok) continue;
                if (vec && n0 + c0 + 32 <= p.b.rows) {
#pragma unroll
                    for (int j = 0; j < 32; j += 4)
                        *reinterpret_cast<float4*>(crow + c0 + j) = make_float4(out[j], out[j + 1], out[j + 2], out[j + 3]);
                } else {
#pragma unroll
                    for (int j = 0; j < 32; ++j)
                        if (n0 + c0 + j < p.b.rows) crow[c0 + j] = out[j];
                }
            }
        }
    } else if (tid == kProducers) {
        // ---- one thread issues the MMAs: every pair of terms, four K steps of 16 per block ----
        const uint32_t idesc = make_idesc(p.a.transposed, p.b.transposed);
        const uint32_t a_step = p.a.transposed ? 2048u : 32u, b_step = p.b.transposed ? 2048u : 32u;
        const uint32_t a_lead = p.a.transposed ? 8192u : 16u, b_lead = p.b.transposed ? 8192u : 16u;
        int s = 0;
        uint32_t round = 0;
        for (int kb = 0; kb < kblocks; ++kb) {
            ok = wait_bounded(ring.bar_full + 8 * s, round & 1, p.status);
            if (!ok) break;
            tmem_fence_after();
            const uint32_t at = sbase + s * ring.stage_bytes, bt = at + ta * kTileBytes;
            for (int ia = 0; ia < ta; ++ia)
                for (int ib = 0; ib < tb; ++ib)
#pragma unroll
                    for (int ks = 0; ks < kKB / 16; ++ks)
                        mma_bf16(tmem_base, desc_sw128(at + ia * kTileBytes + ks * a_step, a_lead),
                                 desc_sw128(bt + ib * kTileBytes + ks * b_step, b_lead), idesc, (kb | ia | ib | ks) != 0 ? 1u : 0u);
            mma_commit(ring.bar_empty + 8 * s);  // arrives when the MMAs issued so far have read their operands and finished
            if (++s == ring.stages) s = 0, ++round;
        }
        if (ok) mma_commit(bar_done);
    }
    tmem_fence_before();
    __syncthreads();
    if (warp == 0) tmem_dealloc128(tmem_base);
}

}  // namespace dqg
}  // namespace bfq

extern "C" int bfq_dequant_gemm(bfq_plan* plan, int64_t m, int64_t n, int64_t k, float alpha, const void* a, int a_kind,
                                int a_transposed, int64_t lda, const uint16_t* a_scales, const void* b, int b_kind,
                                int b_transposed, int64_t ldb, const uint16_t* b_scales, float* c, int64_t ldc, void* stream) {
    using namespace bfq::dqg;
    if (plan == nullptr) return BFQ_ERR_NULL;
    if (m < 0 || n < 0 || k < 0 || k % kKB != 0 || m >= (int64_t(1) << 31) || n >= (int64_t(1) << 31) || k >= (int64_t(1) << 31))
        return BFQ_ERR_STRIDE;
    if (m == 0 || n == 0) return BFQ_OK;
    if (a == nullptr || b == nullptr || c == nullptr) return BFQ_ERR_NULL;
    auto check = [&](const void* data, int kind, int transposed, int64_t ld, const uint16_t* scales, int64_t rows) -> int {
        const bool codes = kind == BFQ_OP_CODES2 || kind == BFQ_OP_CODES4 || kind == BFQ_OP_CODES8;
        if (!codes && kind != BFQ_OP_F32 && kind != BFQ_OP_BF16) return BFQ_ERR_DTYPE;
        if (codes && scales == nullptr) return BFQ_ERR_NULL;
        if ((reinterpret_cast<uintptr_t>(data) & 15u) != 0) return BFQ_ERR_ALIGN;
        const int64_t width = transposed ? rows : k;  // elements of a stored row in use
        if (ld < width) return BFQ_ERR_STRIDE;
        const int ebits = kind == BFQ_OP_F32 ? 32 : (kind == BFQ_OP_BF16 ? 16 : kind);
        if ((ld * ebits) % 128 != 0) return BFQ_ERR_STRIDE;  // stored rows start on 16-byte boundaries
        return BFQ_OK;
    };
    int rc = check(a, a_kind, a_transposed, lda, a_scales, m);
    if (rc == BFQ_OK) rc = check(b, b_kind, b_transposed, ldb, b_scales, n);
    if (rc != BFQ_OK) return rc;
    if (ldc < n || (reinterpret_cast<uintptr_t>(c) & 3u) != 0) return BFQ_ERR_STRIDE;
    int prev = -1;
    if (cudaGetDevice(&prev) != cudaSuccess) return BFQ_ERR_CUDA;
    if (prev != plan->device && cudaSetDevice(plan->device) != cudaSuccess) return BFQ_ERR_CUDA;
    cudaError_t e = cudaSuccess;
    if (k == 0) {
        e = cudaMemset2DAsync(c, size_t(ldc) * 4, 0, size_t(n) * 4, size_t(m), static_cast<cudaStream_t>(stream));
    } else {
        constexpr size_t smem = size_t(kRingBytes) + 8 * (2 * kMaxStages + 1) + 16 + 1024;
        static bool attr_set[bfq::kMaxDevices] = {false};
        if (!attr_set[plan->device]) {
            e = cudaFuncSetAttribute(k_dequant_gemm, cudaFuncAttributeMaxDynamicSharedMemorySize, int(smem));
            attr_set[plan->device] = (e == cudaSuccess);
        }
        if (e == cudaSuccess) {
            Params p;
            p.a = Operand{a, a_scales, lda, a_kind, a_transposed, int(m)};
            p.b = Operand{b, b_scales, ldb, b_kind, b_transposed, int(n)};
            p.c = c, p.ldc = ldc, p.k = int(k), p.alpha = alpha, p.status = plan->status_word;
            const dim3 grid(unsigned((m + kTile - 1) / kTile), unsigned((n + kTile - 1) / kTile));
            k_dequant_gemm<<<grid, kProducers + 32, smem, static_cast<cudaStream_t>(stream)>>>(p);
            e = cudaGetLastError();
        }
    }
    if (prev != plan->device) cudaSetDevice(prev);
    if (e != cudaSuccess) {
        plan->last_cuda_error = static_cast<int>(e);
        return BFQ_ERR_CUDA;
    }
    return BFQ_OK;
}
