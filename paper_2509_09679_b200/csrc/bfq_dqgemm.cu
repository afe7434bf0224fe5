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
constexpr int kStages = 2;
constexpr int kProducers = 256;  // threads 0..127 build A's tile rows, 128..255 B's; all run the epilogue; thread 256 issues the MMAs
constexpr uint32_t kTileBytes = kTile * kKB * 2;  // one bf16 term of one operand: 16 KB
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
// K-major, 128-byte swizzle: rows of 128 bytes, 8-row groups 1024 bytes apart; the start address advances by 32 bytes
// per 16-element K step inside the atom
__device__ __forceinline__ uint64_t desc_sw128(uint32_t addr) {
    return static_cast<uint64_t>((addr & 0x3FFFFu) >> 4) | (static_cast<uint64_t>(1) << 16) |
           (static_cast<uint64_t>(1024 >> 4) << 32) | (static_cast<uint64_t>(1) << 46) | (static_cast<uint64_t>(2) << 61);
}
// bf16 x bf16 -> fp32, both operands K-major, M = 128, N = 128
constexpr uint32_t kIdesc = (1u << 4) | (1u << 7) | (1u << 10) | (uint32_t(kTile >> 3) << 17) | (uint32_t(kTile >> 4) << 24);
__device__ __forceinline__ void mma_bf16(uint32_t d_tmem, uint64_t adesc, uint64_t bdesc, uint32_t accumulate) {
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
        ::"r"(d_tmem), "l"(adesc), "l"(bdesc), "r"(kIdesc), "r"(accumulate)
        : "memory");
}
__device__ __forceinline__ void mma_commit(uint32_t bar) {
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}

// ---- one tile row: 64 consecutive k of operand row `row` (already checked < op.rows), as fp32 ----------------
__device__ __forceinline__ float code_value(uint32_t byte, int shift, int bits) {
    const int q = static_cast<int>((byte >> shift) & ((1u << bits) - 1u));
    return static_cast<float>(q >= (1 << (bits - 1)) ? q - (1 << bits) : q);
}

// codes along the stored row: element k in bits [BITS (k mod 8/BITS), +BITS) of byte k BITS / 8, 16-byte loads; the
// row's scale is applied to the finished row of C
template <int BITS>
__device__ __forceinline__ void codes_along(const Operand& op, int row, int k0, float (&v)[kKB]) {
    const uint4* p = reinterpret_cast<const uint4*>(static_cast<const uint8_t*>(op.data) + (int64_t(row) * op.ld + k0) * BITS / 8);
    constexpr int kPerWord = 32 / BITS;
#pragma unroll
    for (int i = 0; i < kKB * BITS / 128; ++i) {
        const uint4 w4 = __ldg(p + i);
        const uint32_t ws[4] = {w4.x, w4.y, w4.z, w4.w};
#pragma unroll
        for (int j = 0; j < 4; ++j)
#pragma unroll
            for (int e = 0; e < kPerWord; ++e) {
                // sign-extend the field: shift it to the top of the word, then arithmetic shift back
                const int q = static_cast<int>(ws[j] << (32 - BITS * (e + 1))) >> (32 - BITS);
                v[(4 * i + j) * kPerWord + e] = static_cast<float>(q);
            }
    }
}
// codes across stored rows: stored row k0 + k holds this tile row's code in its column `row`; the stored row's scale
// varies along k and is applied here (code x fp16 scale is exact in fp32)
template <int BITS>
__device__ __forceinline__ void codes_across(const Operand& op, int row, int k0, float (&v)[kKB]) {
    const int64_t pitch = op.ld * BITS / 8;
    const uint8_t* p = static_cast<const uint8_t*>(op.data) + int64_t(k0) * pitch + (int64_t(row) * BITS >> 3);
    const int shift = (row * BITS) & 7;
#pragma unroll
    for (int k = 0; k < kKB; ++k) {
        const float s = __half2float(__ushort_as_half(__ldg(op.scales + k0 + k)));
        v[k] = s * code_value(__ldg(p + int64_t(k) * pitch), shift, BITS);
    }
}

__device__ __forceinline__ void load_row(const Operand& op, int row, int k0, float (&v)[kKB]) {
    if (!op.transposed) {
        if (op.kind == BFQ_OP_F32) {
            const float4* p = reinterpret_cast<const float4*>(static_cast<const float*>(op.data) + int64_t(row) * op.ld + k0);
#pragma unroll
            for (int i = 0; i < kKB / 4; ++i) {
                const float4 f = __ldg(p + i);
                v[4 * i] = f.x, v[4 * i + 1] = f.y, v[4 * i + 2] = f.z, v[4 * i + 3] = f.w;
            }
        } else if (op.kind == BFQ_OP_BF16) {
            const uint4* p = reinterpret_cast<const uint4*>(static_cast<const __nv_bfloat16*>(op.data) + int64_t(row) * op.ld + k0);
#pragma unroll
            for (int i = 0; i < kKB / 8; ++i) {
                const uint4 w = __ldg(p + i);
                const uint32_t ws[4] = {w.x, w.y, w.z, w.w};
#pragma unroll
                for (int j = 0; j < 4; ++j) {
                    v[8 * i + 2 * j] = __uint_as_float(ws[j] << 16);
                    v[8 * i + 2 * j + 1] = __uint_as_float(ws[j] & 0xFFFF0000u);
                }
            }
        } else if (op.kind == BFQ_OP_CODES2) {
            codes_along<2>(op, row, k0, v);
        } else if (op.kind == BFQ_OP_CODES4) {
            codes_along<4>(op, row, k0, v);
        } else {
            codes_along<8>(op, row, k0, v);
        }
    } else {
        if (op.kind == BFQ_OP_F32) {
            const float* p = static_cast<const float*>(op.data) + int64_t(k0) * op.ld + row;
#pragma unroll
            for (int k = 0; k < kKB; ++k) v[k] = __ldg(p + int64_t(k) * op.ld);
        } else if (op.kind == BFQ_OP_BF16) {
            const uint16_t* p = static_cast<const uint16_t*>(op.data) + int64_t(k0) * op.ld + row;
#pragma unroll
            for (int k = 0; k < kKB; ++k) v[k] = __uint_as_float(static_cast<uint32_t>(__ldg(p + int64_t(k) * op.ld)) << 16);
        } else if (op.kind == BFQ_OP_CODES2) {
            codes_across<2>(op, row, k0, v);
        } else if (op.kind == BFQ_OP_CODES4) {
            codes_across<4>(op, row, k0, v);
        } else {
            codes_across<8>(op, row, k0, v);
        }
    }
}

// 64 fp32 values of tile row r -> `terms` bf16 tiles (hi, then the rounding remainder) in the swizzled layout:
// 16-byte chunk j of row r sits at chunk j ^ (r & 7) of its 128-byte line; 8-row groups are 1024 bytes apart
__device__ __forceinline__ void store_row(uint32_t tile, int r, int terms, const float (&v)[kKB]) {
    const uint32_t line = tile + (r >> 3) * 1024u + (r & 7) * 128u;
#pragma unroll
    for (int j = 0; j < kKB / 8; ++j) {
        uint32_t hi[4], lo[4];
#pragma unroll
        for (int e = 0; e < 4; ++e) {
            const float a = v[8 * j + 2 * e], b = v[8 * j + 2 * e + 1];
            const __nv_bfloat16 ah = __float2bfloat16_rn(a), bh = __float2bfloat16_rn(b);
            hi[e] = static_cast<uint32_t>(__bfloat16_as_ushort(ah)) | (static_cast<uint32_t>(__bfloat16_as_ushort(bh)) << 16);
            if (terms == 2) {  // the rounding remainder, for operands that are not exact in one bf16 term
                const __nv_bfloat16 al = __float2bfloat16_rn(a - __bfloat162float(ah)), bl = __float2bfloat16_rn(b - __bfloat162float(bh));
                lo[e] = static_cast<uint32_t>(__bfloat16_as_ushort(al)) | (static_cast<uint32_t>(__bfloat16_as_ushort(bl)) << 16);
            }
        }
        const uint32_t at = line + ((j ^ (r & 7)) << 4);
        asm volatile("st.shared.v4.u32 [%0], {%1,%2,%3,%4};" ::"r"(at), "r"(hi[0]), "r"(hi[1]), "r"(hi[2]), "r"(hi[3]) : "memory");
        if (terms == 2)
            asm volatile("st.shared.v4.u32 [%0], {%1,%2,%3,%4};" ::"r"(at + kTileBytes), "r"(lo[0]), "r"(lo[1]), "r"(lo[2]), "r"(lo[3])
                         : "memory");
    }
}

struct Params {
    Operand a, b;
    float* c;
    int64_t ldc;
    int k;
    float alpha;
    int* status;
};

__global__ void __launch_bounds__(kProducers + 32, 1) k_dequant_gemm(const Params p) {
    extern __shared__ uint8_t smem_raw[];
    const uint32_t sbase = (smem_u32(smem_raw) + 1023u) & ~1023u;
    const int tid = threadIdx.x, warp = tid >> 5;
    const int ta = terms_of(p.a.kind, p.a.transposed), tb = terms_of(p.b.kind, p.b.transposed);
    const uint32_t stage_bytes = static_cast<uint32_t>(ta + tb) * kTileBytes;
    const uint32_t bars = sbase + kStages * 4 * kTileBytes;  // full[2], empty[2], done, then the tensor-memory address
    const uint32_t bar_full = bars, bar_empty = bars + 8 * kStages, bar_done = bars + 16 * kStages, tmem_slot = bar_done + 8;

    if (warp == 0) tmem_alloc128(tmem_slot);
    if (tid == kProducers) {
        for (int s = 0; s < kStages; ++s) {
            mbar_init(bar_full + 8 * s, kProducers);
            mbar_init(bar_empty + 8 * s, 1);
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
        // ---- producers: thread = one tile row of A (threads 0..127) or of B (128..255) ----
        const bool for_a = tid < kTile;
        const int r = tid & (kTile - 1);
        const Operand& op = for_a ? p.a : p.b;
        const int row = (for_a ? m0 : n0) + r;
        const int terms = for_a ? ta : tb;
        float v[kKB];
        for (int kb = 0; kb < kblocks && ok; ++kb) {
            const int s = kb & 1;
            if (kb >= kStages) ok = wait_bounded(bar_empty + 8 * s, ((kb >> 1) - 1) & 1, p.status);
            if (!ok) break;
            const uint32_t tile = sbase + s * stage_bytes + (for_a ? 0u : ta * kTileBytes);
            if (row < op.rows) {
                load_row(op, row, kb * kKB, v);
            } else {
#pragma unroll
                for (int k = 0; k < kKB; ++k) v[k] = 0.f;
            }
            store_row(tile, r, terms, v);
            fence_proxy_async();  // the tiles were written through the generic proxy, the tensor core reads them through the async one
            mbar_arrive(bar_full + 8 * s);
        }
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
            const uint32_t tlane = tmem_base + (static_cast<uint32_t>((warp & 3) * 32) << 16);
            const int cbase = 64 * (warp >> 2);
            for (int c0 = cbase; c0 < cbase + 64; c0 += 32) {
                uint32_t acc[32];
                tmem_ld32(tlane + c0, acc);
                tmem_wait_ld32(acc);
#pragma unroll
                for (int j = 0; j < 32; ++j) {
                    const int col = n0 + c0 + j;
                    if (row_ok && col < p.b.rows) {
                        float cs = 1.f;
                        if (col_scaled) cs = __half2float(__ushort_as_half(__ldg(p.b.scales + col)));
                        crow[c0 + j] = __uint_as_float(acc[j]) * rs * cs;
                    }
                }
            }
        }
    } else if (tid == kProducers) {
        // ---- one thread issues the MMAs: every pair of terms, four K steps of 16 per block ----
        for (int kb = 0; kb < kblocks && ok; ++kb) {
            const int s = kb & 1;
            ok = wait_bounded(bar_full + 8 * s, (kb >> 1) & 1, p.status);
            if (!ok) break;
            tmem_fence_after();
            const uint32_t at = sbase + s * stage_bytes, bt = at + ta * kTileBytes;
            for (int ia = 0; ia < ta; ++ia)
                for (int ib = 0; ib < tb; ++ib)
#pragma unroll
                    for (int ks = 0; ks < kKB / 16; ++ks)
                        mma_bf16(tmem_base, desc_sw128(at + ia * kTileBytes + ks * 32), desc_sw128(bt + ib * kTileBytes + ks * 32),
                                 (kb | ia | ib | ks) != 0 ? 1u : 0u);
            mma_commit(bar_empty + 8 * s);  // arrives when the MMAs issued so far have read their operands and finished
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
        constexpr size_t smem = size_t(kStages) * 4 * kTileBytes + 8 * (2 * kStages + 1) + 16 + 1024;
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
