// Pieces shared by the tuned n = 4096 kernels: the thread-role layouts of the three 4-stage phases,
// the shared-memory regrouping layouts, the packed three-shear stage, and the tensor-map encoder.
#pragma once

#include <cuda.h>
#include <cuda_fp16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "bfq_ptx.cuh"

namespace bfq {
namespace f4k {
using namespace ptx;

constexpr int kN = 4096;
constexpr int kGroupThreads = 128;
constexpr int kInSlots = 2;                  // TMA ring depth per group
constexpr uint32_t kRowBytes = kN * 2;       // one bf16 row
constexpr uint32_t kExWords = 4128;          // padded fp32 row (see the layouts below)
constexpr uint32_t kExBytes = kExWords * 4;
constexpr int kCols = 416;                   // tensor-memory columns in use

__device__ __forceinline__ uint4 lds128(uint32_t a) {
    uint4 v;
    asm volatile("ld.shared.v4.u32 {%0,%1,%2,%3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "r"(a));
    return v;
}
__device__ __forceinline__ u64 lds64(uint32_t a) {
    u64 v;
    asm volatile("ld.shared.b64 %0, [%1];" : "=l"(v) : "r"(a));
    return v;
}
__device__ __forceinline__ uint32_t lds32(uint32_t a) {
    uint32_t v;
    asm volatile("ld.shared.u32 %0, [%1];" : "=r"(v) : "r"(a));
    return v;
}
__device__ __forceinline__ void sts32(uint32_t a, uint32_t v) {
    asm volatile("st.shared.u32 [%0], %1;" ::"r"(a), "r"(v) : "memory");
}
__device__ __forceinline__ void sts64(uint32_t a, u64 v) {
    asm volatile("st.shared.b64 [%0], %1;" ::"r"(a), "l"(v) : "memory");
}
// counters in shared memory: add without reading the result back
__device__ __forceinline__ void red_shared_inc(uint32_t a) {
    asm volatile("red.shared.add.u32 [%0], 1;" ::"r"(a) : "memory");
}
__device__ __forceinline__ void red_shared_add64(uint32_t a, u64 v) {
    asm volatile("red.shared.add.u64 [%0], %1;" ::"r"(a), "l"(v) : "memory");
}

// fp16 scale of a row from its absmax, like row_scale() of the generic kernels but with straight-line arithmetic: a / QMAX as
// q0 = a * r, q = fma(fma(-q0, QMAX, a), r, q0) with r = RN(1 / QMAX), which is the correctly rounded quotient for
// every non-negative finite a when QMAX is 1, 7 or 127 (checked exhaustively), and an approximate reciprocal (one
// unit in the last place) for the multiplier applied to the values.
template <int QMAX>
__device__ __forceinline__ uint16_t row_scale_fast(float amax, float* inv) {
    static_assert(QMAX == 1 || QMAX == 7 || QMAX == 127, "quotient checked for these divisors only");
    constexpr float r = 1.0f / QMAX;
    const float q0 = __fmul_rn(amax, r);
    const float sf = __fmaf_rn(__fmaf_rn(-q0, static_cast<float>(QMAX), amax), r, q0);
    const uint16_t bits = sf >= 65520.f ? static_cast<uint16_t>(0x7BFFu) : __half_as_ushort(__float2half_rn(sf));
    const float sc = __half2float(__ushort_as_half(bits));
    float rc;
    asm("rcp.approx.ftz.f32 %0, %1;" : "=f"(rc) : "f"(sc));
    *inv = sc > 0.f ? rc : 0.f;
    return bits;
}

// stores by one thread of a warp or group without a divergent branch around them
__device__ __forceinline__ void sts32_if(bool p, uint32_t a, uint32_t v) {
    asm volatile("{\n\t.reg .pred q;\n\tsetp.ne.u32 q, %0, 0;\n\t@q st.shared.u32 [%1], %2;\n\t}" ::"r"(static_cast<uint32_t>(p)),
                 "r"(a), "r"(v)
                 : "memory");
}
__device__ __forceinline__ void stg16_if(bool p, uint16_t* a, uint16_t v) {
    asm volatile("{\n\t.reg .pred q;\n\tsetp.ne.u32 q, %0, 0;\n\t@q st.global.u16 [%1], %2;\n\t}" ::"r"(static_cast<uint32_t>(p)),
                 "l"(a), "h"(v)
                 : "memory");
}
// the two bf16 halves of a word as fp32 bit patterns, on the integer pipe (a shift would go to the FP32 pipe as a
// multiply)
__device__ __forceinline__ uint32_t bf16_lo(uint32_t w) {
    uint32_t r;
    asm("prmt.b32 %0, %1, 0, 0x1044;" : "=r"(r) : "r"(w));
    return r;
}

constexpr int kTurnBar0 = 8;  // named barriers 8 .. 8 + G - 1 carry the tokens (1 .. G are the groups' own)

// The FP32 pipes and the shared-memory pipe are both heavily used; left alone, the row groups drift into step (all
// rotating, then all regrouping) and the pipes take turns idling.  The groups therefore pass tokens around: a group
// rotates (one phase of four stages) only while it holds a token and hands it on when it starts a regrouping or its
// epilogue, so that some groups' rotations overlap the others' memory phases.  A token is a named barrier per group:
// 128 arrivals from the previous holder + the 128 waiting threads.
struct Turn {
    int wait_id, pass_id;  // named barriers: this group's, the next group's in the ring
    bool on;
    __device__ __forceinline__ void acquire() const {
        if (on) bar_sync(wait_id, 2 * kGroupThreads);
    }
    __device__ __forceinline__ void pass() const {
        if (on) bar_arrive(pass_id, 2 * kGroupThreads);
    }
};

// ---- element held by role t, packed register m, half h in each phase -----------------------------------
//   phase 1: i = m | (t & 15) << 4 | h << 8 | (t >> 4) << 9
//   phase 2: i = (t & 15) | m << 4 | h << 8 | (t >> 4) << 9
//   phase 3: i = h | t << 1 | m << 8
// ---- shared-memory layouts of the two regroupings (word addresses; i = element index bits) -----------
// first:   A1 = i8 + 2*(i4..i7) + 32*(i9 + 2*i10 + 4*i11) + 258*(i0..i3)
// second:  A2 = (i0..i4) + 16*i9 + 32*(i5 + 2*i6 + 4*i7 + 8*i8 + 16*i10 + 32*i11 + 64*i9)
// Both are injective into [0, kExWords); a half-warp's 16 64-bit accesses and a warp's 32 scalar
// stores each cover the 32 banks exactly once.  In the first, the words a thread writes are read by
// the 16 lanes of its own half-warp only.
__device__ __forceinline__ constexpr uint32_t ex1_wr_local(int m) { return 4u * 258u * m; }
__device__ __forceinline__ constexpr uint32_t ex1_rd_local(int m) { return 4u * 2u * m; }
__device__ __forceinline__ constexpr uint32_t ex2_wr_local(int m, int h) {
    return 4u * (16u * (m & 1) + 32u * (m >> 1) + 256u * h);
}
__device__ __forceinline__ constexpr uint32_t ex2_rd_local(int m) {
    return 4u * (256u * (m & 1) + 2064u * ((m >> 1) & 1) + 512u * ((m >> 2) & 1) + 1024u * ((m >> 3) & 1));
}

// ---- one stage on the registers of a thread ---------------------------------------------------------
// Local stage K pairs packed registers m and m | 2^K; both fp32 lanes rotate at once.  T holds
// (nt, nt', sn, sn') for NU consecutive pairs starting at pair U0.  The three shears are issued level
// by level so that dependent instructions are NU apart.
template <int K, int U0, int NU, int CW>
__device__ __forceinline__ void stage_lift(u64 (&P)[16], const uint32_t (&T)[CW]) {
    static_assert(4 * NU <= CW, "chunk too small");
#pragma unroll
    for (int i = 0; i < NU; ++i) {
        const int u = U0 + i, m_lo = ((u >> K) << (K + 1)) | (u & ((1 << K) - 1)), m_hi = m_lo | (1 << K);
        P[m_lo] = fma2(pack2u(T[4 * i], T[4 * i + 1]), P[m_hi], P[m_lo]);
    }
#pragma unroll
    for (int i = 0; i < NU; ++i) {
        const int u = U0 + i, m_lo = ((u >> K) << (K + 1)) | (u & ((1 << K) - 1)), m_hi = m_lo | (1 << K);
        P[m_hi] = fma2(pack2u(T[4 * i + 2], T[4 * i + 3]), P[m_lo], P[m_hi]);
    }
#pragma unroll
    for (int i = 0; i < NU; ++i) {
        const int u = U0 + i, m_lo = ((u >> K) << (K + 1)) | (u & ((1 << K) - 1)), m_hi = m_lo | (1 << K);
        P[m_lo] = fma2(pack2u(T[4 * i], T[4 * i + 1]), P[m_hi], P[m_lo]);
    }
}

// The same stage as two independent FMAs per pair on implicitly scaled values: with true value = d * stored value and
// per-element factors d fixed by the angles alone (d' = cos(theta) * d for both elements of a pair),
//     lo' = lo + k1 * hi,   hi' = hi + k2 * lo      (both from the old values)
// is the rotation.  T holds (k1, k1', k2, k2') for NU consecutive pairs starting at pair U0; the factors are folded into
// k1, k2 when the tables are built and into the constants of the last stage, which is a general 2x2.
template <int K, int U0, int NU, int CW>
__device__ __forceinline__ void stage_scaled(u64 (&P)[16], const uint32_t (&T)[CW]) {
    static_assert(4 * NU <= CW, "chunk too small");
#pragma unroll
    for (int i = 0; i < NU; ++i) {
        const int u = U0 + i, m_lo = ((u >> K) << (K + 1)) | (u & ((1 << K) - 1)), m_hi = m_lo | (1 << K);
        const u64 a = P[m_lo], b = P[m_hi];
        P[m_lo] = fma2(pack2u(T[4 * i], T[4 * i + 1]), b, a);
        P[m_hi] = fma2(pack2u(T[4 * i + 2], T[4 * i + 3]), a, b);
    }
}

// sign carried by element i when it enters stage s: the product of the negations (flip = 1) of the pairs
// it belonged to in stages 0..s-1
__device__ __forceinline__ int sign_before(const uint8_t* __restrict__ flip, int i, int s) {
    // all (at most twelve) flag loads are issued together: a loop with a run-time trip count would wait for each in turn
    int f = 0;
#pragma unroll
    for (int sp = 0; sp < 12; ++sp) {
        const int j = ((i >> (sp + 1)) << sp) | (i & ((1 << sp) - 1));
        const int v = sp < s ? flip[sp * (kN / 2) + j] : 0;
        f ^= v;
    }
    return f ? -1 : 1;
}

// Walsh-Hadamard local stage K: (a, b) -> (a + b, a - b) on packed registers m and m | 2^K, no constants; the
// 1/sqrt(n) is applied later, once
template <int K>
__device__ __forceinline__ void stage_hadamard(u64 (&P)[16]) {
#pragma unroll
    for (int u = 0; u < 8; ++u) {
        const int m_lo = ((u >> K) << (K + 1)) | (u & ((1 << K) - 1)), m_hi = m_lo | (1 << K);
        const u64 a = P[m_lo], b = P[m_hi];
        P[m_lo] = add2(a, b);
        P[m_hi] = sub2(a, b);
    }
}

}  // namespace f4k

// ---- host side: launch that lets the kernel's set-up overlap the tail of the kernel before it in the stream ----
// (the kernel calls grid_dep_wait() before it touches global memory)
template <class... KArgs, class... Args>
static inline cudaError_t launch_overlapped(void (*kern)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t st,
                                            Args&&... args) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid, cfg.blockDim = block, cfg.dynamicSmemBytes = smem, cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr, cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, kern, static_cast<KArgs>(args)...);
}

// ---- host side: cuTensorMapEncodeTiled through the runtime's driver entry point ------------------------
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

static inline EncodeTiledFn encode_tiled() {
    static EncodeTiledFn fn = nullptr;
    static bool tried = false;
    if (!tried) {
        tried = true;
        void* sym = nullptr;
        cudaDriverEntryPointQueryResult qres;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &sym, cudaEnableDefault, &qres) == cudaSuccess &&
            qres == cudaDriverEntryPointSuccess) {
            fn = reinterpret_cast<EncodeTiledFn>(sym);
        }
    }
    return fn;
}


// 3-D map over bf16 rows of 4096: {64 elements, 64 lines, rows}, box = one row, 128-byte swizzle
static inline bool encode_row_map(CUtensorMap* tmap, const void* x, int64_t rows, int64_t ld) {
    const cuuint64_t dims[3] = {64, 64, static_cast<cuuint64_t>(rows)};
    const cuuint64_t strides[2] = {128, static_cast<cuuint64_t>(ld) * 2};
    const cuuint32_t box[3] = {64, 64, 1};
    const cuuint32_t estr[3] = {1, 1, 1};
    return encode_tiled()(tmap, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void*>(x), dims, strides, box, estr,
                          CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
                          CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// the same for fp32 rows: 128 lines of 32 elements per row (16 KB)
static inline bool encode_row_map_f32(CUtensorMap* tmap, const void* x, int64_t rows, int64_t ld) {
    const cuuint64_t dims[3] = {32, 128, static_cast<cuuint64_t>(rows)};
    const cuuint64_t strides[2] = {128, static_cast<cuuint64_t>(ld) * 4};
    const cuuint32_t box[3] = {32, 128, 1};
    const cuuint32_t estr[3] = {1, 1, 1};
    return encode_tiled()(tmap, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 3, const_cast<void*>(x), dims, strides, box, estr,
                          CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
                          CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

}  // namespace bfq
