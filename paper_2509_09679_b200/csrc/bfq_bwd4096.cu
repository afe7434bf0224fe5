// Tuned backward pass for n = 4096 bf16 rows on sm_100a:  dx = Q^T g  and  d-theta summed over rows.
//
// One persistent CTA per SM works on two rows at a time (row pair p of the CTA is rows 2p, 2p+1) with two
// groups of 128 threads.  The upper group recomputes y for a pair and takes the reverse walk through stages 11, 10
// and 9 (which need no regrouping: their partners are in the thread's own registers); y and g then change hands through
// shared memory and the lower group walks stages 8 .. 0 and writes dx, while the upper group is already on the next
// pair.  The split balances the two groups' arithmetic (12 + 3 against 9 stage-equivalents of rotations, the lower
// group also carrying both regroupings).  Each group owns the d-theta accumulators of its stages.  The thread roles,
// phases and regrouping layouts are those of the forward kernel (bfq_n4096.cuh).  Per row pair:
//   1. y = Q x with the three-shear constants, all 12 stages, in the tracked-sign basis sigma.
//   2. y and g are moved to the basis sigma * (-1)^popcount(index).  Any two indices that a stage pairs
//      differ in one bit, so in this basis the high element of every pair of every stage is negated
//      relative to the low one, and there the inverse of a stage's rotation is the SAME three shears
//      with the SAME constants.  The reverse walk therefore reuses the forward tables unchanged.
//   3. for s = 11..0:  d[s][pair] += g_hi*y_lo - g_lo*y_hi on the stage's outputs (the stage-output
//      form of g^T (dG/dtheta) z; its sign in this basis is fixed per pair and applied when the sums
//      are written out), then y and g are both un-rotated.  After stage 0, g is dx up to the parity sign.
// d-theta accumulators are owned by thread role (no atomics): stages 0-7 in the tensor-memory columns the
// constants leave free, stages 8-11 in shared memory (stage 8 the lower group's, 9-11 the upper group's).  Each CTA walks its row pairs in a fixed order and
// writes its sums to its own slot; a second kernel adds the slots in a fixed order: bit-reproducible.
#include <type_traits>

#include "bfq_fast.h"
#include "bfq_generic.cuh"
#include "bfq_n4096.cuh"

namespace bfq {
namespace b4k {
using namespace ptx;
using namespace f4k;

constexpr int kThreads = 128;                // one group; the CTA has two (reverse = threads 0..127, forward = 128..255)
constexpr int kCtaThreads = 2 * kThreads;
constexpr int kSlots = 2;                    // TMA ring depth (row pairs), x and g rings separately
constexpr int kBarRev = 1, kBarFwd = 2, kBarFull = 3, kBarEmpty = 4;  // named barriers
constexpr int kConstCols = 384;              // 12 stages x 32 words
constexpr int kAccCol = 384;                 // accumulators of stages 0..7: 16 columns each
constexpr int kUpperSteps = 8;               // half-stage steps of the reverse walk done by the upper group: stages 11 .. 8
constexpr uint32_t kPairBytes = 2 * kRowBytes;  // two bf16 rows
constexpr int kWideCol = 416;  // wide inverse: (cos, +-sin) of the stage that joins the halves, 64 columns behind either table
constexpr int kInvCols = 416;  // scaled inverse: stages 11..1 (32 columns each, stage s at 32 (s - 1)), then stage 0 (64)
enum : int { kFormScaled = 0, kFormShear = 1 };

struct Smem {
    static constexpr uint32_t kXOff = 0;                                   // [kSlots][2][kRowBytes]
    static constexpr uint32_t kGOff = kXOff + kSlots * kPairBytes;         // [kSlots][2][kRowBytes]
    static constexpr uint32_t kExFOff = kGOff + kSlots * kPairBytes;       // upper group, forward recompute: [2][kExBytes]
    // y0, y1, g0, g1 of a row pair in the regrouping layouts: written by the upper group after stage 8 (this is both
    // the phase-3 -> phase-2 regrouping and the hand-off), re-used by the lower group for the regrouping after stage 4
    static constexpr uint32_t kExROff = kExFOff + 2 * kExBytes;            // [4][kExBytes]
    static constexpr uint32_t kAccOff = kExROff + 4 * kExBytes;            // [16][128] float4: stages 8..11
    static constexpr uint32_t kBarOff = kAccOff + 16 * kThreads * 16;      // mbarriers, one per input slot
    static constexpr uint32_t kTmemOff = kBarOff + 8 * 2 * kSlots;
    static constexpr uint32_t kUsed = kTmemOff + 16;
    static constexpr uint32_t kBytes = kUsed + 1024;
    // wide mode only: the upper group's sums of the stage that joins the halves, [16][128] packed pairs
    static constexpr uint32_t kAcc12Off = (kUsed + 15u) & ~15u;
    static constexpr uint32_t kBytesWide = kAcc12Off + 16 * kThreads * 8 + 1024;
};
static_assert(Smem::kBytesWide <= 232448, "shared memory budget of one CTA");
constexpr int kSlotFloats = 12 * (kN / 2);            // one CTA's sums of stages 0 .. 11
constexpr int kSlotFloatsWide = kSlotFloats + kN;     // ... followed by its share of stage 12's (wide mode)

__device__ __forceinline__ void sts128(uint32_t a, uint4 v) {
    asm volatile("st.shared.v4.u32 [%0], {%1,%2,%3,%4};" ::"r"(a), "r"(v.x), "r"(v.y), "r"(v.z), "r"(v.w) : "memory");
}

struct Addr {
    uint32_t w1, r1, w2, r2;  // per-thread byte offsets inside a regrouping buffer (forward write / read sides)
    uint32_t ex;              // base of the group's regrouping buffers
    int bar;                  // the group's named barrier
};

// ---- regroupings: forward direction (phase 1 -> 2 -> 3) and back, one row array at a time -------------
__device__ __forceinline__ void fwd1_store(const u64 (&P)[16], uint32_t buf, const Addr& a) {
#pragma unroll
    for (int m = 0; m < 16; ++m) sts64(buf + a.w1 + ex1_wr_local(m), P[m]);
}
__device__ __forceinline__ void fwd1_load(u64 (&P)[16], uint32_t buf, const Addr& a) {
#pragma unroll
    for (int m = 0; m < 16; ++m) P[m] = lds64(buf + a.r1 + ex1_rd_local(m));
}
__device__ __forceinline__ void fwd2_store(const u64 (&P)[16], uint32_t buf, const Addr& a) {
#pragma unroll
    for (int m = 0; m < 16; ++m) {
        uint32_t lo, hi;
        unpack2u(P[m], lo, hi);
        sts32(buf + a.w2 + ex2_wr_local(m, 0), lo);
        sts32(buf + a.w2 + ex2_wr_local(m, 1), hi);
    }
}
__device__ __forceinline__ void fwd2_load(u64 (&P)[16], uint32_t buf, const Addr& a) {
#pragma unroll
    for (int m = 0; m < 16; ++m) P[m] = lds64(buf + a.r2 + ex2_rd_local(m));
}
// back from phase 3 to phase 2: the phase-3 owner stores whole packed registers where it read them,
// the phase-2 owner reads scalars where it wrote them
__device__ __forceinline__ void rev2_store(const u64 (&P)[16], uint32_t buf, const Addr& a) {
#pragma unroll
    for (int m = 0; m < 16; ++m) sts64(buf + a.r2 + ex2_rd_local(m), P[m]);
}
__device__ __forceinline__ void rev2_load(u64 (&P)[16], uint32_t buf, const Addr& a) {
#pragma unroll
    for (int m = 0; m < 16; ++m)
        P[m] = pack2u(lds32(buf + a.w2 + ex2_wr_local(m, 0)), lds32(buf + a.w2 + ex2_wr_local(m, 1)));
}
__device__ __forceinline__ void rev1_store(const u64 (&P)[16], uint32_t buf, const Addr& a) {
#pragma unroll
    for (int m = 0; m < 16; ++m) sts64(buf + a.r1 + ex1_rd_local(m), P[m]);
}
__device__ __forceinline__ void rev1_load(u64 (&P)[16], uint32_t buf, const Addr& a) {
#pragma unroll
    for (int m = 0; m < 16; ++m) P[m] = lds64(buf + a.w1 + ex1_wr_local(m));
}

// ---- d-theta of four pairs (U0..U0+3) of local stage K, both rows:  A[i] += g_hi*y_lo - g_lo*y_hi ------
template <int K, int U0>
__device__ __forceinline__ void dtheta4(u64 (&A)[4], const u64 (&Y0)[16], const u64 (&Y1)[16], const u64 (&G0)[16],
                                        const u64 (&G1)[16]) {
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        const int u = U0 + i, m_lo = ((u >> K) << (K + 1)) | (u & ((1 << K) - 1)), m_hi = m_lo | (1 << K);
        u64 neg = mul2(G0[m_lo], Y0[m_hi]);
        neg = fma2(G1[m_lo], Y1[m_hi], neg);
        u64 pos = fma2(G0[m_hi], Y0[m_lo], A[i]);
        pos = fma2(G1[m_hi], Y1[m_lo], pos);
        A[i] = sub2(pos, neg);
    }
}

struct Ctx {
    Addr a;
    uint32_t tlane;     // tensor-memory address of this thread's lane, column 0
    uint32_t acc_smem;  // this thread's first float4 of the shared-memory accumulators
};

// ---- forward recompute: 24 chunks of 16 constants (two per stage), both rows ---------------------------
// Chunk C is in Tcur; the next chunk is requested right after the wait.
template <int C>
__device__ __forceinline__ void fwd_chunks(u64 (&X0)[16], u64 (&X1)[16], uint32_t (&Tcur)[16], uint32_t (&Tnext)[16],
                                           const Ctx& cx) {
    constexpr int s = C / 2, K = s & 3, U0 = 4 * (C & 1);
    tmem_wait_ld16(Tcur);
    if constexpr (C + 1 < 24) tmem_ld16(cx.tlane + 16 * (C + 1), Tnext);
    stage_lift<K, U0, 4, 16>(X0, Tcur);
    stage_lift<K, U0, 4, 16>(X1, Tcur);
    if constexpr (C == 7) {  // inside each half-warp; the group-wide hand-off barrier of the previous row pair
                             // has put every other warp past its reads of these buffers
        fwd1_store(X0, cx.a.ex + 0 * kExBytes, cx.a);
        fwd1_store(X1, cx.a.ex + 1 * kExBytes, cx.a);
        __syncwarp();
        fwd1_load(X0, cx.a.ex + 0 * kExBytes, cx.a);
        fwd1_load(X1, cx.a.ex + 1 * kExBytes, cx.a);
    }
    if constexpr (C == 15) {
        bar_sync(cx.a.bar, kThreads);  // every warp of the group is past its reads of the first layout
        fwd2_store(X0, cx.a.ex + 0 * kExBytes, cx.a);
        fwd2_store(X1, cx.a.ex + 1 * kExBytes, cx.a);
        bar_sync(cx.a.bar, kThreads);
        fwd2_load(X0, cx.a.ex + 0 * kExBytes, cx.a);
        fwd2_load(X1, cx.a.ex + 1 * kExBytes, cx.a);
    }
    if constexpr (C + 1 < 24) fwd_chunks<C + 1>(X0, X1, Tnext, Tcur, cx);
}

// ---- reverse walk: step I handles half c = I & 1 of stage s = 11 - I / 2 ---------------------------------
template <int I>
struct RevStep {
    static constexpr int s = 11 - I / 2, c = I & 1, K = s & 3, U0 = 4 * c;
    static constexpr uint32_t kTCol = 32 * s + 16 * c;
    static constexpr bool kAccInTmem = s < 8;
    static constexpr uint32_t kAccCol = b4k::kAccCol + 16 * s + 8 * c;       // stages 0..7
    static constexpr uint32_t kAccSmem = ((s - 8) * 4 + 2 * c) * kThreads * 16;  // stages 8..11: two float4
};

// steps I .. END-1 (END = 24: down to stage 0); hook(integral_constant<I>) runs after step I (regroupings, hand-off)
template <int I, int END, class F>
__device__ __forceinline__ void rev_steps(u64 (&Y0)[16], u64 (&Y1)[16], u64 (&G0)[16], u64 (&G1)[16],
                                          uint32_t (&Tcur)[16], uint32_t (&Tnext)[16], uint32_t (&Acur)[8],
                                          uint32_t (&Anext)[8], const Ctx& cx, F&& hook) {
    using S = RevStep<I>;
    if constexpr (S::kAccInTmem) {
        tmem_wait_ld16_8(Tcur, Acur);
    } else {
        tmem_wait_ld16(Tcur);
        const uint4 a0 = lds128(cx.acc_smem + S::kAccSmem), a1 = lds128(cx.acc_smem + S::kAccSmem + kThreads * 16);
        Acur[0] = a0.x, Acur[1] = a0.y, Acur[2] = a0.z, Acur[3] = a0.w;
        Acur[4] = a1.x, Acur[5] = a1.y, Acur[6] = a1.z, Acur[7] = a1.w;
    }
    if constexpr (I + 1 < END) {
        using N = RevStep<I + 1>;
        tmem_ld16(cx.tlane + N::kTCol, Tnext);
        if constexpr (N::kAccInTmem) tmem_ld8(cx.tlane + N::kAccCol, Anext);
    }
    {
        u64 A[4];
#pragma unroll
        for (int i = 0; i < 4; ++i) A[i] = pack2u(Acur[2 * i], Acur[2 * i + 1]);
        dtheta4<S::K, S::U0>(A, Y0, Y1, G0, G1);
#pragma unroll
        for (int i = 0; i < 4; ++i) unpack2u(A[i], Acur[2 * i], Acur[2 * i + 1]);
    }
    if constexpr (S::kAccInTmem) {
        tmem_st8(cx.tlane + S::kAccCol, Acur);
    } else {
        sts128(cx.acc_smem + S::kAccSmem, make_uint4(Acur[0], Acur[1], Acur[2], Acur[3]));
        sts128(cx.acc_smem + S::kAccSmem + kThreads * 16, make_uint4(Acur[4], Acur[5], Acur[6], Acur[7]));
    }
    if constexpr (S::s > 0) {  // y below stage 0 is x again: not needed
        stage_lift<S::K, S::U0, 4, 16>(Y0, Tcur);
        stage_lift<S::K, S::U0, 4, 16>(Y1, Tcur);
    }
    stage_lift<S::K, S::U0, 4, 16>(G0, Tcur);
    stage_lift<S::K, S::U0, 4, 16>(G1, Tcur);
    hook(std::integral_constant<int, I>());
    if constexpr (I + 1 < END) rev_steps<I + 1, END>(Y0, Y1, G0, G1, Tnext, Tcur, Anext, Acur, cx, hook);
}

__device__ __forceinline__ uint32_t cvt_bf16x2(float lo, float hi) {
    uint32_t r;
    asm("cvt.rn.bf16x2.f32 %0, %1, %2;" : "=r"(r) : "f"(hi), "f"(lo));
    return r;
}

// element index of (phase P, role t, packed register m, half h)
__device__ __forceinline__ int elem_of(int P, int t, int m, int h) {
    if (P == 0) return m | ((t & 15) << 4) | (h << 8) | ((t >> 4) << 9);
    if (P == 1) return (t & 15) | (m << 4) | (h << 8) | ((t >> 4) << 9);
    return h | (t << 1) | (m << 8);
}

// IN_F32: x, g and dx are fp32.  A row pair of x and of g then fills the whole input ring (one slot of 64 KB instead of
// two of 32 KB): the next pair is requested as soon as the upper group has read g, behind a barrier of that group.
// WIDE (bf16 rows): the launch handles half `half` of n = 8192 rows, i.e. stages 0 .. 11 of that half, whose tables it
// is given.  x rows are the half's 4096 elements (the tensor map starts there); g rows are whole 8192-element rows (16 KB),
// and the gradient that enters the half is the transposed stage-12 rotation of the two halves of g, formed as g is read:
// g'_own = c g_own +- s g_other with (cos, sin) of stage 12 from `tw12`.  dx is written at column 4096 * half.  One input
// slot, as for fp32 rows.  Stage 12's sums g_hi y_lo - g_lo y_hi are the same expression in g' and the halves' outputs
// z before that stage (a rotation keeps the cross product of two vectors), so each launch adds its share while both are
// in registers: half 0 has z_lo and forms g'_hi, half 1 has z_hi and forms g'_lo; the upper group keeps these sums in
// shared memory and the CTA's slot of `partial` is kSlotFloatsWide long (sign of the share included).
// what the CTAs of the upper half use in the wide mode instead of xmap, img, gsign, dsign
struct alignas(64) WideHalf {
    CUtensorMap xmap;
    const float* img;
    const uint32_t* gsign;
    const int8_t* dsign;
};

template <bool IN_F32, bool WIDE = false>
__global__ void __launch_bounds__(kCtaThreads, 1)
k_bwd4096(const __grid_constant__ CUtensorMap xmap, const __grid_constant__ CUtensorMap gmap,
          const float* __restrict__ img_lo, const uint32_t* __restrict__ gsign_lo, const int8_t* __restrict__ dsign_lo,
          void* __restrict__ dx_out, int64_t ld, float* __restrict__ partial, int rows, int* __restrict__ status,
          const float2* __restrict__ tw12, const __grid_constant__ WideHalf upper) {
    static_assert(!(IN_F32 && WIDE), "the wide mode takes bf16 rows");
    // wide mode: even CTAs work on the lower halves of the rows, odd CTAs on the upper halves (CTAs 2i and 2i + 1 take
    // the same row pairs at about the same time, so the second read of a g row comes from L2)
    const int ctas = WIDE ? int(gridDim.x >> 1) : int(gridDim.x);
    const int half = WIDE ? int(blockIdx.x & 1u) : 0;
    const CUtensorMap* const xm = (WIDE && half) ? &upper.xmap : &xmap;
    const float* const img = (WIDE && half) ? upper.img : img_lo;
    const uint32_t* const gsign = (WIDE && half) ? upper.gsign : gsign_lo;
    const int8_t* const dsign = (WIDE && half) ? upper.dsign : dsign_lo;
    // (only dereferenced when dx_out is not null)
    __nv_bfloat16* const dx = static_cast<__nv_bfloat16*>(dx_out) + (WIDE && dx_out != nullptr ? 4096 * half : 0);
    using S = Smem;
    extern __shared__ uint8_t smem_raw[];
    const uint32_t sbase = (smem_u32(smem_raw) + 1023u) & ~1023u;
    const int warp = threadIdx.x >> 5;
    const int t = threadIdx.x & (kThreads - 1);      // role 0..127
    const bool is_fwd = threadIdx.x >= kThreads;     // warps 4..7 recompute y, warps 0..3 walk back
    const int quarter = warp & 3;                    // tensor-memory lane quarter of this warp

    if (warp == 0) tmem_alloc512(sbase + S::kTmemOff);
    if (threadIdx.x < 2 * kSlots) {
        mbar_init(sbase + S::kBarOff + 8 * threadIdx.x, 1);
        mbar_init_fence();
    }
    tmem_fence_before();
    __syncthreads();
    tmem_fence_after();
    uint32_t tmem_base;
    asm volatile("ld.shared.u32 %0, [%1];" : "=r"(tmem_base) : "r"(sbase + S::kTmemOff));

    Ctx cx;
    cx.tlane = tmem_base + (static_cast<uint32_t>(quarter * 32) << 16);
    cx.acc_smem = sbase + S::kAccOff + t * 16;
    {
        const uint32_t t4 = (t >> 4) & 1, t5 = (t >> 5) & 1, t6 = (t >> 6) & 1;
        cx.a.ex = sbase + (is_fwd ? S::kExFOff : S::kExROff);  // the group's own regrouping buffers
        cx.a.bar = is_fwd ? kBarFwd : kBarRev;
        cx.a.w1 = 4u * (2u * (t & 15) + 32u * (t >> 4));
        cx.a.r1 = 4u * (258u * (t & 15) + 32u * (t >> 4));
        cx.a.w2 = 4u * ((t & 15) + 2064u * t4 + 512u * t5 + 1024u * t6);
        cx.a.r2 = 4u * (2u * (t & 15) + 32u * (t >> 4));
    }

    const int pairs = (rows + 1) / 2;
    const int first = WIDE ? int(blockIdx.x >> 1) : int(blockIdx.x);
    const int stride = ctas;
    const int count = first < pairs ? (pairs - first + stride - 1) / stride : 0;
    // both input rings belong to the upper group: one mbarrier per slot counts the x pair and the g pair
    const uint32_t xring = sbase + S::kXOff, gring = sbase + S::kGOff;
    const uint32_t bar_base = sbase + S::kBarOff;

    // a row index past the end is legal for the tensor map: the tile is filled with zeros
    constexpr bool kOneSlot = IN_F32 || WIDE;
    constexpr int kSlotsUsed = kOneSlot ? 1 : kSlots;
    constexpr uint32_t kInRow = IN_F32 ? 2 * kRowBytes : kRowBytes;                // bytes of one x row
    constexpr uint32_t kGRow = (IN_F32 || WIDE) ? 2 * kRowBytes : kRowBytes;       // bytes of one g row
    static_assert(kSlots == 2, "an fp32 / wide row pair takes both bf16 slots of a ring");
    auto request = [&](int k) {
        const int slot = kOneSlot ? 0 : (k & 1);
        const int r0 = 2 * (first + k * stride);
        const uint32_t bar = bar_base + 8 * slot;
        mbar_expect_tx(bar, 2 * kInRow + 2 * kGRow);
        tma_load_3d(xring + slot * kPairBytes, xm, 0, 0, r0, bar);
        tma_load_3d(xring + slot * kPairBytes + kInRow, xm, 0, 0, r0 + 1, bar);
        tma_load_3d(gring + slot * kPairBytes, &gmap, 0, 0, r0, bar);
        tma_load_3d(gring + slot * kPairBytes + kGRow, &gmap, 0, 0, r0 + 1, bar);
    };
    if (is_fwd && t == 0) {
        for (int k = 0; k < kSlotsUsed && k < count; ++k) request(k);
    }
    // constants into tensor memory (each group fills half of the columns), accumulators to zero
    {
        const float4* src = reinterpret_cast<const float4*>(img + t * kConstCols);
        for (int c = is_fwd ? 16 : 0; c < kConstCols; c += 32) {
            uint32_t v[16];
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                const float4 f = __ldg(src + (c >> 2) + i);
                v[4 * i + 0] = __float_as_uint(f.x), v[4 * i + 1] = __float_as_uint(f.y);
                v[4 * i + 2] = __float_as_uint(f.z), v[4 * i + 3] = __float_as_uint(f.w);
            }
            tmem_st16(cx.tlane + c, v);
        }
        if (!is_fwd) {
            uint32_t z[16];
#pragma unroll
            for (int i = 0; i < 16; ++i) z[i] = 0u;
            for (int c = kAccCol; c < 512; c += 16) tmem_st16(cx.tlane + c, z);
            for (int q = 0; q < 16; ++q) sts128(cx.acc_smem + q * kThreads * 16, make_uint4(0u, 0u, 0u, 0u));
        } else if constexpr (WIDE) {
            for (int m = 0; m < 16; ++m) sts64(sbase + S::kAcc12Off + (m * kThreads + t) * 8, 0ull);
        }
        tmem_wait_st();
    }
    tmem_fence_before();
    __syncthreads();
    tmem_fence_after();

    // parity of the role: popcount(t) & 1
    const uint32_t par_t = __popc(t) & 1;
    const uint32_t sgn_a = par_t ? 0x80000000u : 0u, sgn_b = par_t ? 0u : 0x80000000u;
    const uint32_t exr = sbase + S::kExROff;  // where a row pair changes hands

    u64 Y0[16], Y1[16], G0[16], G1[16];
    uint32_t T0[16], T1[16], A0[8], A1[8];
    if (is_fwd) {
        // ================= upper group: y = Q x, then d-theta and the reverse walk of stages 11, 10, 9 =================
        // x tile, phase-1 ownership (as in the forward kernel)
        // (fp32: runs of 64 bytes at byte 64 (t & 15) + 2048 (t >> 4) + 1024 h: chunks 4 (t & 1) + c of line
        // ((t & 15) >> 1) + 16 (t >> 4) + 8 h)
        const uint32_t in_line = IN_F32 ? ((t & 15) >> 1) * 128u + (t >> 4) * 2048u : ((t >> 2) & 3) * 128u + (t >> 4) * 1024u;
        const uint32_t in_x = IN_F32 ? ((((t & 1) << 2) ^ ((t >> 1) & 7)) << 4) : ((((t & 3) << 1) ^ ((t >> 2) & 3)) << 4);
        // fp32 g: elements 2t + 256m, +1 are the 8-byte word t & 1 of chunk (t & 15) >> 1 of line (t >> 4) + 8m
        const uint32_t f_a = (t >> 4) * 128u + ((((t & 15) >> 1) ^ (t >> 4)) << 4) + (t & 1) * 8u;
        // g tile, phase-3 ownership: the 32-bit word of elements 2t + 256m, 2t + 256m + 1 is word t & 3 of
        // 16-byte chunk (t & 31) >> 2 of 128-byte line (t >> 5) + 4m; the swizzle moves the chunk to
        // chunk ^ (line & 7)
        const uint32_t g_x = (((t & 31) >> 2) ^ (t >> 5));
        const uint32_t g_a0 = (t >> 5) * 128u + (g_x << 4) + (t & 3) * 4u;
        const uint32_t g_a1 = (t >> 5) * 128u + ((g_x ^ 4u) << 4) + (t & 3) * 4u;
        const uint4* gsv = reinterpret_cast<const uint4*>(gsign);
        for (int k = 0; k < count; ++k) {
            const int slot = kOneSlot ? 0 : (k & 1);
            // every thread of this group is past its reads of the other input slot (each iteration ends in a
            // barrier with the lower group)
            if (!kOneSlot && t == 0 && k >= 1 && k + 1 < count) request(k + 1);
            tmem_ld16(cx.tlane, T0);
            mbar_wait_bounded(bar_base + 8 * slot, (kOneSlot ? k : (k >> 1)) & 1, status);
#pragma unroll
            for (int r = 0; r < 2; ++r) {
                u64(&X)[16] = r == 0 ? Y0 : Y1;
                const uint32_t src = xring + slot * kPairBytes + r * kInRow + in_line;
                if constexpr (IN_F32) {
                    uint4 w[2][4];
#pragma unroll
                    for (int h = 0; h < 2; ++h)
#pragma unroll
                        for (int c = 0; c < 4; ++c) w[h][c] = lds128(src + 1024u * h + (in_x ^ (c << 4)));
#pragma unroll
                    for (int c = 0; c < 4; ++c) {
                        X[4 * c + 0] = pack2u(w[0][c].x, w[1][c].x);
                        X[4 * c + 1] = pack2u(w[0][c].y, w[1][c].y);
                        X[4 * c + 2] = pack2u(w[0][c].z, w[1][c].z);
                        X[4 * c + 3] = pack2u(w[0][c].w, w[1][c].w);
                    }
                    continue;
                }
                uint4 w[2][2];
#pragma unroll
                for (int h = 0; h < 2; ++h)
#pragma unroll
                    for (int c = 0; c < 2; ++c) w[h][c] = lds128(src + 512u * h + (in_x ^ ((c | (h << 2)) << 4)));
#pragma unroll
                for (int c = 0; c < 2; ++c) {
                    const uint32_t a[4] = {w[0][c].x, w[0][c].y, w[0][c].z, w[0][c].w};
                    const uint32_t b[4] = {w[1][c].x, w[1][c].y, w[1][c].z, w[1][c].w};
#pragma unroll
                    for (int j = 0; j < 4; ++j) {
                        X[8 * c + 2 * j + 0] = pack2u(bf16_lo(a[j]), bf16_lo(b[j]));
                        X[8 * c + 2 * j + 1] = pack2u(a[j] & 0xFFFF0000u, b[j] & 0xFFFF0000u);
                    }
                }
            }
            fwd_chunks<0>(Y0, Y1, T0, T1, cx);
            // y to the parity basis
#pragma unroll
            for (int m = 0; m < 16; ++m) {
                const bool odd = (__builtin_popcount(m) & 1) != 0;  // compile-time after unrolling
                const u64 mask = odd ? pack2u(sgn_b, sgn_a) : pack2u(sgn_a, sgn_b);
                Y0[m] ^= mask;
                Y1[m] ^= mask;
            }
            // g into the same basis
            tmem_ld16(cx.tlane + RevStep<0>::kTCol, T0);
            if constexpr (WIDE) {
                // elements 2t + 256m, +1 of both halves of the row (the upper half is 8192 bytes further on, the same
                // line modulo 8) and (cos, sin) of the two stage-12 pairs they form; y carries the signs of the walk's basis
                // here, the sign of each sum is put right when the sums are written out
                const float sg = half ? -1.f : 1.f;
                const uint32_t acc12 = sbase + S::kAcc12Off + t * 8;
                const uint32_t src = gring;
#pragma unroll
                for (int qq = 0; qq < 4; ++qq) {
                    const uint4 sw = __ldg(gsv + qq * kThreads + t);
                    const uint32_t s4[4] = {sw.x, sw.y, sw.z, sw.w};
#pragma unroll
                    for (int i = 0; i < 4; ++i) {
                        const int m = 4 * qq + i;
                        const float4 cs = __ldg(reinterpret_cast<const float4*>(tw12 + 2 * t + 256 * m));
                        const u64 c2 = pack2(cs.x, cs.z), s2 = pack2(sg * cs.y, sg * cs.w), ns2 = pack2(-sg * cs.y, -sg * cs.w);
                        u64 acc = lds64(acc12 + m * kThreads * 8);
#pragma unroll
                        for (int r = 0; r < 2; ++r) {
                            u64(&G)[16] = r == 0 ? G0 : G1;
                            const u64(&Y)[16] = r == 0 ? Y0 : Y1;
                            const uint32_t at = src + r * kGRow + ((m & 1) ? g_a1 : g_a0) + 512u * m;
                            const uint32_t wo = lds32(at + 8192u * half), wx = lds32(at + 8192u * (half ^ 1));
                            const u64 own = pack2u(bf16_lo(wo), wo & 0xFFFF0000u), oth = pack2u(bf16_lo(wx), wx & 0xFFFF0000u);
                            acc = fma2(fma2(ns2, own, mul2(c2, oth)), Y[m], acc);
                            uint32_t lo, hi;
                            unpack2u(fma2(s2, oth, mul2(c2, own)), lo, hi);
                            G[m] = pack2u(lo ^ ((s4[i] & 0x8000u) << 16), hi ^ (s4[i] & 0x80000000u));
                        }
                        sts64(acc12 + m * kThreads * 8, acc);
                    }
                }
            }
#pragma unroll
            for (int r = 0; r < (WIDE ? 0 : 2); ++r) {
                u64(&G)[16] = r == 0 ? G0 : G1;
                const uint32_t src = gring + slot * kPairBytes + r * kGRow;
#pragma unroll
                for (int qq = 0; qq < 4; ++qq) {
                    const uint4 sw = __ldg(gsv + qq * kThreads + t);  // 2 KB in all: stays in L1
                    const uint32_t s4[4] = {sw.x, sw.y, sw.z, sw.w};
#pragma unroll
                    for (int i = 0; i < 4; ++i) {
                        const int m = 4 * qq + i;
                        if constexpr (IN_F32) {
                            uint32_t lo, hi;
                            unpack2u(lds64(src + f_a + 1024u * m), lo, hi);
                            G[m] = pack2u(lo ^ ((s4[i] & 0x8000u) << 16), hi ^ (s4[i] & 0x80000000u));
                        } else {
                            const uint32_t w = lds32(src + ((m & 1) ? g_a1 : g_a0) + 512u * m) ^ s4[i];
                            G[m] = pack2u(bf16_lo(w), w & 0xFFFF0000u);
                        }
                    }
                }
            }
            if constexpr (kOneSlot) {  // the one slot has been read by every thread of the group: next pair
                bar_sync(cx.a.bar, kThreads);
                if (t == 0 && k + 1 < count) request(k + 1);
            }
            rev_steps<0, kUpperSteps>(Y0, Y1, G0, G1, T0, T1, A0, A1, cx, [](auto) {});
            // phase 3 -> phase 2 regrouping = the hand-over: once the lower group is past its reads of the buffers for
            // the previous pair, store in the layout it reads
            bar_sync(kBarEmpty, kCtaThreads);
            rev2_store(Y0, exr + 0 * kExBytes, cx.a);
            rev2_store(Y1, exr + 1 * kExBytes, cx.a);
            rev2_store(G0, exr + 2 * kExBytes, cx.a);
            rev2_store(G1, exr + 3 * kExBytes, cx.a);
            __threadfence_block();
            bar_arrive(kBarFull, kCtaThreads);
        }
    } else {
        // ================= lower group: stages 8 .. 0, dx =================
        if (count > 0) bar_arrive(kBarEmpty, kCtaThreads);  // the buffers start empty (the upper group's first wait)
        for (int k = 0; k < count; ++k) {
            const int r0 = 2 * (first + k * stride);
            tmem_ld16(cx.tlane + RevStep<kUpperSteps>::kTCol, T0);
            tmem_ld8(cx.tlane + RevStep<kUpperSteps>::kAccCol, A0);
            bar_sync(kBarFull, kCtaThreads);
            rev2_load(Y0, exr + 0 * kExBytes, cx.a);
            rev2_load(Y1, exr + 1 * kExBytes, cx.a);
            rev2_load(G0, exr + 2 * kExBytes, cx.a);
            rev2_load(G1, exr + 3 * kExBytes, cx.a);
            rev_steps<kUpperSteps, 24>(Y0, Y1, G0, G1, T0, T1, A0, A1, cx, [&](auto step) {
                constexpr int I = decltype(step)::value;
                if constexpr (I == 15) {  // phase 2 -> phase 1, inside each half-warp, but the buffers were read across warps
                    bar_sync(cx.a.bar, kThreads);
                    rev1_store(Y0, exr + 0 * kExBytes, cx.a);
                    rev1_store(Y1, exr + 1 * kExBytes, cx.a);
                    rev1_store(G0, exr + 2 * kExBytes, cx.a);
                    rev1_store(G1, exr + 3 * kExBytes, cx.a);
                    __syncwarp();
                    rev1_load(Y0, exr + 0 * kExBytes, cx.a);
                    rev1_load(Y1, exr + 1 * kExBytes, cx.a);
                    rev1_load(G0, exr + 2 * kExBytes, cx.a);
                    rev1_load(G1, exr + 3 * kExBytes, cx.a);
                }
                if constexpr (I == 17) {  // stage 3 has used every value of that regrouping: the buffers are free
                    if (k + 1 < count) bar_arrive(kBarEmpty, kCtaThreads);
                }
            });

            // ---- dx = parity sign * g, bf16, phase-1 ownership: two runs of 16 elements per row ----
            if (dx_out != nullptr) {
#pragma unroll
                for (int r = 0; r < 2; ++r) {
                    if (r0 + r < rows) {
                        const u64(&G)[16] = r == 0 ? G0 : G1;
                        if constexpr (IN_F32) {
                            float* row = static_cast<float*>(dx_out) + static_cast<int64_t>(r0 + r) * ld + 16 * (t & 15) + 512 * (t >> 4);
#pragma unroll
                            for (int h = 0; h < 2; ++h) {
                                uint32_t w[16];
#pragma unroll
                                for (int m = 0; m < 16; ++m) {
                                    uint32_t lo, hi;
                                    unpack2u(G[m], lo, hi);
                                    // element m of half h: parity popcount(m) ^ h ^ popcount(t)
                                    const bool odd_c = ((__builtin_popcount(m) + h) & 1) != 0;
                                    w[m] = (h ? hi : lo) ^ (odd_c ? sgn_b : sgn_a);
                                }
                                uint4* dst = reinterpret_cast<uint4*>(row + 256 * h);
#pragma unroll
                                for (int c = 0; c < 4; ++c) dst[c] = make_uint4(w[4 * c], w[4 * c + 1], w[4 * c + 2], w[4 * c + 3]);
                            }
                            continue;
                        }
                        __nv_bfloat16* row = dx + static_cast<int64_t>(r0 + r) * ld + 16 * (t & 15) + 512 * (t >> 4);
#pragma unroll
                        for (int h = 0; h < 2; ++h) {
                            uint32_t w[8];
#pragma unroll
                            for (int j = 0; j < 8; ++j) {
                                uint32_t lo0, hi0, lo1, hi1;
                                unpack2u(G[2 * j], lo0, hi0);
                                unpack2u(G[2 * j + 1], lo1, hi1);
                                const float e0 = __uint_as_float(h ? hi0 : lo0), e1 = __uint_as_float(h ? hi1 : lo1);
                                // elements m = 2j, 2j+1 of half h: parity popcount(2j) ^ h ^ popcount(t), opposite for 2j+1
                                const bool odd_c = ((__builtin_popcount(2 * j) + h) & 1) != 0;
                                const uint32_t neg_lo = odd_c ? (sgn_b >> 16) : (sgn_a >> 16);  // bit 15: element 2j
                                const uint32_t neg_hi = odd_c ? sgn_a : sgn_b;                  // bit 31: element 2j+1
                                w[j] = cvt_bf16x2(e0, e1) ^ (neg_lo | neg_hi);
                            }
                            uint4* dst = reinterpret_cast<uint4*>(row + 256 * h);
                            dst[0] = make_uint4(w[0], w[1], w[2], w[3]);
                            dst[1] = make_uint4(w[4], w[5], w[6], w[7]);
                        }
                    }
                }
            }
            tmem_wait_st();  // this row pair's accumulator stores land before the next pair reloads them
        }
    }

    // ---- this CTA's sums -> its slot of the partial sums, with the sign of the basis undone ----
    __syncthreads();  // the upper group's sums of stages 9..11 (shared memory) are complete
    float* const slot_out = partial + static_cast<int64_t>(blockIdx.x) * (WIDE ? kSlotFloatsWide : kSlotFloats);
    if constexpr (WIDE) {
        if (is_fwd) {
            // this half's share of stage 12: pairs 2t + 256m, +1; y carried the signs of the basis g enters (the sign
            // words), half 1's share is subtracted
            const float sg = half ? -1.f : 1.f;
            for (int m = 0; m < 16; ++m) {
                float a0, a1;
                unpack2(lds64(sbase + S::kAcc12Off + (m * kThreads + t) * 8), a0, a1);
                const uint32_t sw = __ldg(gsign + (m >> 2) * 4 * kThreads + 4 * t + (m & 3));
                *reinterpret_cast<float2*>(slot_out + kSlotFloats + 2 * t + 256 * m) =
                    make_float2((sw & 0x8000u) ? -sg * a0 : sg * a0, (sw & 0x80000000u) ? -sg * a1 : sg * a1);
            }
        }
    }
    if (!is_fwd) {
        float* out = slot_out;
        for (int s = 0; s < 12; ++s) {
            const int K = s & 3, P = s >> 2;
            for (int c = 0; c < 2; ++c) {
                uint32_t a[8];
                if (s < 8) {
                    tmem_ld8(cx.tlane + kAccCol + 16 * s + 8 * c, a);
                    asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
                } else {
                    const uint32_t base = cx.acc_smem + ((s - 8) * 4 + 2 * c) * kThreads * 16;
                    const uint4 v0 = lds128(base), v1 = lds128(base + kThreads * 16);
                    a[0] = v0.x, a[1] = v0.y, a[2] = v0.z, a[3] = v0.w, a[4] = v1.x, a[5] = v1.y, a[6] = v1.z, a[7] = v1.w;
                }
#pragma unroll
                for (int e = 0; e < 8; ++e) {
                    const int u = 4 * c + (e >> 1), h = e & 1;
                    const int m_lo = ((u >> K) << (K + 1)) | (u & ((1 << K) - 1));
                    const int lo = elem_of(P, t, m_lo, h);
                    const int j = ((lo >> (s + 1)) << s) | (lo & ((1 << s) - 1));
                    out[s * (kN / 2) + j] = __uint_as_float(a[e]) * static_cast<float>(dsign[s * (kN / 2) + j]);
                }
            }
        }
    }
    tmem_fence_before();
    __syncthreads();
    if (warp == 0) tmem_dealloc512(tmem_base);
}

// ---- tables ---------------------------------------------------------------------------------------------------
// One thread per angle: the three-shear constants of pair (s, j), negated when its two elements carry
// opposite signs, at the place the owning role reads them; and the sign that turns the accumulated
// g_hi*y_lo - g_lo*y_hi of the parity basis into d-theta.
__global__ void __launch_bounds__(256) k_build_image_bwd4096(const float4* __restrict__ prep,
                                                              const uint8_t* __restrict__ flip,
                                                              float* __restrict__ img, int8_t* __restrict__ dsign) {
    const int k = blockIdx.x * blockDim.x + threadIdx.x;
    if (k >= 12 * (kN / 2)) return;
    const int s = k / (kN / 2), j = k % (kN / 2);
    const int lo = ((j >> s) << (s + 1)) | (j & ((1 << s) - 1));
    const int hi = lo + (1 << s);
    const int sa = sign_before(flip, lo, s), sb = sign_before(flip, hi, s);
    const int kk = s & 3;
    int r, m, h;
    if (s < 4) {
        r = ((lo >> 4) & 15) | ((lo >> 9) << 4), m = lo & 15, h = (lo >> 8) & 1;
    } else if (s < 8) {
        r = (lo & 15) | ((lo >> 9) << 4), m = (lo >> 4) & 15, h = (lo >> 8) & 1;
    } else {
        r = (lo >> 1) & 127, m = lo >> 8, h = lo & 1;
    }
    const int u = ((m >> (kk + 1)) << kk) | (m & ((1 << kk) - 1));
    const float4 p = prep[k];
    const float sg = (sa == sb) ? 1.f : -1.f;
    float* strip = img + r * kConstCols;
    strip[32 * s + 4 * u + h] = sg * p.x;
    strip[32 * s + 4 * u + h + 2] = sg * p.y;
    dsign[k] = static_cast<int8_t>(-(sa * sb));
}

// One thread per 32-bit word of a bf16 g row in phase-3 ownership (role t, register m): bit 15 / bit 31 set
// when element 2t + 256m / its neighbour must be negated to enter the basis sigma(after stage 11) * parity.
__global__ void __launch_bounds__(256) k_build_gsign4096(const uint8_t* __restrict__ flip, uint32_t* __restrict__ gsign) {
    const int w = blockIdx.x * blockDim.x + threadIdx.x;
    if (w >= 16 * kThreads) return;
    const int m = (w / (4 * kThreads)) * 4 + (w & 3), t = (w >> 2) % kThreads;  // layout [m / 4][t][m % 4]
    const int e = 2 * t + 256 * m;
    const int s0 = sign_before(flip, e, 12) * ((__popc(e) & 1) ? -1 : 1);
    const int s1 = sign_before(flip, e + 1, 12) * ((__popc(e + 1) & 1) ? -1 : 1);
    gsign[w] = (s0 < 0 ? 0x00008000u : 0u) | (s1 < 0 ? 0x80000000u : 0u);
}


// One thread per angle: the constants of the scaled reverse walk (x = Q^T y, stages 11 down to 0).  Element i enters
// reverse stage s carrying the factor e = product of the cosines of the pairs it belongs to in stages s+1..11; stage s
// then is  lo = lo' + j1 hi',  hi = hi' + j2 lo'  with  j1 = tan(theta) e_hi / e_lo,  j2 = -tan(theta) e_lo / e_hi  and
// both factors are multiplied by cos(theta).  Stage 0 is a general 2x2 that absorbs the factors.  Image layout
// [column quad][role][4]; stage s >= 1 at columns 32 (s - 1), stage 0 at 352.  *form is raised when a factor leaves
// [2^-64, 1]: the kernel then walks in the three-shear form.
__global__ void __launch_bounds__(256) k_build_image_inv4096(const double2* __restrict__ cs, float* __restrict__ img,
                                                              int* __restrict__ form) {
    const int k = blockIdx.x * blockDim.x + threadIdx.x;
    if (k >= 12 * (kN / 2)) return;
    const int s = k / (kN / 2), j = k % (kN / 2);
    const int lo = ((j >> s) << (s + 1)) | (j & ((1 << s) - 1));
    const int hi = lo + (1 << s);
    double cl[11], ch[11];
#pragma unroll
    for (int sp = 1; sp < 12; ++sp) {  // all loads issued together
        const int jl = ((lo >> (sp + 1)) << sp) | (lo & ((1 << sp) - 1));
        const int jh = ((hi >> (sp + 1)) << sp) | (hi & ((1 << sp) - 1));
        cl[sp - 1] = sp > s ? cs[sp * (kN / 2) + jl].x : 1.0;
        ch[sp - 1] = sp > s ? cs[sp * (kN / 2) + jh].x : 1.0;
    }
    double el = 1.0, eh = 1.0;
#pragma unroll
    for (int i = 0; i < 11; ++i) el *= cl[i], eh *= ch[i];
    const int kk = s & 3;
    int r, m, h;
    if (s < 4) {
        r = ((lo >> 4) & 15) | ((lo >> 9) << 4), m = lo & 15, h = (lo >> 8) & 1;
    } else if (s < 8) {
        r = (lo & 15) | ((lo >> 9) << 4), m = (lo >> 4) & 15, h = (lo >> 8) & 1;
    } else {
        r = (lo >> 1) & 127, m = lo >> 8, h = lo & 1;
    }
    const int u = ((m >> (kk + 1)) << kk) | (m & ((1 << kk) - 1));
    const double2 own = cs[k];
    float* strip = img + 4 * r;
    auto at = [](int col) { return (col >> 2) * 512 + (col & 3); };
    if (s > 0) {
        const double w = own.y / (own.x * el * eh);  // tan(theta) / (e_lo e_hi)
        const int col = 32 * (s - 1) + 4 * u + h;
        strip[at(col)] = static_cast<float>(w * eh * eh);
        strip[at(col + 2)] = static_cast<float>(-w * el * el);
        const double lim = 5.421010862427522e-20;  // 2^-64
        if (!(fabs(own.x * el) >= lim && fabs(own.x * eh) >= lim)) *form = kFormShear;
    } else {
        const int col = 352 + 8 * u + h;
        strip[at(col + 0)] = static_cast<float>(own.x * el);
        strip[at(col + 2)] = static_cast<float>(own.y * eh);
        strip[at(col + 4)] = static_cast<float>(-own.y * el);
        strip[at(col + 6)] = static_cast<float>(own.x * eh);
    }
}

// =================================================================================================================
// Inverse / transpose for n = 4096 bf16 rows:  x = Q^T y.  The reverse walk of the backward kernel on one array,
// organised like the forward kernel: four row groups of 128 threads per CTA, 32 constants per tensor-memory chunk.
// =================================================================================================================
template <int G>
struct InvSmem {
    static constexpr uint32_t kInOff = 0;                                  // [G][kInSlots][kRowBytes]
    static constexpr uint32_t kExOff = kInOff + G * kInSlots * kRowBytes;  // [G][2][kExBytes]
    static constexpr uint32_t kBarOff = kExOff + G * 2 * kExBytes;         // mbarriers [G][kInSlots]
    static constexpr uint32_t kTmemOff = kBarOff + 8 * G * kInSlots;
    static constexpr uint32_t kUsed = kTmemOff + 16;
    static constexpr uint32_t kBytes = kUsed + 1024;
};

// general 2x2 on local bit 0 (stage 0 of the reverse walk): out_lo = k1*a + k2*b, out_hi = k3*a + k4*b for the
// register pairs (2u, 2u + 1), u = U0..U0+NU-1
template <int U0, int NU>
__device__ __forceinline__ void stage_general_k0(u64 (&P)[16], const uint32_t (&T)[32]) {
    static_assert(8 * NU <= 32, "chunk too small");
#pragma unroll
    for (int i = 0; i < NU; ++i) {
        const int m_lo = 2 * (U0 + i), m_hi = m_lo + 1;
        const u64 K1 = pack2u(T[8 * i], T[8 * i + 1]), K2 = pack2u(T[8 * i + 2], T[8 * i + 3]);
        const u64 K3 = pack2u(T[8 * i + 4], T[8 * i + 5]), K4 = pack2u(T[8 * i + 6], T[8 * i + 7]);
        const u64 a = P[m_lo], b = P[m_hi];
        P[m_lo] = fma2(K2, b, mul2(K1, a));
        P[m_hi] = fma2(K4, b, mul2(K3, a));
    }
}

// stage S (11..0) is in Tcur; the next constants are requested right after the wait.  Three-shear form: stage s at
// column 32 s, all twelve stages alike.  Scaled form: stages 11..1 are two-FMA stages on values that carry the product of
// the cosines of the stages above, stage 0 is a general 2x2 (two chunks) that absorbs the factors.
template <int FORM, int S, class F>
__device__ __forceinline__ void inv_stages(u64 (&P)[16], uint32_t (&Tcur)[32], uint32_t (&Tnext)[32], uint32_t tlane,
                                           const Addr& a, uint32_t buf2, uint32_t buf1, F&& after_phase3) {
    tmem_wait_ld32(Tcur);
    if constexpr (FORM == kFormShear) {
        if constexpr (S > 0) tmem_ld32(tlane + 32 * (S - 1), Tnext);
        stage_lift<S & 3, 0, 8, 32>(P, Tcur);
    } else {
        if constexpr (S > 1) tmem_ld32(tlane + 32 * (S - 2), Tnext);
        if constexpr (S == 1) tmem_ld32(tlane + 352, Tnext);
        if constexpr (S > 0) stage_scaled<S & 3, 0, 8, 32>(P, Tcur);
        if constexpr (S == 0) {
            tmem_ld32(tlane + 384, Tnext);
            stage_general_k0<0, 4>(P, Tcur);
            tmem_wait_ld32(Tnext);
            stage_general_k0<4, 4>(P, Tnext);
        }
    }
    if constexpr (S == 8) {
        bar_sync(a.bar, kThreads);  // every warp is past its scalar reads of the previous row
        rev2_store(P, buf2, a);
        bar_sync(a.bar, kThreads);
        after_phase3();
        rev2_load(P, buf2, a);
    }
    if constexpr (S == 4) {
        __syncwarp();
        rev1_store(P, buf1, a);
        __syncwarp();
        rev1_load(P, buf1, a);
    }
    if constexpr (S > 0) inv_stages<FORM, S - 1>(P, Tnext, Tcur, tlane, a, buf2, buf1, after_phase3);
}

// what the CTAs of the upper half use in the wide mode of the inverse kernel instead of img, img_scaled, form, gsign
struct InvUpper {
    const float* img;
    const float* img_scaled;
    const int* form;
    const uint32_t* gsign;
};

// IN_F32: the rows come in fp32 (16 KB each): one input slot per group instead of two, re-armed after phase 3.
// WIDE (bf16 rows in): n = 8192.  x = Q^T y = (Q_lo^T (+) Q_hi^T) B_12^T y: even CTAs produce the lower 4096 elements of x,
// odd CTAs the upper (CTAs 2i and 2i + 1 work on the same rows at about the same time, so the second read of a row comes
// from L2).  A y row is 16 KB in one slot; the transposed stage-12 rotation y'_own = c y_own +- s y_other with (cos, sin)
// from `tw12` is applied as the row is read, then the half's own twelve stages follow from its own tables.
template <int G, bool OUT_BF16, bool IN_F32 = false, bool WIDE = false>
__global__ void __launch_bounds__(G * kThreads, 1)
k_inv4096(const __grid_constant__ CUtensorMap ymap, const float* __restrict__ img_lo, const float* __restrict__ img_scaled_lo,
          const int* __restrict__ form_lo, const uint32_t* __restrict__ gsign_lo, void* __restrict__ xout, int64_t ldx, int rows,
          int* __restrict__ status, const float2* __restrict__ tw12, const InvUpper upper) {
    static_assert(!(IN_F32 && WIDE), "the wide mode takes bf16 rows");
    const int half = WIDE ? int(blockIdx.x & 1u) : 0;
    const int cta = WIDE ? int(blockIdx.x >> 1) : int(blockIdx.x);
    const int ctas = WIDE ? int((gridDim.x + 1u) >> 1) : int(gridDim.x);
    const float* const img = (WIDE && half) ? upper.img : img_lo;
    const float* const img_scaled = (WIDE && half) ? upper.img_scaled : img_scaled_lo;
    const int* const form = (WIDE && half) ? upper.form : form_lo;
    const uint32_t* const gsign = (WIDE && half) ? upper.gsign : gsign_lo;
    using S = InvSmem<G>;
    extern __shared__ uint8_t smem_raw[];
    const uint32_t sbase = (smem_u32(smem_raw) + 1023u) & ~1023u;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int q = warp & 3, g = warp >> 2;
    const int t = q * 32 + lane;

    if (warp == 0) tmem_alloc512(sbase + S::kTmemOff);
    if (threadIdx.x < G * kInSlots) {
        mbar_init(sbase + S::kBarOff + 8 * threadIdx.x, 1);
        mbar_init_fence();
    }
    tmem_fence_before();
    __syncthreads();
    tmem_fence_after();
    uint32_t tmem_base;
    asm volatile("ld.shared.u32 %0, [%1];" : "=r"(tmem_base) : "r"(sbase + S::kTmemOff));
    const uint32_t tlane = tmem_base + (static_cast<uint32_t>(q * 32) << 16);

    const int first = cta * G + g;
    const int stride = ctas * G;
    const int count = first < rows ? (rows - first + stride - 1) / stride : 0;
    const uint32_t in_base = sbase + S::kInOff + g * kInSlots * kRowBytes;
    const uint32_t bar_base = sbase + S::kBarOff + 8 * g * kInSlots;
    constexpr int kSlotsUsed = (IN_F32 || WIDE) ? 1 : kInSlots;
    constexpr uint32_t kSlotBytes = (IN_F32 || WIDE) ? 2 * kRowBytes : kRowBytes;
    static_assert(kInSlots == 2, "an fp32 row, or a bf16 row of 8192, takes the group's two bf16 slots");
    if (t == 0) {
        for (int k = 0; k < kSlotsUsed && k < count; ++k) {
            mbar_expect_tx(bar_base + 8 * k, kSlotBytes);
            tma_load_3d(in_base + k * kSlotBytes, &ymap, 0, 0, first + k * stride, bar_base + 8 * k);
        }
    }
    // constants: the scaled-form image ([column quad][role][4], coalesced, all loads in flight) unless the table build
    // flagged it out of range; then the three-shear image ([role][384])
    const bool shear = __ldg(form) != 0;
    if (!shear) {
        constexpr int kFillBlocks = (kInvCols / 16 + G - 1) / G;
        float4 fill[kFillBlocks][4];
        const float4* base = reinterpret_cast<const float4*>(img_scaled);
#pragma unroll
        for (int j = 0; j < kFillBlocks; ++j) {
            const int b = g + j * G;
            if (b < kInvCols / 16) {
#pragma unroll
                for (int i = 0; i < 4; ++i) fill[j][i] = __ldg(base + (4 * b + i) * 128 + t);
            }
        }
#pragma unroll
        for (int j = 0; j < kFillBlocks; ++j) {
            const int b = g + j * G;
            if (b < kInvCols / 16) {
                uint32_t v[16];
#pragma unroll
                for (int i = 0; i < 4; ++i) {
                    v[4 * i + 0] = __float_as_uint(fill[j][i].x), v[4 * i + 1] = __float_as_uint(fill[j][i].y);
                    v[4 * i + 2] = __float_as_uint(fill[j][i].z), v[4 * i + 3] = __float_as_uint(fill[j][i].w);
                }
                tmem_st16(tlane + 16 * b, v);
            }
        }
        tmem_wait_st();
    } else {
        const float4* src = reinterpret_cast<const float4*>(img + (q * 32 + lane) * kConstCols);
        for (int c = 16 * g; c < kConstCols; c += 16 * G) {
            uint32_t v[16];
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                const float4 f = __ldg(src + (c >> 2) + i);
                v[4 * i + 0] = __float_as_uint(f.x), v[4 * i + 1] = __float_as_uint(f.y);
                v[4 * i + 2] = __float_as_uint(f.z), v[4 * i + 3] = __float_as_uint(f.w);
            }
            tmem_st16(tlane + c, v);
        }
        tmem_wait_st();
    }
    if constexpr (WIDE) {
        // (cos, sin) of the stage-12 pairs 2t + 256m, +1 for m = 0 .. 15, sin with the sign this half applies it with:
        // 64 columns of the thread's lane, written once by the first group
        static_assert(kWideCol >= kInvCols && kWideCol >= kConstCols && kWideCol + 64 <= 512, "tensor-memory columns");
        if (g == 0) {
            const float sg = half ? -1.f : 1.f;
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                uint32_t v[16];
#pragma unroll
                for (int i = 0; i < 4; ++i) {
                    const float4 cs = __ldg(reinterpret_cast<const float4*>(tw12 + 2 * t + 256 * (4 * j + i)));
                    v[4 * i + 0] = __float_as_uint(cs.x), v[4 * i + 1] = __float_as_uint(sg * cs.y);
                    v[4 * i + 2] = __float_as_uint(cs.z), v[4 * i + 3] = __float_as_uint(sg * cs.w);
                }
                tmem_st16(tlane + kWideCol + 16 * j, v);
            }
            tmem_wait_st();
        }
    }
    tmem_fence_before();
    __syncthreads();
    tmem_fence_after();

    Addr a;
    {
        const uint32_t t4 = (t >> 4) & 1, t5 = (t >> 5) & 1, t6 = (t >> 6) & 1;
        a.ex = sbase + S::kExOff + g * 2 * kExBytes;
        a.bar = 1 + g;
        a.w1 = 4u * (2u * (t & 15) + 32u * (t >> 4));
        a.r1 = 4u * (258u * (t & 15) + 32u * (t >> 4));
        a.w2 = 4u * ((t & 15) + 2064u * t4 + 512u * t5 + 1024u * t6);
        a.r2 = 4u * (2u * (t & 15) + 32u * (t >> 4));
    }
    const uint32_t g_x = (((t & 31) >> 2) ^ (t >> 5));
    const uint32_t g_a0 = (t >> 5) * 128u + (g_x << 4) + (t & 3) * 4u;
    const uint32_t g_a1 = (t >> 5) * 128u + ((g_x ^ 4u) << 4) + (t & 3) * 4u;
    const uint32_t f_a = (t >> 4) * 128u + ((((t & 15) >> 1) ^ (t >> 4)) << 4) + (t & 1) * 8u;  // fp32 rows
    const uint32_t par_t = __popc(t) & 1;
    const uint32_t sgn_a = par_t ? 0x80000000u : 0u, sgn_b = par_t ? 0u : 0x80000000u;
    const uint4* gsv = reinterpret_cast<const uint4*>(gsign);

    // the whole row loop exists once per stage form: the choice is made once per launch, outside the loop
    auto row_loop = [&](auto form_tag) {
    constexpr int FORM = decltype(form_tag)::value;
    constexpr bool kSigns = FORM == kFormShear;  // the three-shear walk runs in the sign-tracked parity basis
    u64 P[16];
    uint32_t T0[32], T1[32];
    for (int k = 0; k < count; ++k) {
        const int row = first + k * stride;
        const int slot = kSlotsUsed == 1 ? 0 : (k & 1);
        tmem_ld32(tlane + (FORM == kFormShear ? 32 * 11 : 32 * 10), T0);
        mbar_wait_bounded(bar_base + 8 * slot, (kSlotsUsed == 1 ? k : (k >> 1)) & 1, status);
        const uint32_t tile = in_base + slot * kSlotBytes;
        if constexpr (WIDE) {
            // elements 2t + 256m, +1 of both halves of the row (the upper half is 8192 bytes further on, the same line
            // modulo 8) and (cos, +-sin) of the two stage-12 pairs they form, eight registers m per tensor-memory load
#pragma unroll
            for (int hh = 0; hh < 2; ++hh) {
                tmem_ld32(tlane + kWideCol + 32 * hh, T1);
                uint32_t s8[8] = {0u, 0u, 0u, 0u, 0u, 0u, 0u, 0u};
                if constexpr (kSigns) {
                    const uint4 sw0 = __ldg(gsv + (2 * hh) * kThreads + t), sw1 = __ldg(gsv + (2 * hh + 1) * kThreads + t);
                    s8[0] = sw0.x, s8[1] = sw0.y, s8[2] = sw0.z, s8[3] = sw0.w;
                    s8[4] = sw1.x, s8[5] = sw1.y, s8[6] = sw1.z, s8[7] = sw1.w;
                }
                uint32_t wo[8], wx[8];
#pragma unroll
                for (int i = 0; i < 8; ++i) {
                    const int m = 8 * hh + i;
                    const uint32_t at = tile + ((m & 1) ? g_a1 : g_a0) + 512u * m;
                    wo[i] = lds32(at + 8192u * half), wx[i] = lds32(at + 8192u * (half ^ 1));
                }
                tmem_wait_ld32(T1);
#pragma unroll
                for (int i = 0; i < 8; ++i) {
                    const u64 own = pack2u(bf16_lo(wo[i]), wo[i] & 0xFFFF0000u), oth = pack2u(bf16_lo(wx[i]), wx[i] & 0xFFFF0000u);
                    const u64 c2 = pack2u(T1[4 * i], T1[4 * i + 2]), s2 = pack2u(T1[4 * i + 1], T1[4 * i + 3]);
                    uint32_t lo, hi;
                    unpack2u(fma2(s2, oth, mul2(c2, own)), lo, hi);
                    P[8 * hh + i] = pack2u(lo ^ ((s8[i] & 0x8000u) << 16), hi ^ (s8[i] & 0x80000000u));
                }
            }
        }
#pragma unroll
        for (int qq = 0; qq < (WIDE ? 0 : 4); ++qq) {
            if constexpr (IN_F32) {
                // elements 2t + 256m, +1 are the 8-byte word t & 1 of 16-byte chunk (t & 15) >> 1 of 128-byte line
                // (t >> 4) + 8m; the swizzle moves the chunk to chunk ^ (line & 7)
                uint32_t s4[4] = {0u, 0u, 0u, 0u};
                if constexpr (kSigns) {
                    const uint4 sw = __ldg(gsv + qq * kThreads + t);
                    s4[0] = sw.x, s4[1] = sw.y, s4[2] = sw.z, s4[3] = sw.w;
                }
#pragma unroll
                for (int i = 0; i < 4; ++i) {
                    const int m = 4 * qq + i;
                    uint32_t lo, hi;
                    unpack2u(lds64(tile + f_a + 1024u * m), lo, hi);
                    P[m] = pack2u(lo ^ ((s4[i] & 0x8000u) << 16), hi ^ (s4[i] & 0x80000000u));
                }
                continue;
            }
            uint32_t s4[4] = {0u, 0u, 0u, 0u};
            if constexpr (kSigns) {
                const uint4 sw = __ldg(gsv + qq * kThreads + t);  // 2 KB in all: stays in L1
                s4[0] = sw.x, s4[1] = sw.y, s4[2] = sw.z, s4[3] = sw.w;
            }
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                const int m = 4 * qq + i;
                const uint32_t w = lds32(tile + ((m & 1) ? g_a1 : g_a0) + 512u * m) ^ s4[i];
                P[m] = pack2u(bf16_lo(w), w & 0xFFFF0000u);
            }
        }
        inv_stages<FORM, 11>(P, T0, T1, tlane, a, a.ex, a.ex + kExBytes, [&]() {
            if (t == 0 && k + kSlotsUsed < count) {
                mbar_expect_tx(bar_base + 8 * slot, kSlotBytes);
                tma_load_3d(in_base + slot * kSlotBytes, &ymap, 0, 0, first + (k + kSlotsUsed) * stride, bar_base + 8 * slot);
            }
        });
        // phase-1 ownership: two runs of 16 consecutive elements; the three-shear form undoes the parity sign here
        const uint32_t sa_ = kSigns ? sgn_a : 0u, sb_ = kSigns ? sgn_b : 0u;
#pragma unroll
        for (int h = 0; h < 2; ++h) {
            const int64_t off = static_cast<int64_t>(row) * ldx + (WIDE ? kN * half : 0) + 16 * (t & 15) + 512 * (t >> 4) + 256 * h;
            if constexpr (OUT_BF16) {
                uint32_t w[8];
#pragma unroll
                for (int j = 0; j < 8; ++j) {
                    uint32_t lo0, hi0, lo1, hi1;
                    unpack2u(P[2 * j], lo0, hi0);
                    unpack2u(P[2 * j + 1], lo1, hi1);
                    const float e0 = __uint_as_float(h ? hi0 : lo0), e1 = __uint_as_float(h ? hi1 : lo1);
                    const bool odd_c = ((__builtin_popcount(2 * j) + h) & 1) != 0;
                    const uint32_t neg_lo = odd_c ? (sb_ >> 16) : (sa_ >> 16);
                    const uint32_t neg_hi = odd_c ? sa_ : sb_;
                    w[j] = cvt_bf16x2(e0, e1) ^ (neg_lo | neg_hi);
                }
                uint4* dst = reinterpret_cast<uint4*>(static_cast<__nv_bfloat16*>(xout) + off);
                dst[0] = make_uint4(w[0], w[1], w[2], w[3]);
                dst[1] = make_uint4(w[4], w[5], w[6], w[7]);
            } else {
                uint32_t w[16];
#pragma unroll
                for (int m = 0; m < 16; ++m) {
                    uint32_t lo, hi;
                    unpack2u(P[m], lo, hi);
                    const bool odd_c = ((__builtin_popcount(m) + h) & 1) != 0;  // parity popcount(m) ^ h ^ popcount(t)
                    w[m] = (h ? hi : lo) ^ (odd_c ? sb_ : sa_);
                }
                uint4* dst = reinterpret_cast<uint4*>(static_cast<float*>(xout) + off);
#pragma unroll
                for (int c = 0; c < 4; ++c) dst[c] = make_uint4(w[4 * c], w[4 * c + 1], w[4 * c + 2], w[4 * c + 3]);
            }
        }
    }
    };
    if (!shear) {
        row_loop(std::integral_constant<int, kFormScaled>());
    } else {
        row_loop(std::integral_constant<int, kFormShear>());
    }
    tmem_fence_before();
    __syncthreads();
    if (warp == 0) tmem_dealloc512(tmem_base);
}

}  // namespace b4k

// ---- host side ---------------------------------------------------------------------------------------------
namespace b4k {
// One thread per angle of stages 0 .. 11 of half `half` of an n = 8192 transform: the staging entries the table builds
// above read (three-shear constants, cos, sin; negation flag), from the (cos, sin) in double that bfq_set_angles left.
__global__ void __launch_bounds__(256) k_prep_half8192(const double2* __restrict__ cs8192, int half, float4* __restrict__ prep,
                                                        uint8_t* __restrict__ flip, double2* __restrict__ cs_half) {
    const int k = blockIdx.x * blockDim.x + threadIdx.x;
    if (k >= 12 * (kN / 2)) return;
    const int s = k / (kN / 2), j = k % (kN / 2);
    const double2 v = cs8192[s * kN + (kN / 2) * half + j];
    cs_half[k] = v;  // what the scaled inverse table is built from
    const double c = v.x, sn = v.y;
    const bool f = c < 0.0;
    const double sp = f ? -sn : sn, cp = f ? -c : c;
    flip[k] = f ? 1 : 0;
    prep[k] = make_float4(static_cast<float>(-sp / (1.0 + cp)), static_cast<float>(sp), static_cast<float>(c),
                          static_cast<float>(sn));
}

// Wide mode: dtheta [13][4096] from the 2 * ctas slots (kSlotFloatsWide floats each; even slots hold the lower half's
// CTAs).  Stage s < 12, angle 2048 h + j = the sum over half h's slots of entry s * 2048 + j; stage 12, angle i =
// the sum over all slots of entry kSlotFloats + i.  A block = 8 slot lanes x 32 angles: lane y adds slots y, y + 8, ...
// in order, then the eight sums are added in lane order, so the result does not depend on timing.
__global__ void __launch_bounds__(256) k_reduce_wide(const float* __restrict__ partial, int ctas, float* __restrict__ out) {
    __shared__ float sh[8][32];
    const int x = threadIdx.x & 31, y = threadIdx.x >> 5;
    const int k = blockIdx.x * 32 + x;  // 13 * 4096 is a multiple of 32
    const int s = k >> 12, r = k & 4095;
    int first = 0, step = 1, count = 2 * ctas, entry = kSlotFloats + r;
    if (s < 12) first = r >> 11, step = 2, count = ctas, entry = s * (kN / 2) + (r & 2047);
    const float* src = partial + static_cast<int64_t>(first) * kSlotFloatsWide + entry;
    float acc = 0.f;
#pragma unroll 4
    for (int c = y; c < count; c += 8) acc += src[static_cast<int64_t>(c) * step * kSlotFloatsWide];
    sh[y][x] = acc;
    __syncthreads();
    if (y == 0) {
        float a = sh[0][x];
#pragma unroll
        for (int i = 1; i < 8; ++i) a += sh[i][x];
        out[k] = a;
    }
}
}  // namespace b4k

// floats the wide mode needs in the plan's partial-sum buffer
size_t bwd8192_partial_floats(int sm_count) { return size_t(2) * sm_count * b4k::kSlotFloatsWide; }

size_t bwd8192_prep_bytes() { return size_t(12) * (f4k::kN / 2) * (sizeof(float4) + 1 + sizeof(double2)); }

bool bwd8192_available(const bfq_plan* plan) {
    return plan->n == 2 * f4k::kN && plan->cc_major == 10 && plan->img_b8192[0] != nullptr && plan->img_b8192[1] != nullptr &&
           plan->prep_half8192 != nullptr && plan->prep8192 != nullptr && plan->img_i8192[0] != nullptr && plan->img_i8192[1] != nullptr &&
           plan->partial_floats >= bwd8192_partial_floats(plan->sm_count) &&
           encode_tiled() != nullptr;
}

// the two halves' tables from the staging area bfq_set_angles filled (cos, sin in double after the 13 x 4096 float4 entries)
cudaError_t bwd8192_build_tables(const bfq_plan* plan, cudaStream_t st) {
    const int count = 12 * (f4k::kN / 2), count8 = 13 * f4k::kN;
    const double2* cs = reinterpret_cast<const double2*>(reinterpret_cast<const float4*>(plan->prep8192) + count8);
    float4* prep = reinterpret_cast<float4*>(plan->prep_half8192);
    uint8_t* flip = reinterpret_cast<uint8_t*>(prep + count);
    double2* cs_half = reinterpret_cast<double2*>(flip + count);  // count is a multiple of 16
    for (int h = 0; h < 2; ++h) {
        b4k::k_prep_half8192<<<(count + 255) / 256, 256, 0, st>>>(cs, h, prep, flip, cs_half);
        b4k::k_build_image_bwd4096<<<(count + 255) / 256, 256, 0, st>>>(prep, flip, plan->img_b8192[h], plan->dsign8192[h]);
        b4k::k_build_gsign4096<<<(16 * b4k::kThreads + 255) / 256, 256, 0, st>>>(flip, plan->gsign8192[h]);
        cudaError_t e = cudaGetLastError();
        if (e != cudaSuccess) return e;
        // the half's scaled reverse walk (inverse kernel) and its range flag: words 1 and 2 of the plan's form flags
        e = cudaMemsetAsync(plan->form_flag + 1 + h, 0, sizeof(int), st);
        if (e != cudaSuccess) return e;
        b4k::k_build_image_inv4096<<<(count + 255) / 256, 256, 0, st>>>(cs_half, plan->img_i8192[h], plan->form_flag + 1 + h);
        e = cudaGetLastError();
        if (e != cudaSuccess) return e;
    }
    return cudaSuccess;
}

// The n = 8192 backward (bf16 rows): both halves of the rows' elements in one launch (grid CTAs each), then one reduction;
// dx and all 13 rows of d-theta.
cudaError_t bwd8192_launch_halves(bfq_plan* plan, const void* x, const void* g, int64_t rows, int64_t ld, void* dx,
                                  float* dtheta, cudaStream_t st) {
    static bool attr_set[kMaxDevices] = {false};
    auto kern = b4k::k_bwd4096<false, true>;
    if (!attr_set[plan->device]) {
        cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, int(b4k::Smem::kBytesWide));
        if (e != cudaSuccess) return e;
        attr_set[plan->device] = true;
    }
    const int64_t pairs = (rows + 1) / 2;
    const int per_half = plan->sm_count / 2 > 0 ? plan->sm_count / 2 : 1;  // one CTA per SM: both halves in one wave
    const int grid = int(pairs < per_half ? pairs : per_half);
    CUtensorMap xmap, gmap;
    b4k::WideHalf upper{};
    // x: one half's 4096 elements of every row; g: whole rows of 8192 bf16 = 128 lines of 128 bytes
    if (!encode_row_map(&xmap, static_cast<const uint16_t*>(x), rows, ld)) return cudaErrorInvalidValue;
    if (!encode_row_map(&upper.xmap, static_cast<const uint16_t*>(x) + f4k::kN, rows, ld)) return cudaErrorInvalidValue;
    {
        const cuuint64_t dims[3] = {64, 128, static_cast<cuuint64_t>(rows)};
        const cuuint64_t strides[2] = {128, static_cast<cuuint64_t>(ld) * 2};
        const cuuint32_t box[3] = {64, 128, 1};
        const cuuint32_t estr[3] = {1, 1, 1};
        if (encode_tiled()(&gmap, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void*>(g), dims, strides, box, estr,
                           CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
                           CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
            return cudaErrorInvalidValue;
    }
    upper.img = plan->img_b8192[1], upper.gsign = plan->gsign8192[1], upper.dsign = plan->dsign8192[1];
    kern<<<2 * grid, b4k::kCtaThreads, b4k::Smem::kBytesWide, st>>>(xmap, gmap, plan->img_b8192[0], plan->gsign8192[0],
                                                                  plan->dsign8192[0], dx, ld, plan->partial, int(rows),
                                                                  plan->status_word, plan->tw + 12 * f4k::kN, upper);
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return e;
    b4k::k_reduce_wide<<<13 * f4k::kN / 32, 256, 0, st>>>(plan->partial, grid, dtheta);
    e = cudaGetLastError();
    if (e != cudaSuccess) return e;
    plan->last_backward_partials = 2 * grid;
    return cudaSuccess;
}

size_t bwd4096_image_bytes() { return size_t(128) * b4k::kConstCols * sizeof(float); }
size_t inv4096_image_bytes() { return size_t(128) * b4k::kInvCols * sizeof(float); }
size_t bwd4096_dsign_bytes() { return size_t(12) * (f4k::kN / 2); }
size_t bwd4096_gsign_bytes() { return size_t(16) * b4k::kThreads * sizeof(uint32_t); }

bool bwd4096_available(const bfq_plan* plan) {
    return plan->n == f4k::kN && plan->cc_major == 10 && plan->img_b4096 != nullptr && plan->prep4096 != nullptr &&
           plan->partial_slots >= plan->sm_count && encode_tiled() != nullptr;
}

// Builds the backward tables from the staging area bfq_set_angles filled (two launches).
cudaError_t bwd4096_build_tables(const bfq_plan* plan, cudaStream_t st) {
    const int count = 12 * (f4k::kN / 2);
    const float4* prep = reinterpret_cast<const float4*>(plan->prep4096);
    const uint8_t* flip = reinterpret_cast<const uint8_t*>(reinterpret_cast<const double2*>(prep + count) + count);
    b4k::k_build_image_bwd4096<<<(count + 255) / 256, 256, 0, st>>>(prep, flip, plan->img_b4096, plan->dsign4096);
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return e;
    b4k::k_build_gsign4096<<<(16 * b4k::kThreads + 255) / 256, 256, 0, st>>>(flip, plan->gsign4096);
    e = cudaGetLastError();
    if (e != cudaSuccess) return e;
    // the scaled reverse walk of the inverse kernel and its range flag (word 1 of the plan's form flags)
    e = cudaMemsetAsync(plan->form_flag + 1, 0, sizeof(int), st);
    if (e != cudaSuccess) return e;
    b4k::k_build_image_inv4096<<<(count + 255) / 256, 256, 0, st>>>(reinterpret_cast<const double2*>(prep + count),
                                                                   plan->img_i4096, plan->form_flag + 1);
    return cudaGetLastError();
}

// f32: x, g and dx are fp32 rows (else bf16)
cudaError_t bwd4096_launch(bfq_plan* plan, const void* x, const void* g, int64_t rows, int64_t ld, void* dx,
                           float* dtheta, bool f32, cudaStream_t st) {
    static bool attr_set[kMaxDevices] = {false};
    if (!attr_set[plan->device]) {
        cudaError_t e = cudaFuncSetAttribute(b4k::k_bwd4096<false>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                             int(b4k::Smem::kBytes));
        if (e == cudaSuccess)
            e = cudaFuncSetAttribute(b4k::k_bwd4096<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, int(b4k::Smem::kBytes));
        if (e != cudaSuccess) return e;
        attr_set[plan->device] = true;
    }
    CUtensorMap xmap, gmap;
    const bool maps = f32 ? (encode_row_map_f32(&xmap, x, rows, ld) && encode_row_map_f32(&gmap, g, rows, ld))
                          : (encode_row_map(&xmap, x, rows, ld) && encode_row_map(&gmap, g, rows, ld));
    if (!maps) return cudaErrorInvalidValue;
    const int64_t pairs = (rows + 1) / 2;
    const int grid = int(pairs < plan->sm_count ? pairs : plan->sm_count);
    if (f32) {
        b4k::k_bwd4096<true><<<grid, b4k::kCtaThreads, b4k::Smem::kBytes, st>>>(xmap, gmap, plan->img_b4096, plan->gsign4096,
                                                                              plan->dsign4096, dx, ld, plan->partial,
                                                                              int(rows), plan->status_word, nullptr, b4k::WideHalf{});
    } else {
        b4k::k_bwd4096<false><<<grid, b4k::kCtaThreads, b4k::Smem::kBytes, st>>>(xmap, gmap, plan->img_b4096, plan->gsign4096,
                                                                               plan->dsign4096, dx, ld, plan->partial,
                                                                               int(rows), plan->status_word, nullptr, b4k::WideHalf{});
    }
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return e;
    const int count = 12 * (f4k::kN / 2);
    k_reduce_partials<<<(count + 31) / 32, 256, 0, st>>>(plan->partial, grid, count, dtheta);
    plan->last_backward_partials = grid;
    return cudaGetLastError();
}

// fp32 rows in, fp32 rows out
cudaError_t inv4096_launch_f32(bfq_plan* plan, const void* y, int64_t rows, int64_t ldy, void* x, int64_t ldx,
                               cudaStream_t st) {
    constexpr int G = 4;
    using S = b4k::InvSmem<G>;
    auto kern = b4k::k_inv4096<G, false, true>;
    static bool attr_set[kMaxDevices] = {false};
    if (!attr_set[plan->device]) {
        cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, int(S::kBytes));
        if (e != cudaSuccess) return e;
        attr_set[plan->device] = true;
    }
    CUtensorMap ymap;
    if (!encode_row_map_f32(&ymap, y, rows, ldy)) return cudaErrorInvalidValue;
    const int64_t want = (rows + G - 1) / G;
    const int grid = int(want < plan->sm_count ? want : plan->sm_count);
    kern<<<grid, G * b4k::kThreads, S::kBytes, st>>>(ymap, plan->img_b4096, plan->img_i4096, plan->form_flag + 1,
                                                    plan->gsign4096, x, ldx, int(rows), plan->status_word, nullptr,
                                                    b4k::InvUpper{});
    return cudaGetLastError();
}

cudaError_t inv4096_launch(bfq_plan* plan, const void* y, int64_t rows, int64_t ldy, void* x, bool x_bf16, int64_t ldx,
                           cudaStream_t st) {
    constexpr int G = 4;
    using S = b4k::InvSmem<G>;
    static bool attr_set[kMaxDevices] = {false};
    if (!attr_set[plan->device]) {
        cudaError_t e = cudaFuncSetAttribute(b4k::k_inv4096<G, true>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                             int(S::kBytes));
        if (e == cudaSuccess)
            e = cudaFuncSetAttribute(b4k::k_inv4096<G, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, int(S::kBytes));
        if (e != cudaSuccess) return e;
        attr_set[plan->device] = true;
    }
    CUtensorMap ymap;
    if (!encode_row_map(&ymap, y, rows, ldy)) return cudaErrorInvalidValue;
    const int64_t want = (rows + G - 1) / G;
    const int grid = int(want < plan->sm_count ? want : plan->sm_count);
    if (x_bf16) {
        b4k::k_inv4096<G, true><<<grid, G * b4k::kThreads, S::kBytes, st>>>(ymap, plan->img_b4096, plan->img_i4096,
                                                                            plan->form_flag + 1, plan->gsign4096, x, ldx,
                                                                            int(rows), plan->status_word, nullptr,
                                                                            b4k::InvUpper{});
    } else {
        b4k::k_inv4096<G, false><<<grid, G * b4k::kThreads, S::kBytes, st>>>(ymap, plan->img_b4096, plan->img_i4096,
                                                                             plan->form_flag + 1, plan->gsign4096, x, ldx,
                                                                             int(rows), plan->status_word, nullptr,
                                                                             b4k::InvUpper{});
    }
    return cudaGetLastError();
}

// n = 8192, bf16 rows in, bf16 or fp32 rows out: the inverse kernel's wide mode, even CTAs on the lower halves of x, odd
// CTAs on the upper halves
cudaError_t inv8192_launch(bfq_plan* plan, const void* y, int64_t rows, int64_t ldy, void* x, bool x_bf16, int64_t ldx,
                           cudaStream_t st) {
    constexpr int G = 4;
    using S = b4k::InvSmem<G>;
    static bool attr_set[kMaxDevices] = {false};
    if (!attr_set[plan->device]) {
        cudaError_t e = cudaFuncSetAttribute(b4k::k_inv4096<G, true, false, true>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                             int(S::kBytes));
        if (e == cudaSuccess)
            e = cudaFuncSetAttribute(b4k::k_inv4096<G, false, false, true>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                     int(S::kBytes));
        if (e != cudaSuccess) return e;
        attr_set[plan->device] = true;
    }
    CUtensorMap ymap;  // whole rows of 8192 bf16 = 128 lines of 128 bytes
    {
        const cuuint64_t dims[3] = {64, 128, static_cast<cuuint64_t>(rows)};
        const cuuint64_t strides[2] = {128, static_cast<cuuint64_t>(ldy) * 2};
        const cuuint32_t box[3] = {64, 128, 1};
        const cuuint32_t estr[3] = {1, 1, 1};
        if (encode_tiled()(&ymap, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void*>(y), dims, strides, box, estr,
                           CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
                           CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
            return cudaErrorInvalidValue;
    }
    const int64_t want = (rows + G - 1) / G;
    const int per_half = plan->sm_count / 2 > 0 ? plan->sm_count / 2 : 1;
    const int grid = 2 * int(want < per_half ? want : per_half);
    const b4k::InvUpper upper{plan->img_b8192[1], plan->img_i8192[1], plan->form_flag + 2, plan->gsign8192[1]};
    const float2* tw12 = plan->tw + 12 * f4k::kN;
    if (x_bf16) {
        b4k::k_inv4096<G, true, false, true><<<grid, G * b4k::kThreads, S::kBytes, st>>>(
            ymap, plan->img_b8192[0], plan->img_i8192[0], plan->form_flag + 1, plan->gsign8192[0], x, ldx, int(rows),
            plan->status_word, tw12, upper);
    } else {
        b4k::k_inv4096<G, false, false, true><<<grid, G * b4k::kThreads, S::kBytes, st>>>(
            ymap, plan->img_b8192[0], plan->img_i8192[0], plan->form_flag + 1, plan->gsign8192[0], x, ldx, int(rows),
            plan->status_word, tw12, upper);
    }
    return cudaGetLastError();
}

}  // namespace bfq
