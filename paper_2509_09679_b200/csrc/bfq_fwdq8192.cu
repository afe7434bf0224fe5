// Tuned forward + INT2 quantization for n = 8192 bf16 rows on sm_100a.
//
// Stages 0-11 of the 13-stage transform never leave a half of the row (their pair strides are at most
// 2048), so a row is two independent 4096-point transforms, each with its own angles, followed by one
// stage that pairs element i of the lower half with element i of the upper half.  The 13 stages of
// rotation constants (425984 bytes) do not fit the tensor memory of one SM, but each half's twelve
// stages do.  So the kernel runs as clusters of two CTAs on the two SMs of a processor cluster:
// CTA rank h holds the constants of half h in its tensor memory and runs the 12-stage pipeline of the
// n = 4096 kernel (same thread roles, phases, regroupings: bfq_n4096.cuh) on half h of every row the
// cluster owns.  For stage 12 the two CTAs swap half of their registers through distributed shared
// memory (rank 0 finishes packed registers 0-7 of both halves, rank 1 registers 8-15), rotate with a
// general 2x2 form that also restores the signs the angle reduction tracked, exchange their absmax,
// and each writes the INT2 codes of the elements it finished.  Every cross-CTA wait is a bounded
// mbarrier wait; the cluster-wide barriers at entry and exit involve every thread unconditionally.
// Stages 0-11 rotate in the scaled two-FMA form of the n = 4096 kernel (every element carries the product of the
// cosines it has been through; stage 12's general 2x2 absorbs the factors), with the three-shear form as the fallback
// the table build selects when a factor leaves [2^-64, 1].
#include <type_traits>

#include "bfq_fast.h"
#include "bfq_generic.cuh"
#include "bfq_n4096.cuh"

namespace bfq {
namespace f8k {
using namespace ptx;
using namespace f4k;

constexpr int kN8 = 8192;
constexpr int kCols8 = 384 + 64;  // 12 stages of this half + this rank's share of stage 12
enum : int { kFormScaled = 0, kFormShear = 1, kFormHadamard = 2 };  // how stages 0..11 rotate (the image must match)

template <int G>
struct Smem {
    static constexpr uint32_t kInOff = 0;                                  // [G][kInSlots][kRowBytes]
    static constexpr uint32_t kExOff = kInOff + G * kInSlots * kRowBytes;  // [G][2][kExBytes]
    static constexpr uint32_t kPeerOff = kExOff + G * 2 * kExBytes;        // [G][8][128] packed pairs from the peer
    static constexpr uint32_t kAmaxOff = kPeerOff + G * 8 * kGroupThreads * 8;  // float [G][2 parities][8]
    static constexpr uint32_t kBarOff = kAmaxOff + 64 * G;                 // mbarriers [G][kInSlots + 2]
    static constexpr uint32_t kTmemOff = kBarOff + 8 * G * (kInSlots + 2);
    static constexpr uint32_t kUsed = kTmemOff + 16;
    static constexpr uint32_t kBytes = kUsed + 1024;
};

struct ExAddr {
    uint32_t w1, r1, w2, r2;
    int bar;
};

__device__ __forceinline__ void regroup1(u64 (&P)[16], const ExAddr& ex) {
#pragma unroll
    for (int m = 0; m < 16; ++m) sts64(ex.w1 + ex1_wr_local(m), P[m]);
    __syncwarp();
#pragma unroll
    for (int m = 0; m < 16; ++m) P[m] = lds64(ex.r1 + ex1_rd_local(m));
}
__device__ __forceinline__ void regroup2(u64 (&P)[16], const ExAddr& ex) {
#pragma unroll
    for (int m = 0; m < 16; ++m) {
        uint32_t lo, hi;
        unpack2u(P[m], lo, hi);
        sts32(ex.w2 + ex2_wr_local(m, 0), lo);
        sts32(ex.w2 + ex2_wr_local(m, 1), hi);
    }
    bar_sync(ex.bar, kGroupThreads);
#pragma unroll
    for (int m = 0; m < 16; ++m) P[m] = lds64(ex.r2 + ex2_rd_local(m));
}

// 12 three-shear stages in chunks of 32 constants; chunk C is in Tcur, chunk C+1 (after the last stage:
// the first half of this rank's stage-12 constants) is requested right after the wait
template <int FORM, int C, class F>
__device__ __forceinline__ void run_chunks(u64 (&P)[16], uint32_t (&Tcur)[32], uint32_t (&Tnext)[32], uint32_t tbase,
                                           const ExAddr& ex, const Turn& turn, F&& issue_next) {
    if constexpr (C == 0 || C == 4 || C == 8) turn.acquire();
    tmem_wait_ld32(Tcur);
    tmem_ld32(tbase + 32 * (C + 1), Tnext);
    if constexpr (FORM == kFormScaled) {
        stage_scaled<C & 3, 0, 8, 32>(P, Tcur);
    } else {
        stage_lift<C & 3, 0, 8, 32>(P, Tcur);
    }
    if constexpr (C == 3) {
        turn.pass();
        regroup1(P, ex);
    }
    if constexpr (C == 7) {
        turn.pass();
        regroup2(P, ex);
        issue_next();
    }
    if constexpr (C == 11) turn.pass();  // before the exchange with the peer CTA: no group waits on it with a token in hand
    if constexpr (C + 1 < 12) run_chunks<FORM, C + 1>(P, Tnext, Tcur, tbase, ex, turn, issue_next);
}

// stage 12 on four (lower-half, upper-half) register pairs: out_lo = k1*a + k2*b, out_hi = k3*a + k4*b
template <int I0>
__device__ __forceinline__ void stage12_quad(u64 (&A)[8], u64 (&B)[8], const uint32_t (&T)[32]) {
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        const u64 K1 = pack2u(T[8 * i], T[8 * i + 1]), K2 = pack2u(T[8 * i + 2], T[8 * i + 3]);
        const u64 K3 = pack2u(T[8 * i + 4], T[8 * i + 5]), K4 = pack2u(T[8 * i + 6], T[8 * i + 7]);
        const u64 a = A[I0 + i], b = B[I0 + i];
        A[I0 + i] = fma2(K2, b, mul2(K1, a));
        B[I0 + i] = fma2(K4, b, mul2(K3, a));
    }
}

struct RuntimeRank {
    uint32_t value;
};

// the fixed Hadamard rotation: twelve constant-free stages with the same two regroupings, no tokens
template <class F>
__device__ __forceinline__ void run_hadamard(u64 (&P)[16], const ExAddr& ex, F&& issue_next) {
    stage_hadamard<0>(P), stage_hadamard<1>(P), stage_hadamard<2>(P), stage_hadamard<3>(P);
    regroup1(P, ex);
    stage_hadamard<0>(P), stage_hadamard<1>(P), stage_hadamard<2>(P), stage_hadamard<3>(P);
    regroup2(P, ex);
    issue_next();
    stage_hadamard<0>(P), stage_hadamard<1>(P), stage_hadamard<2>(P), stage_hadamard<3>(P);
}
// ... and its last stage with the 1/sqrt(8192) of all thirteen
__device__ __forceinline__ void stage12_hadamard(u64 (&A)[8], u64 (&B)[8]) {
    const float k = 0.011048543456039806f;  // 2^-6.5
    const u64 kk = pack2(k, k), nk = pack2(-k, -k);
#pragma unroll
    for (int i = 0; i < 8; ++i) {
        const u64 ka = mul2(kk, A[i]), b = B[i];
        A[i] = fma2(kk, b, ka);
        B[i] = fma2(nk, b, ka);
    }
}

// two INT2 codes of a packed pair (elements e, e+1) as a nibble: bits 0-1 = code(e), bits 2-3 = code(e+1)
__device__ __forceinline__ uint32_t nibble_int2(u64 v, u64 inv2, float inv, bool plain) {
    if (plain) {
        // |v * inv| <= 1.0005: v*inv + 1.5*2^23 has q in {-1, 0, 1} (mod 4) in its two low bits
        uint32_t lo, hi;
        unpack2u(fma2(v, inv2, pack2(12582912.0f, 12582912.0f)), lo, hi);
        return (lo & 3u) | ((hi & 3u) << 2);
    }
    float a, b;
    unpack2(v, a, b);
    const int qa = static_cast<int>(fminf(fmaxf(rintf(a * inv), -2.f), 1.f));
    const int qb = static_cast<int>(fminf(fmaxf(rintf(b * inv), -2.f), 1.f));
    return (static_cast<uint32_t>(qa) & 3u) | ((static_cast<uint32_t>(qb) & 3u) << 2);
}

// BITS = 2 (the tuned workload), 4 or 8: only the epilogue differs.  BITS = 16: the rotated rows themselves in bf16
// (`codes` then points to them, leading dimension ldy); the absmax hand-shake between the two CTAs is kept, since it is
// also what tells a CTA that its peer has read the exchange box of the row.
// STEP: token passing between the row groups of a CTA as in the n = 4096 kernel (0: none).
// ROWS (BITS = 2, 4, 8): the rotated rows are written as well, in bf16, to `yrows` (leading dimension ldy).
// IN_F32: fp32 rows (a half row is 16 KB): one input slot per group instead of two, re-armed after the second
// regrouping's barrier.  BITS = 32 (with IN_F32): the rotated rows in fp32 (`codes` then points to them).
// HADAMARD: y = H x instead of the butterfly (no constants: `img` and `form` are not read, tensor memory stays empty).
template <int G, int BITS, int STEP = 2, bool ROWS = false, bool IN_F32 = false, bool HADAMARD = false>
__global__ void __launch_bounds__(G * kGroupThreads, 1)
k_fwdq8192(const __grid_constant__ CUtensorMap map_lo, const __grid_constant__ CUtensorMap map_hi,
           const float* __restrict__ img, const int* __restrict__ form, uint8_t* __restrict__ codes,
           uint16_t* __restrict__ scales, int64_t ldy, int rows, int* __restrict__ status,
           __nv_bfloat16* __restrict__ yrows) {
    using S = Smem<G>;
    extern __shared__ uint8_t smem_raw[];
    const uint32_t sbase = (smem_u32(smem_raw) + 1023u) & ~1023u;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int q = warp & 3, g = warp >> 2;
    const int t = q * 32 + lane;                  // role within the group: 0..127
    const uint32_t rank = cluster_ctarank();      // which half of every row this CTA transforms
    const uint32_t peer = rank ^ 1u;

    const uint32_t bar_in = sbase + S::kBarOff + 8 * g * (kInSlots + 2);  // [kInSlots] TMA, then swap, then absmax
    const uint32_t bar_swap = bar_in + 8 * kInSlots, bar_amax = bar_swap + 8;
    grid_dep_launch();
    if (warp == 0) tmem_alloc512(sbase + S::kTmemOff);
    if (t == 0) {
        for (int k = 0; k < kInSlots; ++k) mbar_init(bar_in + 8 * k, 1);
        mbar_init(bar_swap, 1);  // per row: this thread's arrive.expect_tx + the peer's 8 KB of asynchronous stores
        mbar_init(bar_amax, 1);
        mbar_init_fence();
    }
    tmem_fence_before();
    __syncthreads();
    tmem_fence_after();
    cluster_sync_all();  // the peer's barriers exist before anything arrives on them
    grid_dep_wait();     // everything above overlaps the end of the kernel before this one
    uint32_t tmem_base;
    asm volatile("ld.shared.u32 %0, [%1];" : "=r"(tmem_base) : "r"(sbase + S::kTmemOff));
    const uint32_t tlane = tmem_base + (static_cast<uint32_t>(q * 32) << 16);

    // row r belongs to group (r / n_clusters) % G of cluster r % n_clusters
    const int n_clusters = gridDim.x >> 1;
    const int first = g * n_clusters + (blockIdx.x >> 1);
    const int stride = n_clusters * G;
    const int count = first < rows ? (rows - first + stride - 1) / stride : 0;
    // rows of group 0, the largest count of the CTA: every group takes that many turns with a token
    const int turns = static_cast<int>(blockIdx.x >> 1) < rows ? (rows - (blockIdx.x >> 1) + stride - 1) / stride : 0;
    static_assert(STEP >= 0 && (STEP == 0 || G % STEP == 0), "the rings must have equal length");
    constexpr int kRings = STEP == 0 ? 1 : STEP;
    Turn turn;
    turn.on = STEP > 0 && !HADAMARD;
    turn.wait_id = kTurnBar0 + g;
    turn.pass_id = kTurnBar0 + (g + STEP) % G;
    const bool seeds_ring = (g + STEP) % G < kRings;  // this group's successor starts with the token
    const uint32_t in_base = sbase + S::kInOff + g * kInSlots * kRowBytes;
    const CUtensorMap* tmap = rank == 0 ? &map_lo : &map_hi;

    constexpr int kSlotsUsed = IN_F32 ? 1 : kInSlots;
    constexpr uint32_t kSlotBytes = IN_F32 ? 2 * kRowBytes : kRowBytes;
    static_assert(kInSlots == 2, "an fp32 half row takes the group's two bf16 slots");
    if (t == 0) {
        for (int k = 0; k < kSlotsUsed && k < count; ++k) {
            mbar_expect_tx(bar_in + 8 * k, kSlotBytes);
            tma_load_3d(in_base + k * kSlotBytes, tmap, 0, 0, first + k * stride, bar_in + 8 * k);
        }
    }
    // constants of this thread's role: image [form][rank][column quad][role][4], all loads in flight together; the
    // scaled-form image is fetched on the assumption that the table build selected it
    constexpr int kFillBlocks = (kCols8 / 16 + G - 1) / G;
    bool shear = false;
    if constexpr (!HADAMARD) {
        float4 fill[kFillBlocks][4];
        auto fetch_image = [&](int which) {
            const float4* base = reinterpret_cast<const float4*>(img) + (static_cast<size_t>(which) * 2 + rank) * (kCols8 / 4) * 128;
#pragma unroll
            for (int j = 0; j < kFillBlocks; ++j) {
                const int b = g + j * G;
                if (b < kCols8 / 16) {
#pragma unroll
                    for (int i = 0; i < 4; ++i) fill[j][i] = __ldg(base + (4 * b + i) * 128 + t);
                }
            }
        };
        fetch_image(kFormScaled);
        shear = __ldg(form) != 0;
        if (shear) fetch_image(kFormShear);
#pragma unroll
        for (int j = 0; j < kFillBlocks; ++j) {
            const int b = g + j * G;
            if (b < kCols8 / 16) {
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
    }
    tmem_fence_before();
    __syncthreads();
    tmem_fence_after();

    ExAddr ex;
    {
        const uint32_t eb1 = sbase + S::kExOff + g * 2 * kExBytes, eb2 = eb1 + kExBytes;
        const uint32_t t4 = (t >> 4) & 1, t5 = (t >> 5) & 1, t6 = (t >> 6) & 1;
        ex.w1 = eb1 + 4u * (2u * (t & 15) + 32u * (t >> 4));
        ex.r1 = eb1 + 4u * (258u * (t & 15) + 32u * (t >> 4));
        ex.w2 = eb2 + 4u * ((t & 15) + 2064u * t4 + 512u * t5 + 1024u * t6);
        ex.r2 = eb2 + 4u * (2u * (t & 15) + 32u * (t >> 4));
        ex.bar = 1 + g;
    }
    // (fp32 rows: runs of 64 bytes at byte 64 (t & 15) + 2048 (t >> 4) + 1024 h: chunks 4 (t & 1) + c of line
    // ((t & 15) >> 1) + 16 (t >> 4) + 8 h)
    const uint32_t in_line = IN_F32 ? ((t & 15) >> 1) * 128u + (t >> 4) * 2048u : ((t >> 2) & 3) * 128u + (t >> 4) * 1024u;
    const uint32_t in_x = IN_F32 ? ((((t & 1) << 2) ^ ((t >> 1) & 7)) << 4) : ((((t & 3) << 1) ^ ((t >> 2) & 3)) << 4);
    const uint32_t my_box = sbase + S::kPeerOff + (g * 8 * kGroupThreads + t) * 8;  // + i * 1024: register i from the peer
    const uint32_t peer_box = map_to_cta(my_box, peer);
    const uint32_t amax_base = sbase + S::kAmaxOff + g * 64;                         // [2][8] floats
    const uint32_t peer_amax = map_to_cta(amax_base, peer);
    const uint32_t peer_bar_swap = map_to_cta(bar_swap, peer), peer_bar_amax = map_to_cta(bar_amax, peer);
    // INT2 codes: elements 2t + 256m, +1 are a nibble of byte (t >> 1) + 64m; lanes t, t^1 share the byte.  The
    // even lane stores the bytes of the lower half of the row, the odd lane those of the upper half.
    uint8_t* const out_t = codes + (t >> 1) + 64 * 8 * rank + ((t & 1) ? 1024 : 0);

    // Waiting for the peer CTA: with bf16 rows and the butterfly one warp of the row group polls and the other three
    // sleep at the group's named barrier (1.4 % faster than all four polling); with fp32 rows or the Hadamard stages
    // the extra barrier costs more than the polling (4.8 % / 3.5 % slower), so there every warp polls
    constexpr bool kOnePoller = !IN_F32 && !HADAMARD;
    auto wait_peer = [&](uint32_t bar, uint32_t parity) {
        if constexpr (kOnePoller) {
            if (q == 0) mbar_wait_cluster_bounded(bar, parity, status);
            bar_sync(ex.bar, kGroupThreads);
        } else {
            mbar_wait_cluster_bounded(bar, parity, status);
        }
    };
    // the whole row loop exists once per stage form: the choice is made once per launch, outside the loop
    // ... and, where rows are the output (BITS >= 16), once per CTA rank, so that "registers 0-7 are mine, 8-15 the peer's"
    // (or the reverse) is a renaming at compile time instead of register moves per row; a CTA only ever runs its own
    // copy.  Measured on 65536 rows: bf16 rows out 0.614 -> 0.596 ms; the code variants got slower with it (INT2 0.658 ->
    // 0.681 ms, INT4 0.633 -> 0.666 ms), so they keep the rank as a run-time value.
    auto row_loop = [&](auto form_tag, auto rank_tag) {
    constexpr int FORM = decltype(form_tag)::value;
    const uint32_t rank = rank_tag.value;
    u64 P[16];
    uint32_t T0[32], T1[32];

    if (seeds_ring) turn.pass();
    for (int k = 0; k < count; ++k) {
        const int row = first + k * stride;
        const int slot = IN_F32 ? 0 : (k & 1);
        if constexpr (FORM != kFormHadamard) tmem_ld32(tlane, T0);
        mbar_wait_bounded(bar_in + 8 * slot, (IN_F32 ? k : (k >> 1)) & 1, status);
        const uint32_t src = in_base + slot * kSlotBytes + in_line;
        if constexpr (IN_F32) {
            // run h holds elements 4c .. 4c+3 in 16-byte chunk c; element m of half h is half h of P[m]
            uint4 w[2][4];
#pragma unroll
            for (int h = 0; h < 2; ++h)
#pragma unroll
                for (int c = 0; c < 4; ++c) w[h][c] = lds128(src + 1024u * h + (in_x ^ (c << 4)));
#pragma unroll
            for (int c = 0; c < 4; ++c) {
                P[4 * c + 0] = pack2u(w[0][c].x, w[1][c].x);
                P[4 * c + 1] = pack2u(w[0][c].y, w[1][c].y);
                P[4 * c + 2] = pack2u(w[0][c].z, w[1][c].z);
                P[4 * c + 3] = pack2u(w[0][c].w, w[1][c].w);
            }
        } else {
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
                    P[8 * c + 2 * j + 0] = pack2u(bf16_lo(a[j]), bf16_lo(b[j]));
                    P[8 * c + 2 * j + 1] = pack2u(a[j] & 0xFFFF0000u, b[j] & 0xFFFF0000u);
                }
            }
        }
        auto issue_next = [&]() {
            if (t == 0 && k + kSlotsUsed < count) {
                mbar_expect_tx(bar_in + 8 * slot, kSlotBytes);
                tma_load_3d(in_base + slot * kSlotBytes, tmap, 0, 0, first + (k + kSlotsUsed) * stride, bar_in + 8 * slot);
            }
        };
        if constexpr (FORM == kFormHadamard) {
            run_hadamard(P, ex, issue_next);
        } else {
            run_chunks<FORM, 0>(P, T0, T1, tlane, ex, turn, issue_next);  // the first 32 of this rank's stage-12 constants are now requested in T0
        }

        // ---- stage 12: rank 0 finishes registers 0-7 of both halves, rank 1 registers 8-15 ----
        u64 A[8], B[8];  // lower-half / upper-half values of the registers this rank finishes
        if (t == 0) {  // this row's incoming bytes: 8 registers from each of the peer's 128 threads, then its absmax
            mbar_expect_tx(bar_swap, 8 * 8 * kGroupThreads);
            mbar_expect_tx(bar_amax, 4);
        }
        if (rank == 0) {
#pragma unroll
            for (int i = 0; i < 8; ++i) st_async_b64(peer_box + i * 1024u, P[8 + i], peer_bar_swap);
        } else {
#pragma unroll
            for (int i = 0; i < 8; ++i) st_async_b64(peer_box + i * 1024u, P[i], peer_bar_swap);
        }
        wait_peer(bar_swap, k & 1);
        if (rank == 0) {
#pragma unroll
            for (int i = 0; i < 8; ++i) A[i] = P[i], B[i] = lds64(my_box + i * 1024u);
        } else {
#pragma unroll
            for (int i = 0; i < 8; ++i) A[i] = lds64(my_box + i * 1024u), B[i] = P[8 + i];
        }
        if constexpr (FORM == kFormHadamard) {
            stage12_hadamard(A, B);
        } else {
            tmem_wait_ld32(T0);
            tmem_ld32(tlane + 416, T1);
            stage12_quad<0>(A, B, T0);
            tmem_wait_ld32(T1);
            stage12_quad<4>(A, B, T1);
        }

        // ---- absmax of the whole row: thread, warp, group, then the peer's half ----
        float m0 = 0.f, m1 = 0.f;
#pragma unroll
        for (int i = 0; i < 8; ++i) {
            float a0, a1, b0, b1;
            unpack2(A[i], a0, a1);
            unpack2(B[i], b0, b1);
            m0 = fmaxf(m0, fmaxf(fabsf(a0), fabsf(b0)));
            m1 = fmaxf(m1, fmaxf(fabsf(a1), fabsf(b1)));
        }
        // non-negative floats order like their bit patterns: one integer max-reduction over the warp
        float amax = fmaxf(m0, m1);
        const uint32_t aslot = amax_base + (k & 1) * 32;
        sts32_if(lane == 0, aslot + q * 4, __reduce_max_sync(0xFFFFFFFFu, __float_as_uint(amax)));
        bar_sync(ex.bar, kGroupThreads);
        {
            const uint4 o = lds128(aslot);
            amax = fmaxf(fmaxf(__uint_as_float(o.x), __uint_as_float(o.y)),
                         fmaxf(__uint_as_float(o.z), __uint_as_float(o.w)));
        }
        if (t == 0) {
            st_async_b32(peer_amax + (k & 1) * 32 + 16, __float_as_uint(amax), peer_bar_amax);
        }
        wait_peer(bar_amax, k & 1);
        amax = fmaxf(amax, __uint_as_float(lds32(aslot + 16)));
        float inv;
        static_assert(!(ROWS && BITS == 16), "BITS = 16 writes the rows already");
        if constexpr (BITS == 16 || ROWS) {
            // A[i] holds elements 2048 rank + 256 i + 2 t (+1), B[i] the same 4096 further on: one 32-bit word each
            uint32_t* yrow = reinterpret_cast<uint32_t*>((BITS == 16 ? reinterpret_cast<__nv_bfloat16*>(codes) : yrows) +
                                                         static_cast<int64_t>(row) * ldy);
#pragma unroll
            for (int i = 0; i < 8; ++i) {
                float a0, a1, b0, b1;
                unpack2(A[i], a0, a1);
                unpack2(B[i], b0, b1);
                const __nv_bfloat162 va = __floats2bfloat162_rn(a0, a1), vb = __floats2bfloat162_rn(b0, b1);
                yrow[1024 * rank + 128 * i + t] = *reinterpret_cast<const uint32_t*>(&va);
                yrow[2048 + 1024 * rank + 128 * i + t] = *reinterpret_cast<const uint32_t*>(&vb);
            }
        }
        if constexpr (BITS == 32) {
            // one 64-bit word of the fp32 row per packed register
            u64* yrow = reinterpret_cast<u64*>(reinterpret_cast<float*>(codes) + static_cast<int64_t>(row) * ldy);
#pragma unroll
            for (int i = 0; i < 8; ++i) {
                yrow[1024 * rank + 128 * i + t] = A[i];
                yrow[2048 + 1024 * rank + 128 * i + t] = B[i];
            }
        }
        if constexpr (BITS == 16 || BITS == 32) continue;
        constexpr int kQmax = BITS >= 16 ? 1 : (1 << (BITS - 1)) - 1;
        const uint16_t s16 = row_scale_fast<kQmax>(amax, &inv);
        stg16_if(rank == 0 && t == 0, scales + row, s16);
        if constexpr (BITS != 2 && BITS < 16) {
            // A[i] holds elements 2048 rank + 256 i + 2 t (+1) of the row, B[i] the same 4096 further on: with 4 or 8 bits
            // a register pair is one byte / one 16-bit word of its own.  |v * inv| < qmax + 1/2 for a normal, unsaturated
            // scale, so v * inv + 1.5 * 2^23 carries the two's complement code in its low mantissa bits.
            const bool plain = (((s16 >> 10) & 31u) != 0u) && (s16 != 0x7BFFu);
            const u64 inv2 = pack2(inv, inv);
            // u = code + 2^(BITS-1) in the low BITS bits of v * inv + (1.5 * 2^23 + 2^(BITS-1)), the bits above them up to
            // bit 22 zero: (hi << BITS) + lo has both fields in place; the XOR turns offset binary into two's complement
            constexpr float kMagic = 12582912.0f + float(1 << (BITS - 1));
            const u64 magic2 = pack2(kMagic, kMagic);
            auto code_fast = [&](u64 v) -> uint32_t {
                uint32_t lo, hi;
                unpack2u(fma2(v, inv2, magic2), lo, hi);
                return ((hi << BITS) + lo) ^ ((1u << (BITS - 1)) | (1u << (2 * BITS - 1)));
            };
            auto code_slow = [&](u64 v) -> uint32_t {
                float a, b;
                unpack2(v, a, b);
                const uint32_t lo = static_cast<uint32_t>(static_cast<int>(fminf(fmaxf(rintf(a * inv), float(-kQmax - 1)), float(kQmax))));
                const uint32_t hi = static_cast<uint32_t>(static_cast<int>(fminf(fmaxf(rintf(b * inv), float(-kQmax - 1)), float(kQmax))));
                constexpr uint32_t kMask = (1u << BITS) - 1u;
                return (lo & kMask) | ((hi & kMask) << BITS);
            };
            const size_t base = static_cast<size_t>(row) * (kN8 * BITS / 8);
            auto store_all = [&](auto&& code2) {  // the scale decides once per row which of the two bodies runs
#pragma unroll
                for (int i = 0; i < 8; ++i) {
                    const uint32_t ca = code2(A[i]), cb = code2(B[i]);
                    if constexpr (BITS == 4) {
                        codes[base + 1024 * rank + 128 * i + t] = static_cast<uint8_t>(ca);
                        codes[base + 2048 + 1024 * rank + 128 * i + t] = static_cast<uint8_t>(cb);
                    } else {
                        uint16_t* c16 = reinterpret_cast<uint16_t*>(codes + base);
                        c16[1024 * rank + 128 * i + t] = static_cast<uint16_t>(ca);
                        c16[2048 + 1024 * rank + 128 * i + t] = static_cast<uint16_t>(cb);
                    }
                }
            };
            if (plain) {
                store_all(code_fast);
            } else {
                store_all(code_slow);
            }
            continue;
        }

        const uint32_t e16 = (s16 >> 10) & 31u;
        const bool plain = (e16 != 0u) && (s16 != 0x7BFFu);  // normal fp16 scale: |v*inv| <= 1.0005, no clipping
        const u64 inv2 = pack2(inv, inv);
        uint8_t* out = out_t + static_cast<size_t>(row) * (kN8 / 4);
        // the nibbles (two codes each) of the lower-half registers in the low halves of the bytes of two words (registers
        // 0-3, 4-7), those of the upper half in two more
        uint32_t wa[2] = {0u, 0u}, wb[2] = {0u, 0u};
        if (plain) {
            // v * inv + (1.5 * 2^23 + 2) has u = code + 2 in {1, 2, 3} in its low bits above the constant pattern
            // C = 0x4B400000, so hi * 4 + lo = 5 C + (4 u_hi + u_lo) and a Horner chain over four registers yields the sum
            // of the nibbles times 256^i plus a constant; one subtraction removes it, one XOR turns u into the code
            const u64 magic2 = pack2(12582914.0f, 12582914.0f);
#pragma unroll
            for (int h = 0; h < 2; ++h) {
#pragma unroll
                for (int i = 3; i >= 0; --i) {
                    uint32_t lo, hi;
                    unpack2u(fma2(A[4 * h + i], inv2, magic2), lo, hi);
                    wa[h] = wa[h] * 256u + (hi * 4u + lo);
                    unpack2u(fma2(B[4 * h + i], inv2, magic2), lo, hi);
                    wb[h] = wb[h] * 256u + (hi * 4u + lo);
                }
                constexpr uint32_t kBias = static_cast<uint32_t>((5ull * 0x4B400000ull * 0x01010101ull) & 0xFFFFFFFFull);
                wa[h] = (wa[h] - kBias) ^ 0x0A0A0A0Au;
                wb[h] = (wb[h] - kBias) ^ 0x0A0A0A0Au;
            }
        } else {
#pragma unroll
            for (int i = 0; i < 8; ++i) {
                wa[i >> 2] |= nibble_int2(A[i], inv2, inv, false) << (8 * (i & 3));
                wb[i >> 2] |= nibble_int2(B[i], inv2, inv, false) << (8 * (i & 3));
            }
        }
        // even lane: bytes of the lower half = its nibbles + the odd lane's; odd lane: bytes of the upper half = the even
        // lane's nibbles + its own.  One exchange per word, then the two nibbles of a byte side by side.
        const bool odd = t & 1;
#pragma unroll
        for (int h = 0; h < 2; ++h) {
            const uint32_t got = __shfl_xor_sync(0xFFFFFFFFu, odd ? wa[h] : wb[h], 1);
            const uint32_t bytes = (odd ? got : wa[h]) + ((odd ? wb[h] : got) << 4);
#pragma unroll
            for (int j = 0; j < 4; ++j) out[64 * (4 * h + j)] = static_cast<uint8_t>(bytes >> (8 * j));
        }
    }
    // a group with fewer rows than group 0 keeps the tokens moving
    for (int k = count; k < turns; ++k) {
#pragma unroll
        for (int ph = 0; ph < 3; ++ph) turn.acquire(), turn.pass();
    }
    if (g < kRings) turn.acquire();  // each ring's first group takes its token back: no arrival stays pending
    };
    auto for_rank = [&](auto form_tag) {
        if constexpr (BITS >= 16) {
            if (rank == 0) {
                row_loop(form_tag, std::integral_constant<uint32_t, 0>());
            } else {
                row_loop(form_tag, std::integral_constant<uint32_t, 1>());
            }
        } else {
            row_loop(form_tag, RuntimeRank{rank});
        }
    };
    if constexpr (HADAMARD) {
        for_rank(std::integral_constant<int, kFormHadamard>());
    } else if (!shear) {
        for_rank(std::integral_constant<int, kFormScaled>());
    } else {
        for_rank(std::integral_constant<int, kFormShear>());
    }

    tmem_fence_before();
    __syncthreads();
    if (warp == 0) tmem_dealloc512(tmem_base);
    cluster_sync_all();  // neither CTA leaves while the other may still write into its shared memory
}

// ---- table preparation -----------------------------------------------------------------------------------
// Step 1 (one thread per angle): cos/sin table entry (fp32 for the generic kernels, double for step 2), the
// three-shear constants of the angle reduced to |phi| <= pi/2 and whether the reduction negates the pair (iff
// cos(theta) < 0: phi = theta -+ pi, sin(phi) = -sin(theta), tan(phi/2) = sin(phi) / (1 + cos(phi))).
__global__ void __launch_bounds__(256) k_prep_angles8192(const float* __restrict__ theta, float2* __restrict__ tw,
                                                          float4* __restrict__ prep, double2* __restrict__ cs,
                                                          int* __restrict__ form) {
    const int k = blockIdx.x * blockDim.x + threadIdx.x;
    if (k == 0) *form = kFormScaled;  // step 2 raises it when the scaled form is out of range
    if (k >= 13 * (kN8 / 2)) return;
    const double th = static_cast<double>(theta[k]);
    double sn, c;
    sincos(th, &sn, &c);
    tw[k] = make_float2(static_cast<float>(c), static_cast<float>(sn));
    cs[k] = make_double2(c, sn);
    const bool f = c < 0.0;
    const double sp = f ? -sn : sn, cp = f ? -c : c;
    prep[k] = make_float4(static_cast<float>(-sp / (1.0 + cp)), static_cast<float>(sp), static_cast<float>(c),
                          static_cast<float>(sn));
}

// factor carried by element i (0..4095) of half `half` when it enters stage s <= 12: the product of the cosines of
// the pairs it belonged to in stages 0..s-1 (stages 0..11 pair inside the half; pair j of such a stage belongs to the
// upper half iff j >= 2048).  Its sign is the tracked sign of the three-shear form.
__device__ __forceinline__ double factor_before8(const double2* __restrict__ cs, int half, int i, int s) {
    double c[12];
#pragma unroll
    for (int sp = 0; sp < 12; ++sp) {  // all loads issued together
        const int j = ((i >> (sp + 1)) << sp) | (i & ((1 << sp) - 1));
        c[sp] = sp < s ? cs[sp * (kN8 / 2) + half * (kN / 2) + j].x : 1.0;
    }
    double d = 1.0;
#pragma unroll
    for (int sp = 0; sp < 12; ++sp) d *= c[sp];
    return d;
}

// Step 2 (one thread per angle): constants of pair (s, j) into both images of the CTA rank that uses them,
// img[form][rank][column quad][role][4]; raises *form when an element's factor leaves the scaled form's range.
__global__ void __launch_bounds__(256) k_build_image8192(const float4* __restrict__ prep, const double2* __restrict__ cs,
                                                          float* __restrict__ img, int* __restrict__ form) {
    const int k = blockIdx.x * blockDim.x + threadIdx.x;
    if (k >= 13 * (kN8 / 2)) return;
    const int s = k / (kN8 / 2), j = k % (kN8 / 2);
    const float4 p = prep[k];
    const double2 own = cs[k];
    constexpr size_t kImage = size_t(128) * kCols8;  // one (form, rank) image
    auto at = [](int r, int col) { return (col >> 2) * 512 + 4 * r + (col & 3); };
    if (s < 12) {
        const int half = j >> 11, jj = j & 2047;
        const int lo = ((jj >> s) << (s + 1)) | (jj & ((1 << s) - 1));  // inside the half
        const int hi = lo + (1 << s);
        const double da = factor_before8(cs, half, lo, s), db = factor_before8(cs, half, hi, s);
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
        const float sg = ((da < 0.0) == (db < 0.0)) ? 1.f : -1.f;
        float* scaled = img + (size_t(kFormScaled) * 2 + half) * kImage;
        float* shear = img + (size_t(kFormShear) * 2 + half) * kImage;
        const int col = 32 * s + 4 * u + h;
        shear[at(r, col)] = sg * p.x;
        shear[at(r, col + 2)] = sg * p.y;
        // k1 = -tan(theta) db/da, k2 = tan(theta) da/db, with one division
        const double w = own.y / (own.x * da * db);
        scaled[at(r, col)] = static_cast<float>(-w * db * db);
        scaled[at(r, col + 2)] = static_cast<float>(w * da * da);
        const double lim = 5.421010862427522e-20;  // 2^-64
        if (!(fabs(own.x * da) >= lim && fabs(own.x * db) >= lim)) *form = kFormShear;
    } else {
        // stage 12: element j of the lower half with element j of the upper half, in phase-3 ownership;
        // registers 0-7 are finished by rank 0, 8-15 by rank 1
        const double da = factor_before8(cs, 0, j, 12), db = factor_before8(cs, 1, j, 12);
        const int sa = da < 0.0 ? -1 : 1, sb = db < 0.0 ? -1 : 1;
        const int r = (j >> 1) & 127, m = j >> 8, h = j & 1;
        float* scaled = img + (size_t(kFormScaled) * 2 + (m >> 3)) * kImage;
        float* shear = img + (size_t(kFormShear) * 2 + (m >> 3)) * kImage;
        const int col = 384 + 8 * (m & 7) + h;
        shear[at(r, col + 0)] = p.z * sa;
        shear[at(r, col + 2)] = -p.w * sb;
        shear[at(r, col + 4)] = p.w * sa;
        shear[at(r, col + 6)] = p.z * sb;
        scaled[at(r, col + 0)] = static_cast<float>(own.x * da);
        scaled[at(r, col + 2)] = static_cast<float>(-own.y * db);
        scaled[at(r, col + 4)] = static_cast<float>(own.y * da);
        scaled[at(r, col + 6)] = static_cast<float>(own.x * db);
    }
}

}  // namespace f8k

// ---- host side ---------------------------------------------------------------------------------------------
// two forms x two CTA ranks
size_t fwdq8192_image_bytes() { return size_t(4) * 128 * f8k::kCols8 * sizeof(float); }
// per angle: float4 (three-shear constants, cos, sin) and double2 (cos, sin)
size_t fwdq8192_prep_bytes() { return size_t(13) * (f8k::kN8 / 2) * (sizeof(float4) + sizeof(double2)); }

cudaError_t fwdq8192_set_angles(const bfq_plan* plan, const float* theta, cudaStream_t st) {
    const int count = 13 * (f8k::kN8 / 2);
    float4* prep = reinterpret_cast<float4*>(plan->prep8192);
    double2* cs = reinterpret_cast<double2*>(prep + count);
    f8k::k_prep_angles8192<<<(count + 255) / 256, 256, 0, st>>>(theta, plan->tw, prep, cs, plan->form_flag);
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return e;
    f8k::k_build_image8192<<<(count + 255) / 256, 256, 0, st>>>(prep, cs, plan->img8192, plan->form_flag);
    return cudaGetLastError();
}

bool fwdq8192_available(const bfq_plan* plan) {
    return plan->n == f8k::kN8 && plan->cc_major == 10 && plan->img8192 != nullptr && plan->sm_count >= 2 &&
           encode_tiled() != nullptr;
}

template <int BITS, bool ROWS = false, bool IN_F32 = false, bool HADAMARD = false>
static cudaError_t fwdq8192_launch_bits(const bfq_plan* plan, const void* x, int64_t rows, int64_t ldx, uint8_t* codes,
                                        uint16_t* scales, int64_t ldy, cudaStream_t st, void* yrows = nullptr) {
    constexpr int G = 4;
    using S = f8k::Smem<G>;
    auto kern = f8k::k_fwdq8192<G, BITS, 2, ROWS, IN_F32, HADAMARD>;
    static bool attr_set[kMaxDevices] = {false};
    if (!attr_set[plan->device]) {
        cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, int(S::kBytes));
        if (e != cudaSuccess) return e;
        attr_set[plan->device] = true;
    }
    CUtensorMap map_lo, map_hi;
    if constexpr (IN_F32) {
        const float* xf = static_cast<const float*>(x);
        if (!encode_row_map_f32(&map_lo, xf, rows, ldx) || !encode_row_map_f32(&map_hi, xf + f4k::kN, rows, ldx))
            return cudaErrorInvalidValue;
    } else {
        const uint16_t* xb = static_cast<const uint16_t*>(x);
        if (!encode_row_map(&map_lo, xb, rows, ldx) || !encode_row_map(&map_hi, xb + f4k::kN, rows, ldx))
            return cudaErrorInvalidValue;
    }
    const int64_t want = (rows + G - 1) / G;
    const int max_clusters = plan->sm_count / 2;
    const int clusters = int(want < max_clusters ? want : max_clusters);
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(2 * clusters, 1, 1);
    cfg.blockDim = dim3(G * f4k::kGroupThreads, 1, 1);
    cfg.dynamicSmemBytes = S::kBytes;
    cfg.stream = st;
    cudaLaunchAttribute attr[2];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = 2;
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;  // the set-up overlaps the previous kernel's tail
    attr[1].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 2;
    return cudaLaunchKernelEx(&cfg, kern, map_lo, map_hi, static_cast<const float*>(plan->img8192),
                              static_cast<const int*>(plan->form_flag), codes, scales, ldy, int(rows), plan->status_word,
                              static_cast<__nv_bfloat16*>(yrows));
}

cudaError_t fwdq8192_launch(const bfq_plan* plan, const void* x, int64_t rows, int64_t ldx, int bits, uint8_t* codes,
                            uint16_t* scales, cudaStream_t st) {
    if (bits == 2) return fwdq8192_launch_bits<2>(plan, x, rows, ldx, codes, scales, 0, st);
    if (bits == 4) return fwdq8192_launch_bits<4>(plan, x, rows, ldx, codes, scales, 0, st);
    return fwdq8192_launch_bits<8>(plan, x, rows, ldx, codes, scales, 0, st);
}

// codes + scales and the rotated rows in bf16 from one pass (weight folding that keeps W Q^T)
cudaError_t fwdq8192_launch_codes_rows(const bfq_plan* plan, const void* x, int64_t rows, int64_t ldx, int bits,
                                       uint8_t* codes, uint16_t* scales, void* y, int64_t ldy, cudaStream_t st) {
    if (bits == 2) return fwdq8192_launch_bits<2, true>(plan, x, rows, ldx, codes, scales, ldy, st, y);
    if (bits == 4) return fwdq8192_launch_bits<4, true>(plan, x, rows, ldx, codes, scales, ldy, st, y);
    return fwdq8192_launch_bits<8, true>(plan, x, rows, ldx, codes, scales, ldy, st, y);
}

// fp32 rows in: codes + scales (bits = 2, 4, 8), or the rotated rows in fp32 (bits = 0, y with leading dimension ldy)
cudaError_t fwdq8192_launch_f32(const bfq_plan* plan, const void* x, int64_t rows, int64_t ldx, int bits, uint8_t* codes,
                                uint16_t* scales, void* y, int64_t ldy, cudaStream_t st) {
    if (bits == 0) return fwdq8192_launch_bits<32, false, true>(plan, x, rows, ldx, static_cast<uint8_t*>(y), nullptr, ldy, st);
    if (bits == 2) return fwdq8192_launch_bits<2, false, true>(plan, x, rows, ldx, codes, scales, 0, st);
    if (bits == 4) return fwdq8192_launch_bits<4, false, true>(plan, x, rows, ldx, codes, scales, 0, st);
    return fwdq8192_launch_bits<8, false, true>(plan, x, rows, ldx, codes, scales, 0, st);
}

// y = H x (the fixed Hadamard rotation) on bf16 rows: codes + scales (bits = 2, 4, 8) or the rotated rows in bf16 (bits = 0)
cudaError_t fwdq8192_launch_hadamard(const bfq_plan* plan, const void* x, int64_t rows, int64_t ldx, int bits, uint8_t* codes,
                                     uint16_t* scales, void* y, int64_t ldy, cudaStream_t st) {
    if (bits == 0)
        return fwdq8192_launch_bits<16, false, false, true>(plan, x, rows, ldx, static_cast<uint8_t*>(y), nullptr, ldy, st);
    if (bits == 2) return fwdq8192_launch_bits<2, false, false, true>(plan, x, rows, ldx, codes, scales, 0, st);
    if (bits == 4) return fwdq8192_launch_bits<4, false, false, true>(plan, x, rows, ldx, codes, scales, 0, st);
    return fwdq8192_launch_bits<8, false, false, true>(plan, x, rows, ldx, codes, scales, 0, st);
}

// y = Q x in bf16 (the weight-only setting: activations stay 16-bit)
cudaError_t fwdq8192_launch_bf16(const bfq_plan* plan, const void* x, int64_t rows, int64_t ldx, void* y, int64_t ldy,
                                 cudaStream_t st) {
    return fwdq8192_launch_bits<16>(plan, x, rows, ldx, static_cast<uint8_t*>(y), nullptr, ldy, st);
}

}  // namespace bfq
