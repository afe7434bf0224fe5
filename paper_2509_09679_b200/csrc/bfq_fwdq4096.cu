// Tuned forward for n = 4096 bf16 rows on sm_100a: learned butterfly or fixed Walsh-Hadamard rotation, fused with
// INT4 quantization or writing the rotated rows in bf16.  The description below is the butterfly + INT4 case.
//
// Design (one persistent CTA per SM, G row groups of 128 threads):
//  * A row is owned by one group of four warps, one warp per scheduler and per tensor-memory lane
//    quarter.  The 12 stages run as three phases of four stages.  In each phase a thread holds 32
//    elements of the row as 16 packed fp32x2 registers: four index bits are the phase's stage bits
//    (so all partners are in the thread's own registers) and the fifth selects the half of the
//    packed register and is never a stage bit of that phase, so every rotation is a packed FMA.
//        phase 1: stage bits 0-3, packed along bit 8     (two runs of 16 consecutive elements)
//        phase 2: stage bits 4-7, packed along bit 8
//        phase 3: stage bits 8-11, packed along bit 0    (adjacent elements -> one code byte)
//    Between phases the row is regrouped through shared memory.  The first regrouping swaps bits
//    0-3 with bits 4-7 among the 16 lanes of a half-warp: 64-bit stores and loads of whole packed
//    registers and a warp-level sync only.  The second crosses warps: scalar stores, 64-bit loads,
//    one named barrier.  The buffer layouts are additive in the index bits (padded, not
//    XOR-swizzled) so that every access is base + immediate and bank-conflict free.
//  * Rotations use the scaled form  lo' = lo + k1*hi, hi' = hi + k2*lo  (two independent FMAs and two constants
//    per pair): every element carries an implicit factor d, the product of the cosines of the rotations it has
//    been through, which the table build folds into k1, k2 and into the general 2x2 of the last stage, so the
//    kernel sees only constants.  The form is singular where a cosine vanishes; when some element's factor leaves
//    [2^-64, 1] the table build raises a flag and the kernel takes the three-shear (lifting) form instead:
//    a += -t*b; b += s*a; a += -t*b  with t = tan(phi/2), s = sin(phi), three FMAs per pair, angles reduced to
//    |phi| <= pi/2 (so |t| <= 1), the sign flips of the reduction tracked per element at table-build time.  Both
//    images have the same layout.
//  * The constants (416 words per thread role, 53248 in all) live in tensor memory, one strip per
//    lane; every group reads the same strips.  They are streamed into registers with tcgen05.ld,
//    one chunk ahead of use.
//  * Rows arrive by TMA (128-byte swizzled tiles, two-deep ring per group, mbarrier completion).
//    The per-row absmax is a warp reduction plus one step across the group's four warps; INT4
//    codes are produced with the magic-number rounding trick, one byte per packed register.
#include <type_traits>

#include "bfq_fast.h"
#include "bfq_generic.cuh"
#include "bfq_n4096.cuh"

namespace bfq {
namespace f4k {

// G row groups per CTA; XB regrouping buffers per group (2: one per regrouping; 1: shared, at the
// price of one more barrier per row)
template <int G, int XB>
struct Smem {
    static constexpr uint32_t kInOff = 0;  // [G][kInSlots][kRowBytes], 1024-byte aligned tiles
    static constexpr uint32_t kExOff = kInOff + G * kInSlots * kRowBytes;  // [G][XB][kExBytes]
    static constexpr uint32_t kBarOff = kExOff + G * XB * kExBytes;       // mbarriers [G][kInSlots]
    static constexpr uint32_t kAmaxOff = kBarOff + 8 * G * kInSlots;      // float [G][2 parities][4 warps]
    static constexpr uint32_t kStatOff = kAmaxOff + 32 * G;               // float [G][2 parities][4 warps][2]: row moments
    static constexpr uint32_t kTmemOff = kStatOff + 64 * G;               // tensor-memory base address
    static constexpr uint32_t kBinsOff = kTmemOff + 16;                   // u64 [16]: the CTA's code counts (statistics)
    static constexpr uint32_t kHistOff = kBinsOff + 128;                  // u32 [G][256]: counts of packed code bytes
    static constexpr uint32_t kUsed = kHistOff + 1024 * G;
    static constexpr uint32_t kBytes = kUsed + 1024;  // slack for the 1024-byte alignment of the TMA tiles
};

// last stage (local bit 3 of phase 3): out_lo = k1*a + k2*b, out_hi = k3*a + k4*b for pairs U0..U0+NU-1
template <int U0, int NU, int CW>
__device__ __forceinline__ void stage_general(u64 (&P)[16], const uint32_t (&T)[CW]) {
    static_assert(8 * NU <= CW, "chunk too small");
#pragma unroll
    for (int i = 0; i < NU; ++i) {
        const int m_lo = U0 + i, m_hi = m_lo | 8;
        const u64 K1 = pack2u(T[8 * i], T[8 * i + 1]), K2 = pack2u(T[8 * i + 2], T[8 * i + 3]);
        const u64 K3 = pack2u(T[8 * i + 4], T[8 * i + 5]), K4 = pack2u(T[8 * i + 6], T[8 * i + 7]);
        const u64 a = P[m_lo], b = P[m_hi];
        P[m_lo] = fma2(K2, b, mul2(K1, a));
        P[m_hi] = fma2(K4, b, mul2(K3, a));
    }
}

struct ExAddr {
    uint32_t w1, r1, w2, r2;  // per-thread byte addresses of the two regroupings (write / read side)
    int bar;                  // named barrier of the group
};

// chunk C of CW words: columns [C*CW, C*CW + CW) of the thread's strip
template <int CW>
struct Chunks {
    static constexpr int kPerStage = 32 / CW;             // chunks per lifting stage
    static constexpr int kLift = 11 * kPerStage;          // chunks of the 11 lifting stages
    static constexpr int kCount = kLift + 64 / CW;        // + the general last stage
    static constexpr int kAfterPhase1 = 4 * kPerStage - 1;  // last chunk of stage 3
    static constexpr int kAfterPhase2 = 8 * kPerStage - 1;  // last chunk of stage 7
};

enum : int { kFormScaled = 0, kFormShear = 1 };  // FORM: how stages 0..10 rotate (the image must match)

template <int FORM, int C, int CW>
__device__ __forceinline__ void run_chunk(u64 (&P)[16], const uint32_t (&T)[CW]) {
    using CH = Chunks<CW>;
    constexpr int NU = CW / 4;
    if constexpr (C < CH::kLift) {
        if constexpr (FORM == kFormScaled) {
            stage_scaled<(C / CH::kPerStage) & 3, (C % CH::kPerStage) * NU, NU, CW>(P, T);
        } else {
            stage_lift<(C / CH::kPerStage) & 3, (C % CH::kPerStage) * NU, NU, CW>(P, T);
        }
    } else {
        stage_general<(C - CH::kLift) * (CW / 8), CW / 8, CW>(P, T);
    }
}

__device__ __forceinline__ void regroup1(u64 (&P)[16], const ExAddr& ex) {
#pragma unroll
    for (int m = 0; m < 16; ++m) sts64(ex.w1 + ex1_wr_local(m), P[m]);
    __syncwarp();
#pragma unroll
    for (int m = 0; m < 16; ++m) P[m] = lds64(ex.r1 + ex1_rd_local(m));
}
template <int XB>
__device__ __forceinline__ void regroup2(u64 (&P)[16], const ExAddr& ex) {
    // with one shared buffer, every warp of the group must be past its reads of the first layout
    if constexpr (XB == 1) bar_sync(ex.bar, kGroupThreads);
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

// Chunk C is in Tcur (load already issued); the load of chunk C+1 is issued right after the wait so
// that exactly one tensor-memory load is in flight while chunk C is being used.  `issue_next` runs
// once per row, after the second regrouping's barrier (all reads of the input slot are done by then).
template <int FORM, int C, int CW, int XB, class F>
__device__ __forceinline__ void run_chunks(u64 (&P)[16], uint32_t (&Tcur)[CW], uint32_t (&Tnext)[CW], uint32_t tbase,
                                           const ExAddr& ex, const Turn& turn, F&& issue_next) {
    using CH = Chunks<CW>;
    if constexpr (C == 0 || C == CH::kAfterPhase1 + 1 || C == CH::kAfterPhase2 + 1) turn.acquire();
    tmem_wait_ld(Tcur);
    if constexpr (C + 1 < CH::kCount) tmem_ld(tbase + CW * (C + 1), Tnext);
    run_chunk<FORM, C, CW>(P, Tcur);
    if constexpr (C == CH::kAfterPhase1) {
        turn.pass();
        regroup1(P, ex);
    }
    if constexpr (C == CH::kAfterPhase2) {
        turn.pass();
        regroup2<XB>(P, ex);
        issue_next();
    }
    if constexpr (C + 1 == CH::kCount) turn.pass();
    if constexpr (C + 1 < CH::kCount) run_chunks<FORM, C + 1, CW, XB>(P, Tnext, Tcur, tbase, ex, turn, issue_next);
}

template <int XB, class F>
__device__ __forceinline__ void run_hadamard(u64 (&P)[16], const ExAddr& ex, F&& issue_next) {
    stage_hadamard<0>(P), stage_hadamard<1>(P), stage_hadamard<2>(P), stage_hadamard<3>(P);
    regroup1(P, ex);
    stage_hadamard<0>(P), stage_hadamard<1>(P), stage_hadamard<2>(P), stage_hadamard<3>(P);
    regroup2<XB>(P, ex);
    issue_next();
    stage_hadamard<0>(P), stage_hadamard<1>(P), stage_hadamard<2>(P), stage_hadamard<3>(P);
}

enum : int { kButterfly = 0, kHadamard = 1 };  // TRANSFORM
enum : int { kOutInt4 = 0, kOutBf16 = 1, kOutInt4Stats = 2, kOutInt2 = 3, kOutInt8 = 4, kOutF32 = 5 };  // OUT

// TRANSFORM: learned butterfly (constants in tensor memory) or the fixed Walsh-Hadamard transform (no constants,
// no tensor memory).  OUT: INT4 codes + fp16 scales, or the rotated rows in bf16 (`yout`, leading dimension ldy), or
// codes + scales + the second and fourth moment of every rotated row (`yout` then points to float [rows][2]) + the
// tensor-wide counts of the 16 code values added to `hist`, or INT2 / INT8 codes + scales.
// STEP: group g passes its token to group (g + STEP) % G, so gcd(STEP, G) groups rotate at a time (0: no tokens).
// ROWS (code outputs only): the rotated rows are written as well, in bf16, to `yout` (weight folding that keeps W Q^T).
// IN_F32: the rows are fp32 (16 KB each): one input slot per group instead of two, re-armed as soon as the group has
// read it (after the second regrouping's barrier), so the load still has most of a row's time to arrive.
template <int G, int CW, int XB, int TRANSFORM, int OUT, int STEP = 2, bool ROWS = false, bool IN_F32 = false>
__global__ void __launch_bounds__(G * kGroupThreads, 1)
k_fwdq4096(const __grid_constant__ CUtensorMap tmap, const float* __restrict__ img, const int* __restrict__ form,
           uint8_t* __restrict__ codes,
           uint16_t* __restrict__ scales, __nv_bfloat16* __restrict__ yout, int64_t ldy, int rows,
           int* __restrict__ status, uint32_t tx_bytes, int wait_limit, unsigned long long* __restrict__ hist) {
    using S = Smem<G, XB>;
    constexpr bool kTmem = TRANSFORM == kButterfly;
    constexpr bool kCount = OUT == kOutInt4Stats;
    constexpr float kPost = TRANSFORM == kHadamard ? 1.0f / 64.0f : 1.0f;  // 1/sqrt(4096), exact
    extern __shared__ uint8_t smem_raw[];
    const uint32_t sbase = (smem_u32(smem_raw) + 1023u) & ~1023u;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int q = warp & 3, g = warp >> 2;
    const int t = q * 32 + lane;  // role within the group: 0..127
    // Constants of this thread's role: the image is stored [column quad][role][4], a warp's load is 512 contiguous
    // bytes, and all of a thread's loads are in flight together, issued before the set-up barrier.  The G warps of a lane quarter share its 26 blocks of 16 columns.  The scaled-form
    // image is fetched on the assumption that the table build selected it; the flag is checked below.
    constexpr int kFillBlocks = (kCols / 16 + G - 1) / G;
    float4 fill[kTmem ? kFillBlocks : 1][4];
    auto fetch_image = [&](const float4* __restrict__ base) {
#pragma unroll
        for (int j = 0; j < kFillBlocks; ++j) {
            const int b = g + j * G;
            if (b < kCols / 16) {
#pragma unroll
                for (int i = 0; i < 4; ++i) fill[j][i] = __ldg(base + (4 * b + i) * 128 + t);
            }
        }
    };
    grid_dep_launch();
    if constexpr (kTmem) {
        if (warp == 0) tmem_alloc512(sbase + S::kTmemOff);
    }
    if (threadIdx.x < G * kInSlots) {
        mbar_init(sbase + S::kBarOff + 8 * threadIdx.x, 1);
        mbar_init_fence();
    }
    if constexpr (kCount) {
        for (uint32_t e = threadIdx.x; e < (128u + 1024u * G) / 4u; e += G * kGroupThreads) sts32(sbase + S::kBinsOff + 4u * e, 0u);
    }
    // everything above overlaps the end of the kernel before this one; global memory is touched from here on
    grid_dep_wait();
    bool shear = false;
    if constexpr (kTmem) {
        fetch_image(reinterpret_cast<const float4*>(img));
        shear = __ldg(form) != 0;
    }
    if constexpr (kTmem) tmem_fence_before();
    __syncthreads();
    if constexpr (kTmem) tmem_fence_after();
    uint32_t tmem_base = 0;
    if constexpr (kTmem) asm volatile("ld.shared.u32 %0, [%1];" : "=r"(tmem_base) : "r"(sbase + S::kTmemOff));
    const uint32_t tlane = tmem_base + (static_cast<uint32_t>(q * 32) << 16);

    // row r belongs to group (r / gridDim.x) % G of CTA r % gridDim.x: a last, partial round of rows spreads over
    // the CTAs instead of filling all groups of the first few
    const int first = g * gridDim.x + blockIdx.x;
    const int stride = gridDim.x * G;
    const int count = first < rows ? (rows - first + stride - 1) / stride : 0;
    // rows of group 0, the largest count of the CTA: every group takes that many turns with a token
    const int turns = static_cast<int>(blockIdx.x) < rows ? (rows - blockIdx.x + stride - 1) / stride : 0;
    const uint32_t in_base = sbase + S::kInOff + g * kInSlots * kRowBytes;
    const uint32_t bar_base = sbase + S::kBarOff + 8 * g * kInSlots;
    static_assert(STEP >= 0 && (STEP == 0 || G % STEP == 0), "the rings must have equal length");
    constexpr int kRings = STEP == 0 ? 1 : STEP;  // gcd(STEP, G)
    Turn turn;
    turn.on = kTmem && STEP > 0;
    turn.wait_id = kTurnBar0 + g;
    turn.pass_id = kTurnBar0 + (g + STEP) % G;
    const bool seeds_ring = (g + STEP) % G < kRings;  // this group's successor starts with the token

    // first rows of this group
    constexpr int kSlotsUsed = IN_F32 ? 1 : kInSlots;                // fp32 rows: one slot of 2 * kRowBytes per group
    constexpr uint32_t kSlotBytes = IN_F32 ? 2 * kRowBytes : kRowBytes;
    static_assert(kInSlots == 2, "an fp32 row takes the group's two bf16 slots");
    if (t == 0) {
        for (int k = 0; k < kSlotsUsed && k < count; ++k) {
            mbar_expect_tx(bar_base + 8 * k, tx_bytes);
            tma_load_3d(in_base + k * kSlotBytes, &tmap, 0, 0, first + k * stride, bar_base + 8 * k);
        }
    }
    // fill tensor memory
    if constexpr (kTmem) {
        if (shear) fetch_image(reinterpret_cast<const float4*>(img) + (kCols / 4) * 128);  // the other image after all
#pragma unroll
        for (int j = 0; j < kFillBlocks; ++j) {
            const int b = g + j * G;
            if (b < kCols / 16) {
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
        tmem_fence_before();
    }
    __syncthreads();
    if constexpr (kTmem) tmem_fence_after();

    ExAddr ex;
    {
        const uint32_t eb1 = sbase + S::kExOff + g * XB * kExBytes;
        const uint32_t eb2 = eb1 + (XB - 1) * kExBytes;
        const uint32_t t4 = (t >> 4) & 1, t5 = (t >> 5) & 1, t6 = (t >> 6) & 1;
        ex.w1 = eb1 + 4u * (2u * (t & 15) + 32u * (t >> 4));
        ex.r1 = eb1 + 4u * (258u * (t & 15) + 32u * (t >> 4));
        ex.w2 = eb2 + 4u * ((t & 15) + 2064u * t4 + 512u * t5 + 1024u * t6);
        ex.r2 = eb2 + 4u * (2u * (t & 15) + 32u * (t >> 4));
        ex.bar = 1 + g;
    }
    // input tile: thread t owns two runs of 32 bytes, at byte 32 (t & 15) + 1024 (t >> 4) + 512 h of the
    // row, i.e. 16-byte chunks 2 (t & 3) + c of 128-byte line ((t >> 2) & 3) + 8 (t >> 4) + 4 h; the TMA
    // swizzle stores chunk j of line l at position j ^ (l & 7)
    // (fp32 rows: runs of 64 bytes at byte 64 (t & 15) + 2048 (t >> 4) + 1024 h: chunks 4 (t & 1) + c of line
    // ((t & 15) >> 1) + 16 (t >> 4) + 8 h)
    const uint32_t in_line = IN_F32 ? ((t & 15) >> 1) * 128u + (t >> 4) * 2048u : ((t >> 2) & 3) * 128u + (t >> 4) * 1024u;
    const uint32_t in_x = IN_F32 ? ((((t & 1) << 2) ^ ((t >> 1) & 7)) << 4) : ((((t & 3) << 1) ^ ((t >> 2) & 3)) << 4);
    const uint32_t amax_base = sbase + S::kAmaxOff + g * 32;
    uint8_t* const out_t = codes + t;
    const uint32_t hist_g = sbase + S::kHistOff + 1024u * g;  // this group's counts of packed code bytes

    // the whole row loop exists once per stage form: the choice is made once per launch, outside the loop
    auto row_loop = [&](auto form_tag) {
    constexpr int FORM = decltype(form_tag)::value;
    u64 P[16];
    uint32_t T0[CW], T1[CW];

    if (seeds_ring) turn.pass();
    for (int k = 0; k < count; ++k) {
        const int row = first + k * stride;
        const int slot = IN_F32 ? 0 : (k & 1);
        if constexpr (kTmem) tmem_ld(tlane, T0);
        mbar_wait_bounded(bar_base + 8 * slot, (IN_F32 ? k : (k >> 1)) & 1, status, wait_limit);
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
            // run (h, c) holds elements 8c..8c+7 of half h; element m of half h is half h of P[m]
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
                mbar_expect_tx(bar_base + 8 * slot, tx_bytes);
                tma_load_3d(in_base + slot * kSlotBytes, &tmap, 0, 0, first + (k + kSlotsUsed) * stride,
                            bar_base + 8 * slot);
            }
        };
        if constexpr (kTmem) {
            run_chunks<FORM, 0, CW, XB>(P, T0, T1, tlane, ex, turn, issue_next);
        } else {
            run_hadamard<XB>(P, ex, issue_next);
        }

        static_assert(!ROWS || OUT == kOutInt4 || OUT == kOutInt2 || OUT == kOutInt8, "rows beside codes only");
        if constexpr (OUT == kOutBf16 || ROWS) {
            // thread t holds elements 2t + 256m, +1: one 32-bit word of the bf16 row per packed register
            uint32_t* out = reinterpret_cast<uint32_t*>(yout + static_cast<int64_t>(row) * ldy) + t;
#pragma unroll
            for (int m = 0; m < 16; ++m) {
                float a, b;
                unpack2(P[m], a, b);
                const __nv_bfloat162 v = __floats2bfloat162_rn(a * kPost, b * kPost);
                out[128 * m] = *reinterpret_cast<const uint32_t*>(&v);
            }
        }
        if constexpr (OUT == kOutF32) {
            // thread t holds elements 2t + 256m, +1: one 64-bit word of the fp32 row per packed register
            u64* out = reinterpret_cast<u64*>(reinterpret_cast<float*>(yout) + static_cast<int64_t>(row) * ldy) + t;
#pragma unroll
            for (int m = 0; m < 16; ++m) {
                float a, b;
                unpack2(P[m], a, b);
                out[128 * m] = pack2(a * kPost, b * kPost);
            }
        }
        if constexpr (OUT == kOutBf16 || OUT == kOutF32) {
            bar_sync(ex.bar, kGroupThreads);  // every warp is past its reads of the second regrouping buffer
            continue;
        }

        // per-row absmax: thread, warp, then the group's four warps
        float m0 = 0.f, m1 = 0.f;
#pragma unroll
        for (int m = 0; m < 16; ++m) {
            float a, b;
            unpack2(P[m], a, b);
            m0 = fmaxf(m0, fabsf(a));
            m1 = fmaxf(m1, fabsf(b));
        }
        // non-negative floats order like their bit patterns: one integer max-reduction over the warp (fmaxf has
        // already dropped NaNs)
        float amax = fmaxf(m0, m1);
        const uint32_t aslot = amax_base + (k & 1) * 16;
        {
            const uint32_t wmax = __reduce_max_sync(0xFFFFFFFFu, __float_as_uint(amax));
            sts32_if(lane == 0, aslot + q * 4, wmax);
        }
        const uint32_t mslot = sbase + S::kStatOff + g * 64 + (k & 1) * 32;
        if constexpr (OUT == kOutInt4Stats) {
            // sum y^2 and sum y^4 of the row: thread (fixed order), warp (xor tree), then the four warps in order
            u64 s2v = pack2(0.f, 0.f), s4v = pack2(0.f, 0.f);
#pragma unroll
            for (int m = 0; m < 16; ++m) {
                const u64 sq = mul2(P[m], P[m]);
                s2v = add2(s2v, sq);
                s4v = fma2(sq, sq, s4v);
            }
            float a2, b2, a4, b4;
            unpack2(s2v, a2, b2), unpack2(s4v, a4, b4);
            float s2 = a2 + b2, s4 = a4 + b4;
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) {
                s2 += __shfl_xor_sync(0xFFFFFFFFu, s2, o);
                s4 += __shfl_xor_sync(0xFFFFFFFFu, s4, o);
            }
            if (lane == 0) sts64(mslot + q * 8, pack2(s2, s4));
        }
        bar_sync(ex.bar, kGroupThreads);
        if constexpr (OUT == kOutInt4Stats) {
            if (t == 0) {
                float s2 = 0.f, s4 = 0.f;
#pragma unroll
                for (int w4 = 0; w4 < 4; ++w4) {
                    float a, b;
                    unpack2(lds64(mslot + w4 * 8), a, b);
                    s2 += a, s4 += b;
                }
                float* rs = reinterpret_cast<float*>(yout) + 2 * static_cast<int64_t>(row);
                rs[0] = s2 * (kPost * kPost), rs[1] = s4 * (kPost * kPost * kPost * kPost);
            }
        }
        {
            const uint4 o = lds128(aslot);
            amax = fmaxf(fmaxf(__uint_as_float(o.x), __uint_as_float(o.y)),
                         fmaxf(__uint_as_float(o.z), __uint_as_float(o.w)));
        }
        constexpr int kQmax = OUT == kOutInt2 ? 1 : (OUT == kOutInt8 ? 127 : 7);
        float inv;
        const uint16_t s16 = row_scale_fast<kQmax>(amax * kPost, &inv);
        inv *= kPost;  // the registers still hold the un-normalised values (kPost is a power of two)
        stg16_if(t == 0, scales + row, s16);

        if constexpr (OUT == kOutInt8) {
            // |v * inv| <= qmax (1 + 2^-10) < qmax + 1/2 for a normal, unsaturated fp16 scale: no clipping; v * inv +
            // 1.5 * 2^23 then has the code (two's complement) in its low mantissa bits
            const bool plain8 = (((s16 >> 10) & 31u) != 0u) && (s16 != 0x7BFFu);
            // thread t holds elements 2t + 256m, +1 = bytes 2t + 256m, +1 of the row
            uint16_t* out16 = reinterpret_cast<uint16_t*>(codes + static_cast<size_t>(row) * kN) + t;
            if (plain8) {
                // u = code + 128 in the low byte of v * inv + (1.5 * 2^23 + 128), whose other low bits are zero:
                // hi * 256 + lo has u_hi, u_lo in its two low bytes; the XOR turns offset binary into two's complement
                const u64 inv2 = pack2(inv, inv), magic2 = pack2(12583040.0f, 12583040.0f);
#pragma unroll
                for (int m = 0; m < 16; ++m) {
                    uint32_t lo, hi;
                    unpack2u(fma2(P[m], inv2, magic2), lo, hi);
                    out16[128 * m] = static_cast<uint16_t>((hi * 256u + lo) ^ 0x8080u);
                }
            } else {
#pragma unroll
                for (int m = 0; m < 16; ++m) {
                    float a, b;
                    unpack2(P[m], a, b);
                    const uint32_t lo = static_cast<uint32_t>(quant1(a, inv, -kQmax - 1, kQmax));
                    const uint32_t hi = static_cast<uint32_t>(quant1(b, inv, -kQmax - 1, kQmax));
                    out16[128 * m] = static_cast<uint16_t>((lo & 0xFFu) | ((hi & 0xFFu) << 8));
                }
            }
            continue;
        }
        if constexpr (OUT == kOutInt2) {
            // elements 2t + 256m, +1 are half of byte t/2 + 64m: the low half for even t, the high half for odd t.
            // The sixteen 4-bit halves (two codes each) travel in the low halves of the bytes of four words, registers
            // 4w .. 4w+3 in word w.
            const bool plain2 = (((s16 >> 10) & 31u) != 0u) && (s16 != 0x7BFFu);
            uint32_t w[4] = {0u, 0u, 0u, 0u};
            if (plain2) {
                // |v * inv| <= 1.0005: v * inv + (1.5 * 2^23 + 2) has u = code + 2 in {1, 2, 3} in its low bits above
                // the constant pattern C = 0x4B400000, so hi * 4 + lo = 5 C + (4 u_hi + u_lo); a Horner chain over four
                // registers gives the nibbles times 256^i plus a constant, one subtraction removes it and one XOR turns
                // every u into the two's complement code
                const u64 inv2 = pack2(inv, inv), magic2 = pack2(12582914.0f, 12582914.0f);
                constexpr uint32_t kBias = static_cast<uint32_t>((5ull * 0x4B400000ull * 0x01010101ull) & 0xFFFFFFFFull);
#pragma unroll
                for (int q4 = 0; q4 < 4; ++q4) {
#pragma unroll
                    for (int i = 3; i >= 0; --i) {
                        uint32_t lo, hi;
                        unpack2u(fma2(P[4 * q4 + i], inv2, magic2), lo, hi);
                        w[q4] = w[q4] * 256u + (hi * 4u + lo);
                    }
                    w[q4] = (w[q4] - kBias) ^ 0x0A0A0A0Au;
                }
            } else {
#pragma unroll
                for (int m = 0; m < 16; ++m) {
                    float a, b;
                    unpack2(P[m], a, b);
                    const uint32_t c = (static_cast<uint32_t>(quant1(a, inv, -2, 1)) & 3u) |
                                       ((static_cast<uint32_t>(quant1(b, inv, -2, 1)) & 3u) << 2);
                    w[m >> 2] |= c << (8 * (m & 3));
                }
            }
            // the even thread writes bytes m = 0..7 (its nibbles + the odd thread's), the odd one 8..15 (the even
            // thread's nibbles + its own): one exchange per word, then the two nibbles of a byte side by side
            const bool odd = t & 1;
            uint8_t* out2 = codes + static_cast<size_t>(row) * (kN / 4) + (t >> 1) + (odd ? 64 * 8 : 0);
#pragma unroll
            for (int h = 0; h < 2; ++h) {
                const uint32_t other = __shfl_xor_sync(0xFFFFFFFFu, odd ? w[h] : w[2 + h], 1);
                const uint32_t bytes = (odd ? other : w[h]) + ((odd ? w[2 + h] : other) << 4);
#pragma unroll
                for (int j = 0; j < 4; ++j) out2[64 * (4 * h + j)] = static_cast<uint8_t>(bytes >> (8 * j));
            }
            continue;
        }

        // codes: thread t holds elements 2t + 256m (+1) = byte t + 128m of the row's packed codes
        const uint32_t e16 = (s16 >> 10) & 31u;
        const bool plain = (e16 != 0u) && (s16 != 0x7BFFu);  // normal fp16 scale: |v*inv| <= 7.004, no clipping
        uint8_t* out = out_t + static_cast<size_t>(row) * (kN / 2);
        if (plain) {
            // q + 8 lands in the low nibble of the fp32 bit pattern of v*inv + (1.5*2^23 + 8), whose other
            // low bits are zero: hi*16 + lo has (q_hi + 8) << 4 | (q_lo + 8) in its low byte
            const u64 inv2 = pack2(inv, inv);
            const u64 magic2 = pack2(12582920.0f, 12582920.0f);
#pragma unroll
            for (int m = 0; m < 16; ++m) {
                uint32_t lo, hi;
                unpack2u(fma2(P[m], inv2, magic2), lo, hi);
                const uint32_t ob = hi * 16u + lo;  // 17 * 0x4B400000 + the offset-binary byte
                out[128 * m] = static_cast<uint8_t>(ob ^ 0x88u);  // offset binary -> two's complement
                // counted by its offset-binary value; the constant is taken off the base address instead of the index
                if constexpr (kCount) red_shared_inc(hist_g - 4u * (17u * 0x4B400000u) + 4u * ob);
            }
        } else {
#pragma unroll
            for (int m = 0; m < 16; ++m) {
                float a, b;
                unpack2(P[m], a, b);
                const int qa = static_cast<int>(fminf(fmaxf(rintf(a * inv), -8.f), 7.f));
                const int qb = static_cast<int>(fminf(fmaxf(rintf(b * inv), -8.f), 7.f));
                const uint32_t byte = static_cast<uint32_t>((qa & 0xF) | ((qb & 0xF) << 4));
                out[128 * m] = static_cast<uint8_t>(byte);
                if constexpr (kCount) red_shared_inc(hist_g + 4u * (byte ^ 0x88u));
            }
        }
    }
    // a group with fewer rows than group 0 keeps the tokens moving
    for (int k = count; k < turns; ++k) {
#pragma unroll
        for (int ph = 0; ph < 3; ++ph) turn.acquire(), turn.pass();
    }
    if (g < kRings) turn.acquire();  // each ring's first group takes its token back: no arrival stays pending
    };
    if (!shear) {
        row_loop(std::integral_constant<int, kFormScaled>());
    } else if constexpr (kTmem) {
        row_loop(std::integral_constant<int, kFormShear>());
    }

    if constexpr (kCount) {
        // counts of the G groups per offset-binary byte (two nibbles code + 8) -> the CTA's 16 code counts -> the caller's
        // histogram, indexed by code + 8.  Integer additions: the result does not depend on their order.
        __syncthreads();
        if (threadIdx.x < 256) {
            uint32_t n = 0;
#pragma unroll
            for (int gg = 0; gg < G; ++gg) n += lds32(sbase + S::kHistOff + 1024u * gg + 4u * threadIdx.x);
            if (n != 0u) {
                red_shared_add64(sbase + S::kBinsOff + 8u * (threadIdx.x & 15u), n);
                red_shared_add64(sbase + S::kBinsOff + 8u * (threadIdx.x >> 4), n);
            }
        }
        __syncthreads();
        if (threadIdx.x < 16) {
            const unsigned long long c = lds64(sbase + S::kBinsOff + 8u * threadIdx.x);
            if (c != 0ull) atomicAdd(hist + threadIdx.x, c);
        }
    }
    if constexpr (kTmem) {
        tmem_fence_before();
        __syncthreads();
        if (warp == 0) tmem_dealloc512(tmem_base);
    }
}

// ---- table preparation -----------------------------------------------------------------------------------
// Step 1 (one thread per angle): the generic (cos, sin) table entry, cos and sin in double for step 2, the
// reduced-angle lifting constants and whether the reduction negates the pair.  The pair is negated iff
// cos(theta) < 0, and phi = theta -+ pi in that case; tan(phi/2) and sin(phi) are odd in phi, so the constants for
// the mirrored rotation G(-theta) are the negatives of the stored ones.
__global__ void __launch_bounds__(256) k_prep_angles4096(const float* __restrict__ theta, float2* __restrict__ tw,
                                                          float4* __restrict__ prep, uint8_t* __restrict__ flip,
                                                          double2* __restrict__ cs, int* __restrict__ form) {
    const int k = blockIdx.x * blockDim.x + threadIdx.x;
    grid_dep_launch();
    grid_dep_wait();
    if (k == 0) *form = kFormScaled;  // step 2 raises it when the scaled form is out of range
    if (k >= 12 * (kN / 2)) return;
    const double th = static_cast<double>(theta[k]);
    double sn, c;
    sincos(th, &sn, &c);
    tw[k] = make_float2(static_cast<float>(c), static_cast<float>(sn));
    cs[k] = make_double2(c, sn);
    // phi = theta -+ pi when cos(theta) < 0 (|phi| <= pi/2 then): sin(phi) = -sin(theta), cos(phi) = -cos(theta), and
    // tan(phi/2) = sin(phi) / (1 + cos(phi)) with a denominator >= 1: no second reduction, no tan
    const bool f = c < 0.0;
    const double sp = f ? -sn : sn, cp = f ? -c : c;
    flip[k] = f ? 1 : 0;
    prep[k] = make_float4(static_cast<float>(-sp / (1.0 + cp)), static_cast<float>(sp), static_cast<float>(c),
                          static_cast<float>(sn));
}

// factor carried by element i when it enters stage s: the product of the cosines of the pairs it belonged to in
// stages 0..s-1 (its sign is the tracked sign of the three-shear form)
__device__ __forceinline__ double factor_before(const double2* __restrict__ cs, int i, int s) {
    double c[11];
#pragma unroll
    for (int sp = 0; sp < 11; ++sp) {  // all loads issued together
        const int j = ((i >> (sp + 1)) << sp) | (i & ((1 << sp) - 1));
        c[sp] = sp < s ? cs[sp * (kN / 2) + j].x : 1.0;
    }
    double d = 1.0;
#pragma unroll
    for (int sp = 0; sp < 11; ++sp) d *= c[sp];
    return d;
}

// Step 2 (one thread per angle): place the constants of pair (s, j) in both tensor-memory images
// img[form][role][column], with the role / register / half of the pair's low element in its phase, and raise *form
// when an element's factor leaves the range the scaled form is used in.
__global__ void __launch_bounds__(256) k_build_image4096(const float4* __restrict__ prep, const double2* __restrict__ cs,
                                                          float* __restrict__ img, int* __restrict__ form) {
    const int k = blockIdx.x * blockDim.x + threadIdx.x;
    grid_dep_launch();
    grid_dep_wait();
    if (k >= 12 * (kN / 2)) return;
    const int s = k / (kN / 2), j = k % (kN / 2);
    const int lo = ((j >> s) << (s + 1)) | (j & ((1 << s) - 1));
    const int hi = lo + (1 << s);
    const double da = factor_before(cs, lo, s), db = factor_before(cs, hi, s);
    const int sa = da < 0.0 ? -1 : 1, sb = db < 0.0 ? -1 : 1;
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
    const double2 own = cs[k];
    // image layout [column quad][role][4]: column col of role r is word ((col >> 2) * 128 + r) * 4 + (col & 3)
    float* scaled = img + kFormScaled * (128 * kCols) + 4 * r;
    float* shear = img + kFormShear * (128 * kCols) + 4 * r;
    auto at = [](int col) { return (col >> 2) * 512 + (col & 3); };
    if (s < 11) {
        const float sg = (sa == sb) ? 1.f : -1.f;
        shear[at(32 * s + 4 * u + h)] = sg * p.x;
        shear[at(32 * s + 4 * u + h + 2)] = sg * p.y;
        // k1 = -tan(theta) db/da, k2 = tan(theta) da/db, with one division
        const double w = own.y / (own.x * da * db);
        scaled[at(32 * s + 4 * u + h)] = static_cast<float>(-w * db * db);
        scaled[at(32 * s + 4 * u + h + 2)] = static_cast<float>(w * da * da);
        const double lim = 5.421010862427522e-20;  // 2^-64
        if (!(fabs(own.x * da) >= lim && fabs(own.x * db) >= lim)) *form = kFormShear;
    } else {
        const int col = 352 + 8 * u + h;
        shear[at(col + 0)] = p.z * sa;
        shear[at(col + 2)] = -p.w * sb;
        shear[at(col + 4)] = p.w * sa;
        shear[at(col + 6)] = p.z * sb;
        scaled[at(col + 0)] = static_cast<float>(own.x * da);
        scaled[at(col + 2)] = static_cast<float>(-own.y * db);
        scaled[at(col + 4)] = static_cast<float>(own.y * da);
        scaled[at(col + 6)] = static_cast<float>(own.x * db);
    }
}

}  // namespace f4k

// ---- host side ---------------------------------------------------------------------------------------------
// two images: scaled form, three-shear form
size_t fwdq4096_image_bytes() { return size_t(2) * 128 * f4k::kCols * sizeof(float); }
// per angle: float4 (three-shear constants, cos, sin), double2 (cos, sin), one negation flag
size_t fwdq4096_prep_bytes() { return size_t(12) * (f4k::kN / 2) * (sizeof(float4) + sizeof(double2) + 1); }

// Builds the generic (cos, sin) table and the tensor-memory image from the angles (two launches).
cudaError_t fwdq4096_set_angles(const bfq_plan* plan, const float* theta, cudaStream_t st) {
    const int count = 12 * (f4k::kN / 2);
    float4* prep = reinterpret_cast<float4*>(plan->prep4096);
    double2* cs = reinterpret_cast<double2*>(prep + count);
    uint8_t* flip = reinterpret_cast<uint8_t*>(cs + count);
    cudaError_t e = launch_overlapped(f4k::k_prep_angles4096, dim3((count + 255) / 256), dim3(256), 0, st, theta, plan->tw,
                                      prep, flip, cs, plan->form_flag);
    if (e != cudaSuccess) return e;
    return launch_overlapped(f4k::k_build_image4096, dim3((count + 255) / 256), dim3(256), 0, st, prep, cs, plan->img4096,
                             plan->form_flag);
}

bool fwdq4096_available(const bfq_plan* plan) {
    return plan->n == f4k::kN && plan->cc_major == 10 && plan->img4096 != nullptr && encode_tiled() != nullptr;
}

template <int G, int CW, int XB, int TRANSFORM, int OUT, bool ROWS = false, bool IN_F32 = false>
static cudaError_t launch_variant(const bfq_plan* plan, const CUtensorMap& tmap, int64_t rows, uint8_t* codes,
                                  uint16_t* scales, void* y, int64_t ldy, cudaStream_t st,
                                  unsigned long long* hist = nullptr) {
    using S = f4k::Smem<G, XB>;
    static bool attr_set[kMaxDevices] = {false};
    auto kern = f4k::k_fwdq4096<G, CW, XB, TRANSFORM, OUT, 2, ROWS, IN_F32>;
    if (!attr_set[plan->device]) {
        cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, int(S::kBytes));
        if (e != cudaSuccess) return e;
        attr_set[plan->device] = true;
    }
    const int64_t want = (rows + G - 1) / G;
    const int grid = int(want < plan->sm_count ? want : plan->sm_count);
    // bytes a row's load is expected to deliver and the bound on polls of its barrier; the test hook announces more
    // bytes than arrive, so that every wait runs out (quickly) and reports through the status word
    const uint32_t tx_bytes = (IN_F32 ? 2 : 1) * f4k::kRowBytes + (plan->test_stuck_wait ? 16u : 0u);
    const int wait_limit = plan->test_stuck_wait ? 4096 : (1 << 22);
    return launch_overlapped(kern, dim3(grid), dim3(G * f4k::kGroupThreads), S::kBytes, st, tmap, plan->img4096,
                             plan->form_flag, codes, scales, static_cast<__nv_bfloat16*>(y), ldy, int(rows),
                             plan->status_word, tx_bytes, wait_limit, hist);
}

// Four row groups per CTA, 32-word constant chunks, one buffer per regrouping (measured fastest among the
// configurations that compile without spills; more groups did not help).
// hadamard: the fixed Walsh-Hadamard transform instead of the plan's butterfly.  y != nullptr: write the rotated
// rows in bf16 instead of INT4 codes + scales.
cudaError_t fwdq4096_launch(const bfq_plan* plan, const void* x, int64_t rows, int64_t ldx, bool hadamard,
                            uint8_t* codes, uint16_t* scales, void* y, int64_t ldy, cudaStream_t st) {
    CUtensorMap tmap;
    if (!encode_row_map(&tmap, x, rows, ldx)) return cudaErrorInvalidValue;
    using namespace f4k;
    if (!hadamard) {
        return y == nullptr ? launch_variant<4, 32, 2, kButterfly, kOutInt4>(plan, tmap, rows, codes, scales, y, ldy, st)
                            : launch_variant<4, 32, 2, kButterfly, kOutBf16>(plan, tmap, rows, codes, scales, y, ldy, st);
    }
    return y == nullptr ? launch_variant<4, 32, 2, kHadamard, kOutInt4>(plan, tmap, rows, codes, scales, y, ldy, st)
                        : launch_variant<4, 32, 2, kHadamard, kOutBf16>(plan, tmap, rows, codes, scales, y, ldy, st);
}

// INT2 / INT8 codes: same kernel, other packing in the epilogue
cudaError_t fwdq4096_launch_bits(const bfq_plan* plan, const void* x, int64_t rows, int64_t ldx, bool hadamard, int bits,
                                 uint8_t* codes, uint16_t* scales, cudaStream_t st) {
    CUtensorMap tmap;
    if (!encode_row_map(&tmap, x, rows, ldx)) return cudaErrorInvalidValue;
    using namespace f4k;
    if (hadamard) {
        return bits == 2 ? launch_variant<4, 32, 2, kHadamard, kOutInt2>(plan, tmap, rows, codes, scales, nullptr, 0, st)
                         : launch_variant<4, 32, 2, kHadamard, kOutInt8>(plan, tmap, rows, codes, scales, nullptr, 0, st);
    }
    return bits == 2 ? launch_variant<4, 32, 2, kButterfly, kOutInt2>(plan, tmap, rows, codes, scales, nullptr, 0, st)
                     : launch_variant<4, 32, 2, kButterfly, kOutInt8>(plan, tmap, rows, codes, scales, nullptr, 0, st);
}

// weight folding that keeps the rotated rows: codes + scales and W Q^T in bf16 (leading dimension ldy) from one pass
cudaError_t fwdq4096_launch_codes_rows(const bfq_plan* plan, const void* x, int64_t rows, int64_t ldx, int bits,
                                       uint8_t* codes, uint16_t* scales, void* y, int64_t ldy, cudaStream_t st) {
    CUtensorMap tmap;
    if (!encode_row_map(&tmap, x, rows, ldx)) return cudaErrorInvalidValue;
    using namespace f4k;
    if (bits == 4) return launch_variant<4, 32, 2, kButterfly, kOutInt4, true>(plan, tmap, rows, codes, scales, y, ldy, st);
    if (bits == 2) return launch_variant<4, 32, 2, kButterfly, kOutInt2, true>(plan, tmap, rows, codes, scales, y, ldy, st);
    return launch_variant<4, 32, 2, kButterfly, kOutInt8, true>(plan, tmap, rows, codes, scales, y, ldy, st);
}

// fp32 rows in: codes + scales (bits = 2, 4, 8), or the rotated rows in fp32 (bits = 0, y with leading dimension ldy)
cudaError_t fwdq4096_launch_f32(const bfq_plan* plan, const void* x, int64_t rows, int64_t ldx, int bits, uint8_t* codes,
                                uint16_t* scales, void* y, int64_t ldy, cudaStream_t st) {
    CUtensorMap tmap;
    if (!encode_row_map_f32(&tmap, x, rows, ldx)) return cudaErrorInvalidValue;
    using namespace f4k;
    if (bits == 0) return launch_variant<4, 32, 2, kButterfly, kOutF32, false, true>(plan, tmap, rows, codes, scales, y, ldy, st);
    if (bits == 4) return launch_variant<4, 32, 2, kButterfly, kOutInt4, false, true>(plan, tmap, rows, codes, scales, nullptr, 0, st);
    if (bits == 2) return launch_variant<4, 32, 2, kButterfly, kOutInt2, false, true>(plan, tmap, rows, codes, scales, nullptr, 0, st);
    return launch_variant<4, 32, 2, kButterfly, kOutInt8, false, true>(plan, tmap, rows, codes, scales, nullptr, 0, st);
}

// bfq_forward_quant_stats on the tuned path: codes + scales + row moments + code counts from one launch of k_fwdq4096
// (hist must have been zeroed on the same stream).
cudaError_t fwdq4096_launch_stats(const bfq_plan* plan, const void* x, int64_t rows, int64_t ldx, uint8_t* codes,
                                  uint16_t* scales, unsigned long long* hist, float* rowstats, cudaStream_t st) {
    CUtensorMap tmap;
    if (!encode_row_map(&tmap, x, rows, ldx)) return cudaErrorInvalidValue;
    using namespace f4k;
    return launch_variant<4, 32, 2, kButterfly, kOutInt4Stats>(plan, tmap, rows, codes, scales, rowstats, 0, st, hist);
}

}  // namespace bfq
