// Generic register/shared-memory butterfly kernels: every supported n (16..8192), fp32 or
// bf16 rows, all four operations.  These are the reference-quality CUDA path; the tuned
// kernels for the headline shapes live in their own files and must agree with these.
//
// Mapping.  A row of n = 2^LOG_N elements is owned by TPR = n/16 threads, 16 elements each.
// The L stages are grouped into phases of (up to) four consecutive stages whose pair strides
// fall inside the 16 elements a thread holds, so a phase runs entirely in registers.  Between
// phases the row is regrouped through shared memory (one write + one read of the row, XOR
// swizzled so that both sides hit 32 distinct banks).  Twiddles (cos, sin) come from the plan's
// fp32 table through the read-only cache and are reused for the R rows a thread holds.
#pragma once

#include <cuda_bf16.h>
#include <cuda_fp16.h>
#include <cuda_runtime.h>
#include <stdint.h>

namespace bfq {

enum : int { kF32 = 0, kBF16 = 1 };
enum : int { kModeForward = 0, kModeForwardQuant = 1, kModeInverse = 2, kModeHadamard = 3, kModeHadamardQuant = 4 };

struct GenericParams {
    const float2* tw;  // [L][n/2] (cos, sin)
    const void* x;     // input rows
    int xt;
    int64_t ldx;
    void* y;           // output rows (forward / inverse / fold's optional rotated rows), may be null
    int yt;
    int64_t ldy;
    uint8_t* codes;    // forward_quant
    uint16_t* scales;
    int bits;
    int64_t rows;
    // optional statistics of the rotated rows (quantizing modes only; both null or both set)
    unsigned long long* hist;  // [2^bits] counts of every code value over all rows, index = code + 2^(bits-1)
    float* rowstats;           // [rows][2]: sum of y^2 and sum of y^4 of each rotated row
};

struct BackwardParams {
    const float2* tw;
    const void* x;
    int xt;
    const void* g;
    int gt;
    int64_t ld;
    void* dx;  // may be null
    int dxt;
    float* partial;  // [gridDim.x * GROUPS][L][n/2]
    int64_t rows;
};

template <int LOG_N>
struct Geo {
    static constexpr int kN = 1 << LOG_N;
    static constexpr int kHalf = kN / 2;
    static constexpr int kTPR = kN / 16;                      // threads per row
    static constexpr int kThreads = kTPR > 256 ? kTPR : 256;  // CTA size
    static constexpr int kGroups = kThreads / kTPR;           // rows processed side by side
    static constexpr int kPhases = (LOG_N + 3) / 4;
    static constexpr int kWarpsPerRow = kTPR >= 32 ? kTPR / 32 : 1;
};

// Which 4 index bits are thread-local in phase P: the phase's stage bits [4P, 4P+ns) and, when
// fewer than four stages remain, the lowest (4-ns) index bits as filler.
template <int LOG_N, int P>
struct Phase {
    static constexpr int kB0 = 4 * P;
    static constexpr int kNs = (LOG_N - kB0 >= 4) ? 4 : (LOG_N - kB0);
    static constexpr int kF = 4 - kNs;
    static constexpr int kMid = kB0 - kF;  // bits of t that sit below the stage bits
    static_assert(kNs >= 1, "phase without stages");
    static_assert(P == 0 || kF <= kB0, "filler bits must lie below the stage bits");
    // element index held in local slot e (0..15) by thread t (0..TPR-1) of the row
    __device__ __forceinline__ static int idx(int t, int e) {
        const int e_lo = e & ((1 << kF) - 1);
        const int e_hi = e >> kF;
        const int t_lo = t & ((1 << kMid) - 1);
        const int t_hi = t >> kMid;
        return e_lo | (t_lo << kF) | (e_hi << kB0) | (t_hi << (kB0 + kNs));
    }
};

__device__ __forceinline__ int swz(int i) { return i ^ ((i >> 4) & 31); }

template <int LOG_N, int P, int R, bool INV>
__device__ __forceinline__ void phase_rotate(float (&v)[R][16], const float2* __restrict__ tw, int t) {
    using PH = Phase<LOG_N, P>;
#pragma unroll
    for (int kk = 0; kk < PH::kNs; ++kk) {
        const int k = INV ? (PH::kNs - 1 - kk) : kk;
        const int b = PH::kB0 + k;  // stage = index bit of the pair stride
        const int lb = PH::kF + k;  // same bit inside the local slot number
#pragma unroll
        for (int q = 0; q < 8; ++q) {
            const int e_lo = ((q >> lb) << (lb + 1)) | (q & ((1 << lb) - 1));
            const int e_hi = e_lo | (1 << lb);
            const int i = PH::idx(t, e_lo);
            const int j = ((i >> (b + 1)) << b) | (i & ((1 << b) - 1));
            const float2 cs = __ldg(&tw[b * Geo<LOG_N>::kHalf + j]);
#pragma unroll
            for (int r = 0; r < R; ++r) {
                const float a = v[r][e_lo], bb = v[r][e_hi];
                if (!INV) {
                    v[r][e_lo] = cs.x * a - cs.y * bb;
                    v[r][e_hi] = cs.y * a + cs.x * bb;
                } else {
                    v[r][e_lo] = cs.x * a + cs.y * bb;
                    v[r][e_hi] = cs.x * bb - cs.y * a;
                }
            }
        }
    }
}

// regroup the R rows held by this row's threads from phase PF's ownership to phase PT's
template <int LOG_N, int PF, int PT, int R>
__device__ __forceinline__ void exchange(float (&v)[R][16], float* rowbuf, int t) {
    constexpr int N = Geo<LOG_N>::kN;
#pragma unroll
    for (int r = 0; r < R; ++r)
#pragma unroll
        for (int e = 0; e < 16; ++e) rowbuf[r * N + swz(Phase<LOG_N, PF>::idx(t, e))] = v[r][e];
    __syncthreads();
#pragma unroll
    for (int r = 0; r < R; ++r)
#pragma unroll
        for (int e = 0; e < 16; ++e) v[r][e] = rowbuf[r * N + swz(Phase<LOG_N, PT>::idx(t, e))];
    __syncthreads();
}

// all stages forward, starting in phase-P ownership, ending in the last phase's ownership
template <int LOG_N, int P, int R>
__device__ __forceinline__ void forward_from(float (&v)[R][16], const float2* tw, float* rowbuf, int t) {
    phase_rotate<LOG_N, P, R, false>(v, tw, t);
    if constexpr (P + 1 < Geo<LOG_N>::kPhases) {
        exchange<LOG_N, P, P + 1, R>(v, rowbuf, t);
        forward_from<LOG_N, P + 1, R>(v, tw, rowbuf, t);
    }
}

// Walsh-Hadamard version of a phase: (a, b) -> (a + b, a - b) on every pair of the phase's stages, no table;
// the 1/sqrt(n) normalisation is applied once at the end by the caller
template <int LOG_N, int P, int R>
__device__ __forceinline__ void phase_hadamard(float (&v)[R][16]) {
    using PH = Phase<LOG_N, P>;
#pragma unroll
    for (int k = 0; k < PH::kNs; ++k) {
        const int lb = PH::kF + k;
#pragma unroll
        for (int q = 0; q < 8; ++q) {
            const int e_lo = ((q >> lb) << (lb + 1)) | (q & ((1 << lb) - 1));
            const int e_hi = e_lo | (1 << lb);
#pragma unroll
            for (int r = 0; r < R; ++r) {
                const float a = v[r][e_lo], bb = v[r][e_hi];
                v[r][e_lo] = a + bb;
                v[r][e_hi] = a - bb;
            }
        }
    }
}
template <int LOG_N, int P, int R>
__device__ __forceinline__ void hadamard_from(float (&v)[R][16], float* rowbuf, int t) {
    phase_hadamard<LOG_N, P, R>(v);
    if constexpr (P + 1 < Geo<LOG_N>::kPhases) {
        exchange<LOG_N, P, P + 1, R>(v, rowbuf, t);
        hadamard_from<LOG_N, P + 1, R>(v, rowbuf, t);
    }
}

// all stages transposed, starting in phase-P ownership (P = last phase), ending in phase 0's
template <int LOG_N, int P, int R>
__device__ __forceinline__ void inverse_from(float (&v)[R][16], const float2* tw, float* rowbuf, int t) {
    phase_rotate<LOG_N, P, R, true>(v, tw, t);
    if constexpr (P > 0) {
        exchange<LOG_N, P, P - 1, R>(v, rowbuf, t);
        inverse_from<LOG_N, P - 1, R>(v, tw, rowbuf, t);
    }
}

// ---- row I/O in phase-0 ownership: thread t holds elements [16 t, 16 t + 16) -------------------
__device__ __forceinline__ void load16(const void* base, int dt, int64_t off, bool valid, float (&v)[16]) {
    if (!valid) {
#pragma unroll
        for (int e = 0; e < 16; ++e) v[e] = 0.f;
        return;
    }
    if (dt == kF32) {
        const float4* p = reinterpret_cast<const float4*>(static_cast<const float*>(base) + off);
#pragma unroll
        for (int c = 0; c < 4; ++c) {
            const float4 f = __ldg(p + c);
            v[4 * c + 0] = f.x, v[4 * c + 1] = f.y, v[4 * c + 2] = f.z, v[4 * c + 3] = f.w;
        }
    } else {
        const uint4* p = reinterpret_cast<const uint4*>(static_cast<const __nv_bfloat16*>(base) + off);
#pragma unroll
        for (int c = 0; c < 2; ++c) {
            const uint4 u = __ldg(p + c);
            const uint32_t w[4] = {u.x, u.y, u.z, u.w};
#pragma unroll
            for (int k = 0; k < 4; ++k) {
                v[8 * c + 2 * k + 0] = __uint_as_float(w[k] << 16);
                v[8 * c + 2 * k + 1] = __uint_as_float(w[k] & 0xFFFF0000u);
            }
        }
    }
}

__device__ __forceinline__ uint32_t pack_bf16x2(float lo, float hi) {
    const uint32_t a = __bfloat16_as_ushort(__float2bfloat16_rn(lo));
    const uint32_t b = __bfloat16_as_ushort(__float2bfloat16_rn(hi));
    return a | (b << 16);
}

__device__ __forceinline__ void store16(void* base, int dt, int64_t off, const float (&v)[16]) {
    if (dt == kF32) {
        float4* p = reinterpret_cast<float4*>(static_cast<float*>(base) + off);
#pragma unroll
        for (int c = 0; c < 4; ++c) p[c] = make_float4(v[4 * c], v[4 * c + 1], v[4 * c + 2], v[4 * c + 3]);
    } else {
        uint4* p = reinterpret_cast<uint4*>(static_cast<__nv_bfloat16*>(base) + off);
#pragma unroll
        for (int c = 0; c < 2; ++c) {
            uint4 u;
            u.x = pack_bf16x2(v[8 * c + 0], v[8 * c + 1]);
            u.y = pack_bf16x2(v[8 * c + 2], v[8 * c + 3]);
            u.z = pack_bf16x2(v[8 * c + 4], v[8 * c + 5]);
            u.w = pack_bf16x2(v[8 * c + 6], v[8 * c + 7]);
            p[c] = u;
        }
    }
}

// fp16 scale of a row from its absmax: s = amax / qmax in fp32, rounded to fp16 (nearest even),
// saturating at 65504.  Returns the fp16 bits; *inv = 1/s (0 for a zero scale).
__device__ __forceinline__ uint16_t row_scale(float amax, int qmax, float* inv) {
    const float sf = __fdiv_rn(amax, static_cast<float>(qmax));
    uint16_t bits;
    if (sf >= 65520.f) {
        bits = 0x7BFFu;
    } else {
        bits = __half_as_ushort(__float2half_rn(sf));
    }
    const float s = __half2float(__ushort_as_half(bits));
    *inv = s > 0.f ? __frcp_rn(s) : 0.f;
    return bits;
}

__device__ __forceinline__ int quant1(float y, float inv, int qmin, int qmax) {
    float q = rintf(y * inv);
    q = fminf(fmaxf(q, static_cast<float>(qmin)), static_cast<float>(qmax));
    return static_cast<int>(q);
}

// 16 consecutive elements -> packed two's-complement codes, stored with one vector store
__device__ __forceinline__ void store_codes16(uint8_t* dst, int bits, const float (&v)[16], float inv) {
    const int qmax = (1 << (bits - 1)) - 1, qmin = -(1 << (bits - 1));
    if (bits == 4) {
        uint32_t w[2] = {0u, 0u};
#pragma unroll
        for (int e = 0; e < 16; ++e)
            w[e >> 3] |= (static_cast<uint32_t>(quant1(v[e], inv, qmin, qmax)) & 0xFu) << (4 * (e & 7));
        *reinterpret_cast<uint2*>(dst) = make_uint2(w[0], w[1]);
    } else if (bits == 2) {
        uint32_t w = 0u;
#pragma unroll
        for (int e = 0; e < 16; ++e) w |= (static_cast<uint32_t>(quant1(v[e], inv, qmin, qmax)) & 0x3u) << (2 * e);
        *reinterpret_cast<uint32_t*>(dst) = w;
    } else {
        uint32_t w[4] = {0u, 0u, 0u, 0u};
#pragma unroll
        for (int e = 0; e < 16; ++e)
            w[e >> 2] |= (static_cast<uint32_t>(quant1(v[e], inv, qmin, qmax)) & 0xFFu) << (8 * (e & 3));
        *reinterpret_cast<uint4*>(dst) = make_uint4(w[0], w[1], w[2], w[3]);
    }
}

// max over the TPR threads of a row; red: per-CTA scratch [R][warps in CTA]
template <int LOG_N>
__device__ __forceinline__ float row_max(float m, float* red, int r, int group, int t) {
    using G = Geo<LOG_N>;
    if constexpr (G::kTPR < 32) {
#pragma unroll
        for (int o = G::kTPR / 2; o > 0; o >>= 1) m = fmaxf(m, __shfl_xor_sync(0xFFFFFFFFu, m, o));
        return m;
    } else {
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) m = fmaxf(m, __shfl_xor_sync(0xFFFFFFFFu, m, o));
        constexpr int W = G::kWarpsPerRow;
        float* slot = red + (r * G::kGroups + group) * W;
        if ((t & 31) == 0) slot[t >> 5] = m;
        __syncthreads();
        float mm = slot[0];
#pragma unroll
        for (int w = 1; w < W; ++w) mm = fmaxf(mm, slot[w]);
        return mm;
    }
}

// sum over the TPR threads of a row in a fixed order (shuffle tree, then warps in index order); red as in row_max
template <int LOG_N>
__device__ __forceinline__ float row_sum(float v, float* red, int r, int group, int t) {
    using G = Geo<LOG_N>;
    if constexpr (G::kTPR < 32) {
#pragma unroll
        for (int o = G::kTPR / 2; o > 0; o >>= 1) v += __shfl_xor_sync(0xFFFFFFFFu, v, o);
        return v;
    } else {
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xFFFFFFFFu, v, o);
        constexpr int W = G::kWarpsPerRow;
        float* slot = red + (r * G::kGroups + group) * W;
        __syncthreads();  // the slot's previous use (a maximum or another sum) has been read by everyone
        if ((t & 31) == 0) slot[t >> 5] = v;
        __syncthreads();
        float acc = slot[0];
#pragma unroll
        for (int w = 1; w < W; ++w) acc += slot[w];
        return acc;
    }
}

template <int LOG_N, int R, int MODE>
__global__ void __launch_bounds__(Geo<LOG_N>::kThreads) k_generic(const GenericParams p) {
    using G = Geo<LOG_N>;
    extern __shared__ __align__(16) float smem[];
    float* red = smem + G::kGroups * R * G::kN;  // [R][kGroups][warps per row]
    unsigned int* shist = reinterpret_cast<unsigned int*>(red + R * G::kGroups * G::kWarpsPerRow);  // [256], stats only
    const bool stats = (MODE == kModeForwardQuant || MODE == kModeHadamardQuant) && p.hist != nullptr;
    if (stats) {
        for (int i = threadIdx.x; i < 256; i += blockDim.x) shist[i] = 0u;
        __syncthreads();
    }
    const int group = threadIdx.x / G::kTPR;
    const int t = threadIdx.x % G::kTPR;
    float* rowbuf = smem + group * R * G::kN;
    constexpr int kRowsPerTile = G::kGroups * R;
    const int64_t tiles = (p.rows + kRowsPerTile - 1) / kRowsPerTile;

    for (int64_t tile = blockIdx.x; tile < tiles; tile += gridDim.x) {
        const int64_t row0 = tile * kRowsPerTile + group * R;
        float v[R][16];
#pragma unroll
        for (int r = 0; r < R; ++r) load16(p.x, p.xt, (row0 + r) * p.ldx + t * 16, row0 + r < p.rows, v[r]);

        if constexpr (MODE == kModeInverse) {
            if constexpr (G::kPhases > 1) exchange<LOG_N, 0, G::kPhases - 1, R>(v, rowbuf, t);
            inverse_from<LOG_N, G::kPhases - 1, R>(v, p.tw, rowbuf, t);
        } else if constexpr (MODE == kModeHadamard || MODE == kModeHadamardQuant) {
            hadamard_from<LOG_N, 0, R>(v, rowbuf, t);
            if constexpr (G::kPhases > 1) exchange<LOG_N, G::kPhases - 1, 0, R>(v, rowbuf, t);
            // 1/sqrt(n): a power of two for even log2 n
            const float scale = (LOG_N & 1) ? 0.70710678118654752f / static_cast<float>(1 << (LOG_N / 2))
                                            : 1.0f / static_cast<float>(1 << (LOG_N / 2));
#pragma unroll
            for (int r = 0; r < R; ++r)
#pragma unroll
                for (int e = 0; e < 16; ++e) v[r][e] *= scale;
        } else {
            forward_from<LOG_N, 0, R>(v, p.tw, rowbuf, t);
            if constexpr (G::kPhases > 1) exchange<LOG_N, G::kPhases - 1, 0, R>(v, rowbuf, t);
        }

        if (p.y != nullptr) {
#pragma unroll
            for (int r = 0; r < R; ++r)
                if (row0 + r < p.rows) store16(p.y, p.yt, (row0 + r) * p.ldy + t * 16, v[r]);
        }
        if constexpr (MODE == kModeForwardQuant || MODE == kModeHadamardQuant) {
            const int qmax = (1 << (p.bits - 1)) - 1;
            const int64_t row_bytes = (static_cast<int64_t>(G::kN) * p.bits) >> 3;
#pragma unroll
            for (int r = 0; r < R; ++r) {
                float m = 0.f;
#pragma unroll
                for (int e = 0; e < 16; ++e) m = fmaxf(m, fabsf(v[r][e]));
                m = row_max<LOG_N>(m, red, r, group, t);
                float inv;
                const uint16_t s16 = row_scale(m, qmax, &inv);
                if (row0 + r < p.rows) {
                    if (t == 0) p.scales[row0 + r] = s16;
                    store_codes16(p.codes + (row0 + r) * row_bytes + t * 2 * p.bits, p.bits, v[r], inv);
                }
                if (stats) {  // uniform over the CTA: the barriers inside row_sum are reached by every thread
                    float s2 = 0.f, s4 = 0.f;
#pragma unroll
                    for (int e = 0; e < 16; ++e) {
                        const float sq = v[r][e] * v[r][e];
                        s2 += sq;
                        s4 = fmaf(sq, sq, s4);
                    }
                    s2 = row_sum<LOG_N>(s2, red, r, group, t);
                    s4 = row_sum<LOG_N>(s4, red, r, group, t);
                    if (row0 + r < p.rows) {
                        if (t == 0) {
                            p.rowstats[2 * (row0 + r)] = s2;
                            p.rowstats[2 * (row0 + r) + 1] = s4;
                        }
                        const int qmin = -(1 << (p.bits - 1));
#pragma unroll
                        for (int e = 0; e < 16; ++e) atomicAdd(&shist[quant1(v[r][e], inv, qmin, qmax) - qmin], 1u);
                    }
                }
            }
            if constexpr (G::kTPR >= 32) __syncthreads();  // red[] is reused by the next tile
        }
    }
    if (stats) {  // integer counts: the order of the additions does not matter
        __syncthreads();
        for (int i = threadIdx.x; i < (1 << p.bits); i += blockDim.x)
            if (shist[i] != 0u) atomicAdd(&p.hist[i], static_cast<unsigned long long>(shist[i]));
    }
}

// ---- backward ------------------------------------------------------------------------------------
// One thread owns the same pairs (stage, j) for every row its row group processes, so its d-theta sums need no
// atomics: they are kept in shared memory (one array [L][n/2] per row group; at n = 8192, where that would not fit
// beside the row buffer, the last stage's eight sums per thread stay in registers) for all rows of the CTA and written
// to the CTA's partial-sum slot once, at the end.  Rows are assigned to CTAs statically (tile = blockIdx.x + k *
// gridDim.x), which fixes the summation order.
template <int LOG_N>
struct BwdAcc {
    static constexpr int kSmemStages = LOG_N > 12 ? 12 : LOG_N;  // stages whose sums live in shared memory
    static constexpr int kFloats = kSmemStages * Geo<LOG_N>::kHalf;
};

template <int LOG_N, int P, int R>
__device__ __forceinline__ void backward_phase(float (&v)[R][16], float (&w)[R][16], const float2* __restrict__ tw,
                                               int t, float* __restrict__ sacc, float (&racc)[8]) {
    using PH = Phase<LOG_N, P>;
#pragma unroll
    for (int kk = 0; kk < PH::kNs; ++kk) {
        const int k = PH::kNs - 1 - kk;
        const int b = PH::kB0 + k;
        const int lb = PH::kF + k;
#pragma unroll
        for (int q = 0; q < 8; ++q) {
            const int e_lo = ((q >> lb) << (lb + 1)) | (q & ((1 << lb) - 1));
            const int e_hi = e_lo | (1 << lb);
            const int i = PH::idx(t, e_lo);
            const int j = ((i >> (b + 1)) << b) | (i & ((1 << b) - 1));
            const float2 cs = __ldg(&tw[b * Geo<LOG_N>::kHalf + j]);
            float d = 0.f;
#pragma unroll
            for (int r = 0; r < R; ++r) {
                // stage-output form of g^T (dG/dtheta) z:  g_hi * z'_lo - g_lo * z'_hi
                d += w[r][e_hi] * v[r][e_lo] - w[r][e_lo] * v[r][e_hi];
            }
            if (b < BwdAcc<LOG_N>::kSmemStages) {
                sacc[b * Geo<LOG_N>::kHalf + j] += d;
            } else {
                racc[q] += d;
            }
#pragma unroll
            for (int r = 0; r < R; ++r) {
                const float a = v[r][e_lo], bb = v[r][e_hi];
                v[r][e_lo] = cs.x * a + cs.y * bb;
                v[r][e_hi] = cs.x * bb - cs.y * a;
                const float ga = w[r][e_lo], gb = w[r][e_hi];
                w[r][e_lo] = cs.x * ga + cs.y * gb;
                w[r][e_hi] = cs.x * gb - cs.y * ga;
            }
        }
    }
}

template <int LOG_N, int P, int R>
__device__ __forceinline__ void backward_from(float (&v)[R][16], float (&w)[R][16], const float2* tw, float* rowbuf,
                                              int t, float* sacc, float (&racc)[8]) {
    backward_phase<LOG_N, P, R>(v, w, tw, t, sacc, racc);
    if constexpr (P > 0) {
        exchange<LOG_N, P, P - 1, R>(v, rowbuf, t);
        exchange<LOG_N, P, P - 1, R>(w, rowbuf, t);
        backward_from<LOG_N, P - 1, R>(v, w, tw, rowbuf, t, sacc, racc);
    }
}

// the pairs thread t owns in phase P (and the phases after it): zero the shared-memory sums (ZERO) or copy the sums to
// the partial-sum slot in global memory
template <int LOG_N, int P, bool ZERO>
__device__ __forceinline__ void visit_partials(int t, float* __restrict__ sacc, const float (&racc)[8], float* __restrict__ part) {
    using PH = Phase<LOG_N, P>;
#pragma unroll
    for (int k = 0; k < PH::kNs; ++k) {
        const int b = PH::kB0 + k;
        const int lb = PH::kF + k;
#pragma unroll
        for (int q = 0; q < 8; ++q) {
            const int e_lo = ((q >> lb) << (lb + 1)) | (q & ((1 << lb) - 1));
            const int i = PH::idx(t, e_lo);
            const int j = ((i >> (b + 1)) << b) | (i & ((1 << b) - 1));
            const int at = b * Geo<LOG_N>::kHalf + j;
            if (b < BwdAcc<LOG_N>::kSmemStages) {
                if (ZERO) sacc[at] = 0.f; else part[at] = sacc[at];
            } else if (!ZERO) {
                part[at] = racc[q];
            }
        }
    }
    if constexpr (P + 1 < Geo<LOG_N>::kPhases) visit_partials<LOG_N, P + 1, ZERO>(t, sacc, racc, part);
}

template <int LOG_N, int R>
__global__ void __launch_bounds__(Geo<LOG_N>::kThreads, 1) k_backward_generic(const BackwardParams p) {
    using G = Geo<LOG_N>;
    extern __shared__ __align__(16) float smem[];
    const int group = threadIdx.x / G::kTPR;
    const int t = threadIdx.x % G::kTPR;
    float* rowbuf = smem + group * R * G::kN;
    float* sacc = smem + G::kGroups * R * G::kN + group * BwdAcc<LOG_N>::kFloats;
    float* part = p.partial + (static_cast<int64_t>(blockIdx.x) * G::kGroups + group) * (LOG_N * G::kHalf);
    float racc[8];
#pragma unroll
    for (int q = 0; q < 8; ++q) racc[q] = 0.f;
    visit_partials<LOG_N, 0, true>(t, sacc, racc, part);  // each slot is only ever touched by its owner: no barrier

    constexpr int kRowsPerTile = G::kGroups * R;
    const int64_t tiles = (p.rows + kRowsPerTile - 1) / kRowsPerTile;
    for (int64_t tile = blockIdx.x; tile < tiles; tile += gridDim.x) {
        const int64_t row0 = tile * kRowsPerTile + group * R;
        float v[R][16], w[R][16];
#pragma unroll
        for (int r = 0; r < R; ++r) {
            load16(p.x, p.xt, (row0 + r) * p.ld + t * 16, row0 + r < p.rows, v[r]);
            load16(p.g, p.gt, (row0 + r) * p.ld + t * 16, row0 + r < p.rows, w[r]);
        }
        forward_from<LOG_N, 0, R>(v, p.tw, rowbuf, t);  // v = y = Q x, last-phase ownership
        if constexpr (G::kPhases > 1) exchange<LOG_N, 0, G::kPhases - 1, R>(w, rowbuf, t);
        backward_from<LOG_N, G::kPhases - 1, R>(v, w, p.tw, rowbuf, t, sacc, racc);
        if (p.dx != nullptr) {
#pragma unroll
            for (int r = 0; r < R; ++r)
                if (row0 + r < p.rows) store16(p.dx, p.dxt, (row0 + r) * p.ld + t * 16, w[r]);
        }
    }
    visit_partials<LOG_N, 0, false>(t, sacc, racc, part);
}

// dtheta[k] = sum over the partial slots in a fixed order (=> reproducible bits).  A block of 256 threads = 8 slot lanes
// x 32 angles (launch with (count + 31) / 32 blocks): lane y adds slots y, y + 8, ... in order, then the eight sums are
// added in lane order.  One thread per angle walking all slots took 13 - 18 us for 148 slots; this takes about 3.
static __global__ void __launch_bounds__(256) k_reduce_partials(const float* __restrict__ partial, int slots, int count,
                                                               float* __restrict__ out) {
    __shared__ float sh[8][32];
    const int x = threadIdx.x & 31, y = threadIdx.x >> 5;
    const int k = blockIdx.x * 32 + x;
    float acc = 0.f;
    if (k < count) {
#pragma unroll 4
        for (int s = y; s < slots; s += 8) acc += partial[static_cast<int64_t>(s) * count + k];
    }
    sh[y][x] = acc;
    __syncthreads();
    if (y == 0 && k < count) {
        float a = sh[0][x];
#pragma unroll
        for (int i = 1; i < 8; ++i) a += sh[i][x];
        out[k] = a;
    }
}

// twiddle table from angles: (cos, sin) evaluated in double, rounded once to fp32
static __global__ void k_build_twiddles(const float* __restrict__ theta, int count, float2* __restrict__ tw) {
    const int k = blockIdx.x * blockDim.x + threadIdx.x;
    if (k >= count) return;
    double s, c;
    sincos(static_cast<double>(theta[k]), &s, &c);
    tw[k] = make_float2(static_cast<float>(c), static_cast<float>(s));
}

}  // namespace bfq
