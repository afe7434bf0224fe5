// Composite transform for row lengths that are not a power of two (paper Sec. 3.3, "Kronecker product
// construction"): d = n1 * n2, Q = Q1 (x) Q2 with Q2 the plan's butterfly on n2 = 2^k points and Q1 a dense
// orthogonal n1 x n1 factor, Q1 = (I - A)(I + A)^{-1} with A skew-symmetric (Cayley transform; the paper's
// example is d = 5120 = 40 x 128 with 780 + 448 parameters).
//
// Seen as an n1 x n2 matrix X (row r = the r-th run of n2 consecutive elements), one token maps to
//     Y = Q1 (X Q2^T):   the butterfly on every run, then the dense factor across the runs.
//
// This file holds the Cayley solve and the kernels that work for every (n1 <= 64, n2 <= 1024, n1 n2 <= 16384);
// the tensor-core kernels for 40 x 128 live in bfq_comp5120d.cu (both factors as MMAs) and bfq_comp5120.cu (fp32
// butterfly + MMA dense factor) and must agree with these.
#include <cuda_runtime.h>

#include "bfq_fast.h"
#include "bfq_generic.cuh"

namespace bfq {
namespace comp {

// ---- Q1 = (I - A)(I + A)^{-1} -------------------------------------------------------------------------------
// (I - A) and (I + A)^{-1} commute, so Q1 solves (I + A) Q1 = I - A: Gauss-Jordan with partial pivoting on the
// augmented matrix [I + A | I - A], one CTA, float64 in shared memory (I + A has all singular values >= 1).
constexpr int kCayleyThreads = 256;

__global__ void __launch_bounds__(kCayleyThreads) k_cayley(const float* __restrict__ params, int n1, float* __restrict__ q1) {
    extern __shared__ double aug[];  // [n1][2 n1]
    __shared__ int pivot_row;
    const int t = threadIdx.x, w = 2 * n1;
    for (int e = t; e < n1 * n1; e += kCayleyThreads) {
        const int i = e / n1, j = e % n1;
        double a = 0.0;
        if (i < j) a = static_cast<double>(params[i * n1 - i * (i + 1) / 2 + (j - i - 1)]);
        if (i > j) a = -static_cast<double>(params[j * n1 - j * (j + 1) / 2 + (i - j - 1)]);
        const double id = (i == j) ? 1.0 : 0.0;
        aug[i * w + j] = id + a;
        aug[i * w + n1 + j] = id - a;
    }
    __syncthreads();
    for (int col = 0; col < n1; ++col) {
        if (t == 0) {
            int best = col;
            double bv = fabs(aug[col * w + col]);
            for (int r = col + 1; r < n1; ++r) {
                const double v = fabs(aug[r * w + col]);
                if (v > bv) bv = v, best = r;
            }
            pivot_row = best;
        }
        __syncthreads();
        const int pr = pivot_row;
        if (pr != col) {
            for (int j = t; j < w; j += kCayleyThreads) {
                const double tmp = aug[col * w + j];
                aug[col * w + j] = aug[pr * w + j];
                aug[pr * w + j] = tmp;
            }
        }
        __syncthreads();
        const double inv = 1.0 / aug[col * w + col];
        __syncthreads();
        for (int j = t; j < w; j += kCayleyThreads) aug[col * w + j] *= inv;
        __syncthreads();
        // eliminate the column from every other row; the factors are read before any row changes them
        for (int e = t; e < n1 * w; e += kCayleyThreads) {
            const int r = e / w, j = e % w;
            if (r == col || j == col) continue;
            aug[r * w + j] -= aug[r * w + col] * aug[col * w + j];
        }
        __syncthreads();
        for (int r = t; r < n1; r += kCayleyThreads)
            if (r != col) aug[r * w + col] = 0.0;
        __syncthreads();
    }
    for (int e = t; e < n1 * n1; e += kCayleyThreads) q1[e] = static_cast<float>(aug[(e / n1) * w + n1 + (e % n1)]);
}

// ---- generic composite forward: one token per CTA iteration ----------------------------------------------------
constexpr int kThreads = 256;
constexpr int kWarps = kThreads / 32;

struct CompositeParams {
    const float2* tw;  // [log2 n2][n2/2] (cos, sin) of Q2
    const float* q1;   // [n1][n1] row-major
    int n1, n2, log_n2;
    const void* x;
    int xt;
    int64_t ldx;
    void* y;  // unquantized output rows, or null
    int yt;
    int64_t ldy;
    uint8_t* codes;  // quantized output, or null
    uint16_t* scales;
    int bits;
    int64_t rows;
    int inverse;  // 1: x = (Q1 kron Q2)^T y: inverse butterfly on every run (stages last to first, G^T), then Q1^T
};

__global__ void __launch_bounds__(kThreads) k_composite_generic(const CompositeParams p) {
    extern __shared__ float sm[];
    const int n1 = p.n1, n2 = p.n2, d = n1 * n2, h2 = n2 >> 1, n1p = (n1 + 7) & ~7;
    float* buf = sm;             // [n1][n2] the token, then X Q2^T
    float* out = sm + d;         // [n1][n2] Y
    float* q1s = sm + 2 * d;     // [n1p][n1], rows n1..n1p-1 zero
    __shared__ float red[kWarps];
    const int t = threadIdx.x;
    for (int e = t; e < n1p * n1; e += kThreads) {  // row i of the factor applied: Q1[i][:] or, for the inverse, Q1[:][i]
        const int i = e / n1, k = e - i * n1;
        q1s[e] = i < n1 ? (p.inverse ? p.q1[k * n1 + i] : p.q1[e]) : 0.f;
    }

    for (int64_t row = blockIdx.x; row < p.rows; row += gridDim.x) {
        __syncthreads();  // previous token's readers of buf / out are done
        for (int c = t; c < d / 16; c += kThreads) {
            float v[16];
            load16(p.x, p.xt, row * p.ldx + 16 * c, true, v);
#pragma unroll
            for (int e = 0; e < 16; ++e) buf[16 * c + e] = v[e];
        }
        // Q2 (or Q2^T) on every run: stage s couples lo and lo + 2^s inside the run
        for (int ss = 0; ss < p.log_n2; ++ss) {
            __syncthreads();
            const int s = p.inverse ? p.log_n2 - 1 - ss : ss;
            const float sgn = p.inverse ? -1.f : 1.f;
            const float2* tws = p.tw + s * h2;
            for (int pr = t; pr < d / 2; pr += kThreads) {
                const int r = pr / h2, q = pr - r * h2;
                const int lo = r * n2 + (((q >> s) << (s + 1)) | (q & ((1 << s) - 1))), hi = lo + (1 << s);
                float2 cs = __ldg(tws + q);
                cs.y *= sgn;
                const float a = buf[lo], b = buf[hi];
                buf[lo] = fmaf(cs.x, a, -cs.y * b);
                buf[hi] = fmaf(cs.y, a, cs.x * b);
            }
        }
        __syncthreads();
        // Q1 across the runs: Y[i][j] = sum_k Q1[i][k] X'[k][j]; a thread owns one j and eight i
        float amax = 0.f;
        for (int item = t; item < n2 * (n1p / 8); item += kThreads) {
            const int j = item % n2, i0 = 8 * (item / n2);
            float acc[8] = {0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f};
            for (int k = 0; k < n1; ++k) {
                const float v = buf[k * n2 + j];
#pragma unroll
                for (int u = 0; u < 8; ++u) acc[u] = fmaf(q1s[(i0 + u) * n1 + k], v, acc[u]);
            }
#pragma unroll
            for (int u = 0; u < 8; ++u)
                if (i0 + u < n1) {
                    out[(i0 + u) * n2 + j] = acc[u];
                    amax = fmaxf(amax, fabsf(acc[u]));
                }
        }
        float inv = 0.f;
        if (p.codes != nullptr) {  // per-token scale over all d elements (Sec. 3.4 quantizer)
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) amax = fmaxf(amax, __shfl_xor_sync(0xffffffffu, amax, o));
            if ((t & 31) == 0) red[t >> 5] = amax;
            __syncthreads();
            amax = red[0];
#pragma unroll
            for (int wi = 1; wi < kWarps; ++wi) amax = fmaxf(amax, red[wi]);
            const uint16_t sb = row_scale(amax, (1 << (p.bits - 1)) - 1, &inv);
            if (t == 0) p.scales[row] = sb;
        } else {
            __syncthreads();
        }
        for (int c = t; c < d / 16; c += kThreads) {
            float v[16];
#pragma unroll
            for (int e = 0; e < 16; ++e) v[e] = out[16 * c + e];
            if (p.codes != nullptr)
                store_codes16(p.codes + (row * d + 16 * c) * p.bits / 8, p.bits, v, inv);
            if (p.y != nullptr) store16(p.y, p.yt, row * p.ldy + 16 * c, v);
        }
    }
}

}  // namespace comp

cudaError_t cayley_launch(const float* params, int n1, float* q1, cudaStream_t st) {
    const size_t smem = sizeof(double) * 2 * n1 * n1;
    cudaError_t e = cudaFuncSetAttribute(comp::k_cayley, cudaFuncAttributeMaxDynamicSharedMemorySize, int(smem));
    if (e != cudaSuccess) return e;
    comp::k_cayley<<<1, comp::kCayleyThreads, smem, st>>>(params, n1, q1);
    return cudaGetLastError();
}

cudaError_t composite_generic_launch(const bfq_plan* plan, const float* q1, int n1, const void* x, int xt, int64_t rows,
                                     int64_t ldx, void* y, int yt, int64_t ldy, int bits, uint8_t* codes,
                                     uint16_t* scales, bool inverse, cudaStream_t st) {
    comp::CompositeParams p{};
    p.tw = plan->tw, p.q1 = q1, p.n1 = n1, p.n2 = plan->n, p.log_n2 = plan->log_n;
    p.x = x, p.xt = xt, p.ldx = ldx, p.y = y, p.yt = yt, p.ldy = ldy;
    p.codes = codes, p.scales = scales, p.bits = bits, p.rows = rows, p.inverse = inverse ? 1 : 0;
    const int d = n1 * plan->n, n1p = (n1 + 7) & ~7;
    const size_t smem = sizeof(float) * (size_t(2) * d + size_t(n1p) * n1);
    cudaError_t e = cudaFuncSetAttribute(comp::k_composite_generic, cudaFuncAttributeMaxDynamicSharedMemorySize, int(smem));
    if (e != cudaSuccess) return e;
    const int64_t cap = int64_t(plan->sm_count) * 4;
    const int grid = int(rows < cap ? rows : cap);
    comp::k_composite_generic<<<grid, comp::kThreads, smem, st>>>(p);
    return cudaGetLastError();
}

}  // namespace bfq
