// Register-only measurement of FP32 FMA issue rates on the current GPU: how many cycles one scheduler needs per
// packed (fma.rn.f32x2) or scalar FMA when the instruction reads three distinct registers, as every rotation of a
// butterfly with per-pair constants does, and when it reads two.  No global traffic inside the timed loops; each warp
// times itself with the SM clock.  The numbers put the roofline's nominal "128 lanes per SM per cycle" beside what the
// register file actually delivers to this instruction pattern.
#include "../../include/bfq.h"

#include <cuda_runtime.h>
#include <stdint.h>

#include "bfq_ptx.cuh"

namespace bfq {
namespace rates {
using namespace ptx;

constexpr int kThreads = 512;  // four warps per scheduler
constexpr int kIters = 2048;
enum : int { kPacked3 = 0, kPacked2 = 1, kScalar3 = 2, kScalar2 = 3, kPatterns = 4 };

__device__ __forceinline__ long long sm_clock() {
    long long c;
    asm volatile("mov.u64 %0, %%clock64;" : "=l"(c));
    return c;
}

// One scaled butterfly stage pattern on 16 packed registers: lo' = k1*hi + lo, hi' = k2*lo + hi (three distinct register
// operands per FMA), or the same with the constant replaced by an operand already read (two distinct).
template <int PATTERN>
__global__ void __launch_bounds__(kThreads, 1) k_rate(const float* __restrict__ seed, unsigned long long* __restrict__ cycles,
                                                       float* __restrict__ sink) {
    u64 P[16];
    uint32_t T[32];
#pragma unroll
    for (int i = 0; i < 16; ++i) P[i] = pack2(seed[(threadIdx.x + i) & 255], seed[(threadIdx.x + 3 * i + 1) & 255]);
#pragma unroll
    for (int i = 0; i < 32; ++i) T[i] = __float_as_uint(0.01f * seed[(7 * threadIdx.x + i) & 255]);
    __syncthreads();
    const long long t0 = sm_clock();
    for (int it = 0; it < kIters; ++it) {
#pragma unroll
        for (int K = 0; K < 4; ++K) {
#pragma unroll
            for (int u = 0; u < 8; ++u) {
                const int lo = ((u >> K) << (K + 1)) | (u & ((1 << K) - 1)), hi = lo | (1 << K);
                const u64 k1 = pack2u(T[4 * u], T[4 * u + 1]), k2 = pack2u(T[4 * u + 2], T[4 * u + 3]);
                const u64 a = P[lo], b = P[hi];
                if constexpr (PATTERN == kPacked3) {
                    P[lo] = fma2(k1, b, a);
                    P[hi] = fma2(k2, a, b);
                } else if constexpr (PATTERN == kPacked2) {
                    P[lo] = fma2(b, b, a);
                    P[hi] = fma2(a, a, b);
                } else {
                    float a0, a1, b0, b1;
                    unpack2(a, a0, a1);
                    unpack2(b, b0, b1);
                    const float c0 = __uint_as_float(T[4 * u]), c1 = __uint_as_float(T[4 * u + 1]);
                    const float c2 = __uint_as_float(T[4 * u + 2]), c3 = __uint_as_float(T[4 * u + 3]);
                    if constexpr (PATTERN == kScalar3) {
                        P[lo] = pack2(fmaf(c0, b0, a0), fmaf(c1, b1, a1));
                        P[hi] = pack2(fmaf(c2, a0, b0), fmaf(c3, a1, b1));
                    } else {
                        P[lo] = pack2(fmaf(b0, b0, a0), fmaf(b1, b1, a1));
                        P[hi] = pack2(fmaf(a0, a0, b0), fmaf(a1, a1, b1));
                    }
                }
            }
        }
    }
    const long long t1 = sm_clock();
    float acc = 0.f;
#pragma unroll
    for (int i = 0; i < 16; ++i) {
        float a, b;
        unpack2(P[i], a, b);
        acc += a + b;
    }
    if (acc == 12345.678f) sink[0] = acc;  // keeps the loop alive
    if ((threadIdx.x & 31) == 0) atomicMax(cycles + PATTERN, static_cast<unsigned long long>(t1 - t0));
}

}  // namespace rates
}  // namespace bfq

extern "C" int bfq_measure_fma_rates(float* cycles_per_instruction) {
    using namespace bfq::rates;
    if (cycles_per_instruction == nullptr) return BFQ_ERR_NULL;
    float host_seed[256];
    for (int i = 0; i < 256; ++i) host_seed[i] = 0.001f * static_cast<float>(i % 7) - 0.003f;
    float* seed = nullptr;
    unsigned long long* cyc = nullptr;
    cudaError_t e = cudaMalloc(&seed, sizeof(host_seed) + sizeof(float));
    if (e == cudaSuccess) e = cudaMalloc(&cyc, kPatterns * sizeof(unsigned long long));
    if (e == cudaSuccess) e = cudaMemcpy(seed, host_seed, sizeof(host_seed), cudaMemcpyHostToDevice);
    if (e == cudaSuccess) e = cudaMemset(cyc, 0, kPatterns * sizeof(unsigned long long));
    int sms = 1;
    int dev = 0;
    if (e == cudaSuccess) e = cudaGetDevice(&dev);
    if (e == cudaSuccess) e = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
    if (e == cudaSuccess) {
        float* sink = seed + 256;
        for (int rep = 0; rep < 2; ++rep) {  // the first round warms the clocks up; the maximum over warps is kept
            if (rep == 1) cudaMemset(cyc, 0, kPatterns * sizeof(unsigned long long));
            k_rate<kPacked3><<<sms, kThreads>>>(seed, cyc, sink);
            k_rate<kPacked2><<<sms, kThreads>>>(seed, cyc, sink);
            k_rate<kScalar3><<<sms, kThreads>>>(seed, cyc, sink);
            k_rate<kScalar2><<<sms, kThreads>>>(seed, cyc, sink);
        }
        e = cudaDeviceSynchronize();
    }
    unsigned long long host_cyc[kPatterns] = {0, 0, 0, 0};
    if (e == cudaSuccess) e = cudaMemcpy(host_cyc, cyc, sizeof(host_cyc), cudaMemcpyDeviceToHost);
    cudaFree(seed);
    cudaFree(cyc);
    if (e != cudaSuccess) return BFQ_ERR_CUDA;
    // every scheduler runs kThreads / 128 warps; a warp issues 64 (packed) or 128 (scalar) FMAs per iteration
    const double warps_per_scheduler = kThreads / 128.0;
    for (int p = 0; p < kPatterns; ++p) {
        const double per_warp = (p < 2 ? 64.0 : 128.0) * kIters;
        cycles_per_instruction[p] = static_cast<float>(static_cast<double>(host_cyc[p]) / (per_warp * warps_per_scheduler));
    }
    return BFQ_OK;
}
