// Register-only measurement of FP32 FMA issue rates on the current GPU: how many cycles one scheduler needs per
// packed (fma.rn.f32x2) or scalar FMA when the instruction reads three distinct registers, as every rotation of a
// butterfly with per-pair constants does, and when it reads two.  No global traffic inside the timed loops; each warp
// times itself with the SM clock.  The numbers put the roofline's nominal "128 lanes per SM per cycle" beside what the
// register file actually delivers to this instruction pattern.
//
// Second measurement: SM cycles per tcgen05.mma (bf16 x bf16 -> fp32, M = 128, K = 16) as a function of N, operands in
// shared memory, one thread issuing back to back.  It prices the alternative of running merged butterfly stages as
// small dense blocks on the tensor cores (a 16 x 16 block per MMA) against the FP32 path.
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

// ---- tensor-core issue rate for small N -----------------------------------------------------------------------
constexpr int kMmaShapes = 4;
constexpr int kMmaIters = 256;  // x 4 K steps of 16
__constant__ int c_mma_n[kMmaShapes] = {16, 64, 128, 256};

__device__ __forceinline__ uint64_t desc_k_major_sw128(uint32_t addr) {
    // K-major tile, 128-byte swizzle: 8-row groups 1024 bytes apart
    return static_cast<uint64_t>((addr & 0x3FFFFu) >> 4) | (static_cast<uint64_t>(1) << 16) |
           (static_cast<uint64_t>(1024 >> 4) << 32) | (static_cast<uint64_t>(1) << 46) | (static_cast<uint64_t>(2) << 61);
}

// One CTA per SM; zero operands (the cycle count does not depend on the values); every wait is bounded.
__global__ void __launch_bounds__(128, 1) k_mma_rate(unsigned long long* __restrict__ cycles, int* __restrict__ status) {
    extern __shared__ uint8_t smem_raw[];
    const uint32_t sbase = (smem_u32(smem_raw) + 1023u) & ~1023u;
    const uint32_t a_tile = sbase, b_tile = sbase + 16384u, bar = sbase + 49152u, slot = bar + 8u;
    for (uint32_t e = threadIdx.x; e < 49152u / 16u; e += blockDim.x)
        asm volatile("st.shared.v4.u32 [%0], {%1,%1,%1,%1};" ::"r"(sbase + 16u * e), "r"(0u) : "memory");
    if (threadIdx.x == 0) {
        mbar_init(bar, 1);
        mbar_init_fence();
    }
    if (threadIdx.x < 32) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], 256;" ::"r"(slot) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    tmem_fence_before();
    __syncthreads();
    tmem_fence_after();
    uint32_t tmem = 0;
    asm volatile("ld.shared.u32 %0, [%1];" : "=r"(tmem) : "r"(slot));
    if (threadIdx.x == 0) {
        uint32_t parity = 0;
        for (int sh = 0; sh < kMmaShapes; ++sh) {
            const uint32_t n = static_cast<uint32_t>(c_mma_n[sh]);
            // fp32 accumulator, bf16 operands, both K-major, M = 128
            const uint32_t idesc = (1u << 4) | (1u << 7) | (1u << 10) | ((n >> 3) << 17) | ((128u >> 4) << 24);
            const long long t0 = sm_clock();
            for (int it = 0; it < kMmaIters; ++it) {
#pragma unroll
                for (uint32_t ks = 0; ks < 4; ++ks) {
                    asm volatile(
                        "{\n\t.reg .pred p;\n\t"
                        "setp.ne.b32 p, %4, 0;\n\t"
                        "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
                        ::"r"(tmem), "l"(desc_k_major_sw128(a_tile + 32u * ks)), "l"(desc_k_major_sw128(b_tile + 32u * ks)),
                        "r"(idesc), "r"(static_cast<uint32_t>(it | ks))
                        : "memory");
                }
            }
            asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
            bool done = false;
            for (int i = 0; i < (1 << 24) && !done; ++i) done = mbar_try_wait(bar, parity);
            const long long t1 = sm_clock();
            if (!done) {
                atomicExch(status, 1);
                break;
            }
            parity ^= 1u;
            atomicMax(cycles + sh, static_cast<unsigned long long>(t1 - t0));
        }
    }
    tmem_fence_before();
    __syncthreads();
    if (threadIdx.x < 32) asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, 256;" ::"r"(tmem) : "memory");
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

extern "C" int bfq_measure_mma_rates(float* cycles_per_mma) {
    using namespace bfq::rates;
    if (cycles_per_mma == nullptr) return BFQ_ERR_NULL;
    unsigned long long* cyc = nullptr;
    cudaError_t e = cudaMalloc(&cyc, (kMmaShapes + 1) * sizeof(unsigned long long));
    if (e == cudaSuccess) e = cudaMemset(cyc, 0, (kMmaShapes + 1) * sizeof(unsigned long long));
    int sms = 1, dev = 0;
    if (e == cudaSuccess) e = cudaGetDevice(&dev);
    if (e == cudaSuccess) e = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
    constexpr int kSmem = 49152 + 16 + 1024;
    if (e == cudaSuccess) e = cudaFuncSetAttribute(k_mma_rate, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmem);
    unsigned long long host[kMmaShapes + 1] = {0, 0, 0, 0, 0};
    if (e == cudaSuccess) {
        int* status = reinterpret_cast<int*>(cyc + kMmaShapes);
        for (int rep = 0; rep < 2; ++rep) {  // the second round counts
            if (rep == 1) cudaMemset(cyc, 0, kMmaShapes * sizeof(unsigned long long));
            k_mma_rate<<<sms, 128, kSmem>>>(cyc, status);
        }
        e = cudaDeviceSynchronize();
    }
    if (e == cudaSuccess) e = cudaMemcpy(host, cyc, sizeof(host), cudaMemcpyDeviceToHost);
    cudaFree(cyc);
    if (e != cudaSuccess) return BFQ_ERR_CUDA;
    if (host[kMmaShapes] != 0) return BFQ_ERR_DEVICE_TIMEOUT;
    for (int s = 0; s < kMmaShapes; ++s)
        cycles_per_mma[s] = static_cast<float>(static_cast<double>(host[s]) / (4.0 * kMmaIters));
    return BFQ_OK;
}
