// bfq_backward_noalloc: the backward pass for callers that must not allocate device memory.
//
// Some hosts of this library cannot let it call cudaMalloc: a serving process whose device memory is
// owned in full by a framework's caching allocator (a raw allocation can fail or fragment it), or a
// latency-critical loop in which the device-wide synchronisation that cudaMalloc / cudaFree imply is
// not acceptable.  bfq_plan_create allocates (tables, partial sums), so such callers cannot use the
// plan-based entry points.  This entry point needs no plan: everything the backward pass needs
// beyond the caller's own buffers (the cos/sin table and the per-CTA partial sums of d-theta) lives
// in one fixed array in the library's device data segment, which every GPU that loads the library
// holds until the process exits.
//
// Consequences of the shared array: the row length is limited to BFQ_NOALLOC_MAX_N; all calls (from
// any stream or thread) use the same bytes, so two calls that overlap on one GPU race; the array
// keeps the previous call's contents, and each call rewrites the table and overwrites exactly the
// partial sums it is going to read (every CTA stores its finished sums into its own slots).
#include "../../include/bfq.h"

#include <cuda_runtime.h>

#include "bfq_generic.cuh"
#include "bfq_plan.h"

namespace bfq {
namespace noalloc {

constexpr size_t kScratchBytes = size_t(8) << 20;  // 8 MiB per GPU
constexpr size_t kTableBytes = size_t(10) * (BFQ_NOALLOC_MAX_N / 2) * sizeof(float2);  // 40 KiB at n = 1024

// In host code this name is only a handle for cudaGetSymbolAddress, never a device address.
static __device__ __align__(256) unsigned char g_scratch[kScratchBytes];

struct PerDevice {
    void* base = nullptr;  // device address of g_scratch on this GPU
    int sm_count = 0;
};
static PerDevice g_dev[kMaxDevices];

// First call on a device (that device being current): resolve the array's device address.
static cudaError_t setup(int device, PerDevice** out) {
    PerDevice& d = g_dev[device];
    if (d.base == nullptr) {
        void* p = nullptr;
        cudaError_t e = cudaGetSymbolAddress(&p, g_scratch);
        if (e != cudaSuccess) return e;
        int sms = 0;
        e = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, device);
        if (e != cudaSuccess) return e;
        d.sm_count = sms;
        d.base = p;
    }
    *out = &d;
    return cudaSuccess;
}

template <int LOG_N>
static cudaError_t launch(int device, const PerDevice& d, BackwardParams p, const float* theta, float* dtheta,
                          cudaStream_t st) {
    using G = Geo<LOG_N>;
    constexpr int R = 1;
    constexpr size_t smem = sizeof(float) * size_t(G::kGroups) * (size_t(R) * G::kN + BwdAcc<LOG_N>::kFloats);
    constexpr int count = LOG_N * G::kHalf;
    auto kern = k_backward_generic<LOG_N, R>;
    static bool attr_set[kMaxDevices] = {false};
    cudaError_t e;
    if (!attr_set[device]) {
        e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, int(smem));
        if (e != cudaSuccess) return e;
        attr_set[device] = true;
    }
    float2* tw = reinterpret_cast<float2*>(d.base);
    float* partial = reinterpret_cast<float*>(static_cast<unsigned char*>(d.base) + kTableBytes);
    // as many CTAs as the array has room for partial sums, at most two per SM
    const int64_t max_slots = int64_t((kScratchBytes - kTableBytes) / (sizeof(float) * count));
    int64_t cap = max_slots / G::kGroups;
    if (cap > 2 * int64_t(d.sm_count)) cap = 2 * int64_t(d.sm_count);
    if (cap < 1) return cudaErrorInvalidValue;
    constexpr int rows_per_tile = G::kGroups * R;
    const int64_t tiles = (p.rows + rows_per_tile - 1) / rows_per_tile;
    const int grid = int(tiles < cap ? tiles : cap);
    k_build_twiddles<<<(count + 255) / 256, 256, 0, st>>>(theta, count, tw);
    e = cudaGetLastError();
    if (e != cudaSuccess) return e;
    p.tw = tw;
    p.partial = partial;  // every CTA overwrites its own slots with its finished sums
    kern<<<grid, G::kThreads, smem, st>>>(p);
    e = cudaGetLastError();
    if (e != cudaSuccess) return e;
    k_reduce_partials<<<(count + 31) / 32, 256, 0, st>>>(partial, grid * G::kGroups, count, dtheta);
    return cudaGetLastError();
}

}  // namespace noalloc
}  // namespace bfq

using namespace bfq;

extern "C" int bfq_backward_noalloc(int n, const float* theta, const void* x, bfq_dtype xt, const void* g,
                                    bfq_dtype gt, int64_t rows, int64_t ld, void* dx, bfq_dtype dxt, float* dtheta,
                                    void* stream) {
    int log_n = 0;
    while ((1 << log_n) < n && log_n < 30) ++log_n;
    if (n < BFQ_MIN_N || n > BFQ_MAX_N || (1 << log_n) != n) return BFQ_ERR_UNSUPPORTED_N;
    if (n > BFQ_NOALLOC_MAX_N) return BFQ_ERR_TOO_LARGE;
    if (theta == nullptr || dtheta == nullptr) return BFQ_ERR_NULL;
    if ((x == nullptr || g == nullptr) && rows != 0) return BFQ_ERR_NULL;
    const auto dtype_ok = [](int dt) { return dt == BFQ_F32 || dt == BFQ_BF16; };
    if (!dtype_ok(xt) || !dtype_ok(gt) || (dx != nullptr && !dtype_ok(dxt))) return BFQ_ERR_DTYPE;
    const auto esize = [](int dt) { return dt == BFQ_F32 ? 4 : 2; };
    if (rows < 0 || ld < n || ((ld * esize(xt)) & 15) != 0 || ((ld * esize(gt)) & 15) != 0 ||
        (dx != nullptr && ((ld * esize(dxt)) & 15) != 0))
        return BFQ_ERR_STRIDE;
    const auto misaligned = [](const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) != 0; };
    if (misaligned(x) || misaligned(g) || misaligned(dx) || misaligned(dtheta) ||
        (reinterpret_cast<uintptr_t>(theta) & 3u) != 0)
        return BFQ_ERR_ALIGN;
    int device = 0;
    if (cudaGetDevice(&device) != cudaSuccess || device < 0 || device >= kMaxDevices) return BFQ_ERR_CUDA;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    if (rows == 0) {
        return cudaMemsetAsync(dtheta, 0, sizeof(float) * size_t(log_n) * (n / 2), st) == cudaSuccess ? BFQ_OK
                                                                                                       : BFQ_ERR_CUDA;
    }
    noalloc::PerDevice* d = nullptr;
    if (noalloc::setup(device, &d) != cudaSuccess) return BFQ_ERR_CUDA;
    BackwardParams p{};
    p.x = x, p.xt = xt, p.g = g, p.gt = gt, p.ld = ld, p.dx = dx, p.dxt = dxt, p.rows = rows;
    cudaError_t e;
    switch (log_n) {
        case 4: e = noalloc::launch<4>(device, *d, p, theta, dtheta, st); break;
        case 5: e = noalloc::launch<5>(device, *d, p, theta, dtheta, st); break;
        case 6: e = noalloc::launch<6>(device, *d, p, theta, dtheta, st); break;
        case 7: e = noalloc::launch<7>(device, *d, p, theta, dtheta, st); break;
        case 8: e = noalloc::launch<8>(device, *d, p, theta, dtheta, st); break;
        case 9: e = noalloc::launch<9>(device, *d, p, theta, dtheta, st); break;
        case 10: e = noalloc::launch<10>(device, *d, p, theta, dtheta, st); break;
        default: return BFQ_ERR_TOO_LARGE;
    }
    return e == cudaSuccess ? BFQ_OK : BFQ_ERR_CUDA;
}
