// C ABI of the bfq library: plan management, argument validation, kernel dispatch.
// See include/bfq.h for the contract of every entry point.
#include "../../include/bfq.h"

#include <cuda_runtime.h>

#include <cstdio>
#include <cstdlib>
#include <new>

#include "bfq_fast.h"
#include "bfq_generic.cuh"
#include "bfq_plan.h"

namespace bfq {

static bool env_flag(const char* name) {
    const char* v = std::getenv(name);
    return v != nullptr && v[0] != '\0' && v[0] != '0';
}

static int ilog2_exact(int64_t n) {
    int L = 0;
    while ((int64_t(1) << L) < n) ++L;
    return (int64_t(1) << L) == n ? L : -1;
}

struct DeviceGuard {
    int prev = -1;
    bool switched = false;
    cudaError_t err = cudaSuccess;
    explicit DeviceGuard(int device) {
        err = cudaGetDevice(&prev);
        if (err == cudaSuccess && prev != device) {
            err = cudaSetDevice(device);
            switched = (err == cudaSuccess);
        }
    }
    ~DeviceGuard() {
        if (switched) cudaSetDevice(prev);
    }
};

static int cuda_fail(bfq_plan* plan, cudaError_t e) {
    if (plan != nullptr) plan->last_cuda_error = static_cast<int>(e);
    if (env_flag("BFQ_LOG")) std::fprintf(stderr, "[bfq] CUDA error %d: %s\n", int(e), cudaGetErrorString(e));
    return BFQ_ERR_CUDA;
}

static bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }
static int esize(int dt) { return dt == BFQ_F32 ? 4 : 2; }
static bool dtype_ok(int dt) { return dt == BFQ_F32 || dt == BFQ_BF16; }

static int check_rows(const void* p, int dt, int64_t rows, int64_t ld, int n) {
    if (p == nullptr && rows != 0) return BFQ_ERR_NULL;  // an empty batch may come with a null pointer
    if (!dtype_ok(dt)) return BFQ_ERR_DTYPE;
    if (rows < 0 || ld < n || ((ld * esize(dt)) & 15) != 0) return BFQ_ERR_STRIDE;
    if (!aligned16(p)) return BFQ_ERR_ALIGN;
    return BFQ_OK;
}

// ---- generic kernel dispatch ------------------------------------------------------------------------
template <int LOG_N, int R, int MODE>
static cudaError_t launch_generic_t(const bfq_plan* plan, const GenericParams& p, cudaStream_t st) {
    using G = Geo<LOG_N>;
    // rows being regrouped + per-row reduction slots + the 256-bin code histogram of the statistics variant
    constexpr size_t smem =
        sizeof(float) * (size_t(G::kGroups) * R * G::kN + size_t(R) * G::kGroups * G::kWarpsPerRow + 256);
    static int blocks_per_sm[kMaxDevices] = {0};
    auto kern = k_generic<LOG_N, R, MODE>;
    int& occ = blocks_per_sm[plan->device];
    if (occ == 0) {
        cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, int(smem));
        if (e != cudaSuccess) return e;
        int o = 0;
        e = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&o, kern, G::kThreads, smem);
        if (e != cudaSuccess) return e;
        occ = o > 0 ? o : 1;
    }
    constexpr int rows_per_tile = G::kGroups * R;
    const int64_t tiles = (p.rows + rows_per_tile - 1) / rows_per_tile;
    const int64_t cap = int64_t(plan->sm_count) * occ;
    const int grid = int(tiles < cap ? tiles : cap);
    kern<<<grid, G::kThreads, smem, st>>>(p);
    return cudaGetLastError();
}

template <int MODE>
static cudaError_t launch_generic(const bfq_plan* plan, const GenericParams& p, cudaStream_t st) {
    switch (plan->log_n) {
        case 4: return launch_generic_t<4, 2, MODE>(plan, p, st);
        case 5: return launch_generic_t<5, 2, MODE>(plan, p, st);
        case 6: return launch_generic_t<6, 2, MODE>(plan, p, st);
        case 7: return launch_generic_t<7, 2, MODE>(plan, p, st);
        case 8: return launch_generic_t<8, 2, MODE>(plan, p, st);
        case 9: return launch_generic_t<9, 2, MODE>(plan, p, st);
        case 10: return launch_generic_t<10, 2, MODE>(plan, p, st);
        case 11: return launch_generic_t<11, 4, MODE>(plan, p, st);
        case 12: return launch_generic_t<12, 4, MODE>(plan, p, st);
        case 13: return launch_generic_t<13, 4, MODE>(plan, p, st);
        default: return cudaErrorInvalidValue;
    }
}

template <int LOG_N, int R>
static cudaError_t launch_backward_t(bfq_plan* plan, BackwardParams p, float* dtheta, cudaStream_t st) {
    using G = Geo<LOG_N>;
    // row buffers + the d-theta sums of every row group
    constexpr size_t smem = sizeof(float) * size_t(G::kGroups) * (size_t(R) * G::kN + BwdAcc<LOG_N>::kFloats);
    static int blocks_per_sm[kMaxDevices] = {0};
    auto kern = k_backward_generic<LOG_N, R>;
    int& occ = blocks_per_sm[plan->device];
    if (occ == 0) {
        cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, int(smem));
        if (e != cudaSuccess) return e;
        int o = 0;
        e = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&o, kern, G::kThreads, smem);
        if (e != cudaSuccess) return e;
        occ = o > 0 ? o : 1;
    }
    constexpr int rows_per_tile = G::kGroups * R;
    const int64_t tiles = (p.rows + rows_per_tile - 1) / rows_per_tile;
    int64_t cap = int64_t(plan->sm_count) * (occ < kBackwardCtasPerSm ? occ : kBackwardCtasPerSm);
    if (cap * G::kGroups > plan->partial_slots) cap = plan->partial_slots / G::kGroups;
    if (cap < 1) return cudaErrorInvalidValue;
    const int grid = int(tiles < cap ? tiles : cap);
    p.partial = plan->partial;
    kern<<<grid, G::kThreads, smem, st>>>(p);
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return e;
    const int count = LOG_N * G::kHalf;
    k_reduce_partials<<<(count + 31) / 32, 256, 0, st>>>(plan->partial, grid * G::kGroups, count, dtheta);
    plan->last_backward_partials = grid * G::kGroups;
    return cudaGetLastError();
}

static cudaError_t launch_backward(bfq_plan* plan, const BackwardParams& p, float* dtheta, cudaStream_t st) {
    switch (plan->log_n) {
        case 4: return launch_backward_t<4, 1>(plan, p, dtheta, st);
        case 5: return launch_backward_t<5, 1>(plan, p, dtheta, st);
        case 6: return launch_backward_t<6, 1>(plan, p, dtheta, st);
        case 7: return launch_backward_t<7, 1>(plan, p, dtheta, st);
        case 8: return launch_backward_t<8, 1>(plan, p, dtheta, st);
        case 9: return launch_backward_t<9, 1>(plan, p, dtheta, st);
        case 10: return launch_backward_t<10, 1>(plan, p, dtheta, st);
        case 11: return launch_backward_t<11, 1>(plan, p, dtheta, st);
        case 12: return launch_backward_t<12, 1>(plan, p, dtheta, st);
        case 13: return launch_backward_t<13, 1>(plan, p, dtheta, st);
        default: return cudaErrorInvalidValue;
    }
}

// slots needed by the generic backward for this n: CTAs * row groups per CTA
static int64_t backward_slots(int log_n, int sm_count) {
    const int n = 1 << log_n;
    const int tpr = n / 16;
    const int threads = tpr > 256 ? tpr : 256;
    return int64_t(sm_count) * kBackwardCtasPerSm * (threads / tpr);
}

// frees everything a plan owns (every pointer is null or valid) and the plan itself
static void release_plan(bfq_plan* plan) {
    cudaFree(plan->tw);
    cudaFree(plan->img4096);
    cudaFree(plan->prep4096);
    cudaFree(plan->img_b4096);
    cudaFree(plan->img_i4096);
    cudaFree(plan->img8192);
    cudaFree(plan->prep8192);
    for (int h = 0; h < 2; ++h) {
        cudaFree(plan->img_b8192[h]);
        cudaFree(plan->img_i8192[h]);
        cudaFree(plan->dsign8192[h]);
        cudaFree(plan->gsign8192[h]);
    }
    cudaFree(plan->prep_half8192);
    cudaFree(plan->dsign4096);
    cudaFree(plan->gsign4096);
    cudaFree(plan->partial);
    cudaFree(plan->status_word);
    if (plan->host_in != nullptr) cudaStreamDestroy(plan->host_in);
    if (plan->host_out != nullptr) cudaStreamDestroy(plan->host_out);
    for (int i = 0; i < 8; ++i)
        if (plan->host_ev[i] != nullptr) cudaEventDestroy(plan->host_ev[i]);
    cudaFree(plan->dense128);
    if (plan->theta_host != nullptr) cudaFreeHost(plan->theta_host);
    if (plan->theta_event != nullptr) cudaEventDestroy(plan->theta_event);
    std::free(plan->comp5120);
    delete plan;
}

}  // namespace bfq

using namespace bfq;

extern "C" {

int bfq_plan_create(bfq_plan** out, int n, int64_t max_rows, int device) {
    if (out == nullptr) return BFQ_ERR_NULL;
    *out = nullptr;
    if (n < BFQ_MIN_N || n > BFQ_MAX_N || ilog2_exact(n) < 0) return BFQ_ERR_UNSUPPORTED_N;
    if (max_rows < 0) return BFQ_ERR_STRIDE;
    if (device < 0 || device >= kMaxDevices) return BFQ_ERR_CUDA;
    int count = 0;
    cudaError_t e = cudaGetDeviceCount(&count);
    if (e != cudaSuccess) return cuda_fail(nullptr, e);
    if (device >= count) return BFQ_ERR_CUDA;
    DeviceGuard guard(device);
    if (guard.err != cudaSuccess) return cuda_fail(nullptr, guard.err);

    bfq_plan* plan = new (std::nothrow) bfq_plan();
    if (plan == nullptr) return BFQ_ERR_WORKSPACE;
    plan->n = n;
    plan->log_n = ilog2_exact(n);
    plan->device = device;
    cudaDeviceProp prop;
    e = cudaGetDeviceProperties(&prop, device);
    if (e != cudaSuccess) {
        delete plan;
        return cuda_fail(nullptr, e);
    }
    plan->sm_count = prop.multiProcessorCount;
    plan->cc_major = prop.major;
    const size_t angles = size_t(plan->log_n) * (n / 2);
    plan->partial_slots = backward_slots(plan->log_n, plan->sm_count);
    e = cudaMalloc(&plan->tw, angles * sizeof(float2));
    plan->partial_floats = size_t(plan->partial_slots) * angles;
    if (n == 8192 && plan->partial_floats < bwd8192_partial_floats(plan->sm_count))
        plan->partial_floats = bwd8192_partial_floats(plan->sm_count);
    if (e == cudaSuccess) e = cudaMalloc(&plan->partial, plan->partial_floats * sizeof(float));
    if (e == cudaSuccess && n == 4096) e = cudaMalloc(&plan->img4096, fwdq4096_image_bytes());
    if (e == cudaSuccess && n == 4096) e = cudaMalloc(&plan->prep4096, fwdq4096_prep_bytes());
    if (e == cudaSuccess && n == 8192) e = cudaMalloc(&plan->img8192, fwdq8192_image_bytes());
    if (e == cudaSuccess && n == 8192) e = cudaMalloc(&plan->prep8192, fwdq8192_prep_bytes());
    for (int h = 0; h < 2 && n == 8192; ++h) {
        if (e == cudaSuccess) e = cudaMalloc(&plan->img_b8192[h], bwd4096_image_bytes());
        if (e == cudaSuccess) e = cudaMalloc(&plan->img_i8192[h], inv4096_image_bytes());
        if (e == cudaSuccess) e = cudaMalloc(&plan->dsign8192[h], bwd4096_dsign_bytes());
        if (e == cudaSuccess) e = cudaMalloc(&plan->gsign8192[h], bwd4096_gsign_bytes());
    }
    if (e == cudaSuccess && n == 8192) e = cudaMalloc(&plan->prep_half8192, bwd8192_prep_bytes());
    if (e == cudaSuccess && n == 4096) e = cudaMalloc(&plan->img_b4096, bwd4096_image_bytes());
    if (e == cudaSuccess && n == 4096) e = cudaMalloc(&plan->img_i4096, inv4096_image_bytes());
    if (e == cudaSuccess && n == 4096) e = cudaMalloc(&plan->dsign4096, bwd4096_dsign_bytes());
    if (e == cudaSuccess && n == 4096) e = cudaMalloc(&plan->gsign4096, bwd4096_gsign_bytes());
    if (e == cudaSuccess && n == 128) e = cudaMalloc(&plan->dense128, comp5120d_image_bytes());
    if (e == cudaSuccess && n == 128) {  // the composite kernel's constants are computed on the host from the angles
        e = cudaMallocHost(&plan->theta_host, angles * sizeof(float));
        if (e == cudaSuccess) e = cudaEventCreateWithFlags(&plan->theta_event, cudaEventDisableTiming);
        if (e == cudaSuccess) {
            plan->comp5120 = std::calloc(1, comp5120_param_bytes());
            if (plan->comp5120 == nullptr) e = cudaErrorMemoryAllocation;
        }
    }
    if (e == cudaSuccess) e = cudaStreamCreateWithFlags(&plan->host_in, cudaStreamNonBlocking);
    if (e == cudaSuccess) e = cudaStreamCreateWithFlags(&plan->host_out, cudaStreamNonBlocking);
    for (int i = 0; i < 8 && e == cudaSuccess; ++i) e = cudaEventCreateWithFlags(&plan->host_ev[i], cudaEventDisableTiming);
    if (e == cudaSuccess) e = cudaMalloc(&plan->status_word, 4 * sizeof(int));
    if (e == cudaSuccess) e = cudaMemset(plan->status_word, 0, 4 * sizeof(int));
    if (e == cudaSuccess) plan->form_flag = plan->status_word + 1;
    if (e == cudaSuccess) e = cudaDeviceSynchronize();
    if (e != cudaSuccess) {
        release_plan(plan);
        return cuda_fail(nullptr, e);
    }
    *out = plan;
    return BFQ_OK;
}

int bfq_plan_destroy(bfq_plan* plan) {
    if (plan == nullptr) return BFQ_ERR_NULL;
    DeviceGuard guard(plan->device);
    cudaDeviceSynchronize();
    release_plan(plan);
    return BFQ_OK;
}

int bfq_set_angles(bfq_plan* plan, const float* theta, void* stream) {
    if (plan == nullptr || theta == nullptr) return BFQ_ERR_NULL;
    if ((reinterpret_cast<uintptr_t>(theta) & 3u) != 0) return BFQ_ERR_ALIGN;
    DeviceGuard guard(plan->device);
    if (guard.err != cudaSuccess) return cuda_fail(plan, guard.err);
    cudaError_t e;
    if (plan->img4096 != nullptr) {
        e = fwdq4096_set_angles(plan, theta, static_cast<cudaStream_t>(stream));
    } else if (plan->img8192 != nullptr) {
        e = fwdq8192_set_angles(plan, theta, static_cast<cudaStream_t>(stream));
    } else {
        const int count = plan->log_n * (plan->n / 2);
        k_build_twiddles<<<(count + 255) / 256, 256, 0, static_cast<cudaStream_t>(stream)>>>(theta, count, plan->tw);
        e = cudaGetLastError();
    }
    if (e == cudaSuccess && plan->dense128 != nullptr) e = comp5120d_set_angles(plan, static_cast<cudaStream_t>(stream));
    if (e == cudaSuccess && plan->theta_host != nullptr) {
        e = cudaMemcpyAsync(plan->theta_host, theta, sizeof(float) * plan->log_n * (plan->n / 2), cudaMemcpyDeviceToHost,
                            static_cast<cudaStream_t>(stream));
        if (e == cudaSuccess) e = cudaEventRecord(plan->theta_event, static_cast<cudaStream_t>(stream));
        plan->comp5120_valid = false;
    }
    if (e != cudaSuccess) return cuda_fail(plan, e);
    plan->angles_set = true;
    plan->bwd_tables_valid = false;
    return BFQ_OK;
}

int bfq_forward(bfq_plan* plan, const void* x, bfq_dtype xt, int64_t rows, int64_t ldx, void* y, bfq_dtype yt,
                int64_t ldy, void* stream) {
    if (plan == nullptr) return BFQ_ERR_NULL;
    int rc = check_rows(x, xt, rows, ldx, plan->n);
    if (rc == BFQ_OK) rc = check_rows(y, yt, rows, ldy, plan->n);
    if (rc != BFQ_OK) return rc;
    if (!plan->angles_set) return BFQ_ERR_WORKSPACE;
    if (rows == 0) return BFQ_OK;
    DeviceGuard guard(plan->device);
    if (guard.err != cudaSuccess) return cuda_fail(plan, guard.err);
    if (xt == BFQ_BF16 && yt == BFQ_BF16 && x != y && rows < (int64_t(1) << 31) && !env_flag("BFQ_GENERIC_ONLY") &&
        fwdq4096_available(plan)) {
        cudaError_t e = fwdq4096_launch(plan, x, rows, ldx, false, nullptr, nullptr, y, ldy,
                                        static_cast<cudaStream_t>(stream));
        return e == cudaSuccess ? BFQ_OK : cuda_fail(plan, e);
    }
    if (xt == BFQ_F32 && yt == BFQ_F32 && x != y && rows < (int64_t(1) << 31) && !env_flag("BFQ_GENERIC_ONLY") &&
        fwdq4096_available(plan)) {  // fp32 rows in and out on the tuned kernel
        cudaError_t e = fwdq4096_launch_f32(plan, x, rows, ldx, 0, nullptr, nullptr, y, ldy, static_cast<cudaStream_t>(stream));
        return e == cudaSuccess ? BFQ_OK : cuda_fail(plan, e);
    }
    if (xt == BFQ_F32 && yt == BFQ_F32 && x != y && rows < (int64_t(1) << 31) && !env_flag("BFQ_GENERIC_ONLY") &&
        fwdq8192_available(plan)) {
        cudaError_t e = fwdq8192_launch_f32(plan, x, rows, ldx, 0, nullptr, nullptr, y, ldy, static_cast<cudaStream_t>(stream));
        return e == cudaSuccess ? BFQ_OK : cuda_fail(plan, e);
    }
    if (xt == BFQ_BF16 && yt == BFQ_BF16 && x != y && rows < (int64_t(1) << 31) && !env_flag("BFQ_GENERIC_ONLY") &&
        fwdq8192_available(plan)) {
        cudaError_t e = fwdq8192_launch_bf16(plan, x, rows, ldx, y, ldy, static_cast<cudaStream_t>(stream));
        return e == cudaSuccess ? BFQ_OK : cuda_fail(plan, e);
    }
    GenericParams p{};
    p.tw = plan->tw, p.x = x, p.xt = xt, p.ldx = ldx, p.y = y, p.yt = yt, p.ldy = ldy, p.rows = rows;
    cudaError_t e = launch_generic<kModeForward>(plan, p, static_cast<cudaStream_t>(stream));
    return e == cudaSuccess ? BFQ_OK : cuda_fail(plan, e);
}

static int forward_quant_impl(bfq_plan* plan, const void* x, int xt, int64_t rows, int64_t ldx, int bits,
                              uint8_t* codes, uint16_t* scales, void* y, int yt, void* stream,
                              unsigned long long* hist = nullptr, float* rowstats = nullptr) {
    if (plan == nullptr) return BFQ_ERR_NULL;
    int rc = check_rows(x, xt, rows, ldx, plan->n);
    if (rc != BFQ_OK) return rc;
    if ((codes == nullptr || scales == nullptr) && rows != 0) return BFQ_ERR_NULL;
    if (bits != 2 && bits != 4 && bits != 8) return BFQ_ERR_BITS;
    if (!aligned16(codes) || (reinterpret_cast<uintptr_t>(scales) & 1u) != 0) return BFQ_ERR_ALIGN;
    if (y != nullptr) {
        rc = check_rows(y, yt, rows, plan->n, plan->n);
        if (rc != BFQ_OK) return rc;
    }
    if (!plan->angles_set) return BFQ_ERR_WORKSPACE;
    if (rows == 0) return BFQ_OK;
    DeviceGuard guard(plan->device);
    if (guard.err != cudaSuccess) return cuda_fail(plan, guard.err);
    cudaError_t e;
    if (hist != nullptr) {  // statistics: the histogram starts at zero
        e = cudaMemsetAsync(hist, 0, sizeof(unsigned long long) << bits, static_cast<cudaStream_t>(stream));
        if (e != cudaSuccess) return cuda_fail(plan, e);
        if (xt == BFQ_BF16 && bits == 4 && y == nullptr && rows < (int64_t(1) << 31) && !env_flag("BFQ_GENERIC_ONLY") &&
            fwdq4096_available(plan)) {
            e = fwdq4096_launch_stats(plan, x, rows, ldx, codes, scales, hist, rowstats, static_cast<cudaStream_t>(stream));
            return e == cudaSuccess ? BFQ_OK : cuda_fail(plan, e);
        }
    } else if (xt == BFQ_BF16 && bits == 4 && y == nullptr && rows < (int64_t(1) << 31) && !env_flag("BFQ_GENERIC_ONLY") &&
        fwdq4096_available(plan)) {
        e = fwdq4096_launch(plan, x, rows, ldx, false, codes, scales, nullptr, 0, static_cast<cudaStream_t>(stream));
        return e == cudaSuccess ? BFQ_OK : cuda_fail(plan, e);
    }
    // fp32 rows (activations or weights), codes only: the tuned n = 4096 kernel reads them through its fp32 tensor map
    if (hist == nullptr && xt == BFQ_F32 && y == nullptr && rows < (int64_t(1) << 31) && !env_flag("BFQ_GENERIC_ONLY") &&
        fwdq4096_available(plan)) {
        e = fwdq4096_launch_f32(plan, x, rows, ldx, bits, codes, scales, nullptr, 0, static_cast<cudaStream_t>(stream));
        return e == cudaSuccess ? BFQ_OK : cuda_fail(plan, e);
    }
    if (hist == nullptr && xt == BFQ_F32 && y == nullptr && rows < (int64_t(1) << 31) && !env_flag("BFQ_GENERIC_ONLY") &&
        fwdq8192_available(plan)) {
        e = fwdq8192_launch_f32(plan, x, rows, ldx, bits, codes, scales, nullptr, 0, static_cast<cudaStream_t>(stream));
        return e == cudaSuccess ? BFQ_OK : cuda_fail(plan, e);
    }
    // weight folding that keeps W Q^T in bf16: codes and rows from one pass of the tuned kernels
    if (hist == nullptr && xt == BFQ_BF16 && y != nullptr && yt == BFQ_BF16 && rows < (int64_t(1) << 31) &&
        !env_flag("BFQ_GENERIC_ONLY")) {
        if (fwdq4096_available(plan)) {
            e = fwdq4096_launch_codes_rows(plan, x, rows, ldx, bits, codes, scales, y, plan->n, static_cast<cudaStream_t>(stream));
            return e == cudaSuccess ? BFQ_OK : cuda_fail(plan, e);
        }
        if (fwdq8192_available(plan)) {
            e = fwdq8192_launch_codes_rows(plan, x, rows, ldx, bits, codes, scales, y, plan->n, static_cast<cudaStream_t>(stream));
            return e == cudaSuccess ? BFQ_OK : cuda_fail(plan, e);
        }
    }
    if (hist == nullptr && xt == BFQ_BF16 && (bits == 2 || bits == 8) && y == nullptr && rows < (int64_t(1) << 31) &&
        !env_flag("BFQ_GENERIC_ONLY") && fwdq4096_available(plan)) {
        e = fwdq4096_launch_bits(plan, x, rows, ldx, false, bits, codes, scales, static_cast<cudaStream_t>(stream));
        return e == cudaSuccess ? BFQ_OK : cuda_fail(plan, e);
    }
    if (hist == nullptr && xt == BFQ_BF16 && y == nullptr && rows < (int64_t(1) << 31) &&
        !env_flag("BFQ_GENERIC_ONLY") && fwdq8192_available(plan)) {
        e = fwdq8192_launch(plan, x, rows, ldx, bits, codes, scales, static_cast<cudaStream_t>(stream));
        return e == cudaSuccess ? BFQ_OK : cuda_fail(plan, e);
    }
    GenericParams p{};
    p.tw = plan->tw, p.x = x, p.xt = xt, p.ldx = ldx, p.y = y, p.yt = yt, p.ldy = plan->n;
    p.codes = codes, p.scales = scales, p.bits = bits, p.rows = rows, p.hist = hist, p.rowstats = rowstats;
    e = launch_generic<kModeForwardQuant>(plan, p, static_cast<cudaStream_t>(stream));
    return e == cudaSuccess ? BFQ_OK : cuda_fail(plan, e);
}

int bfq_forward_quant(bfq_plan* plan, const void* x, bfq_dtype xt, int64_t rows, int64_t ldx, int bits,
                      uint8_t* codes, uint16_t* scales_f16, void* stream) {
    return forward_quant_impl(plan, x, xt, rows, ldx, bits, codes, scales_f16, nullptr, BFQ_F32, stream);
}

// ---- rows in host memory ----------------------------------------------------------------------------------
static size_t host_row_bytes(int n, int xt, int bits) {
    return size_t(n) * (xt == BFQ_F32 ? 4 : 2) + size_t(n) * bits / 8 + 2;
}

size_t bfq_forward_quant_host_workspace(const bfq_plan* plan, bfq_dtype xt, int bits, int64_t chunk_rows) {
    if (plan == nullptr || chunk_rows <= 0 || (bits != 2 && bits != 4 && bits != 8)) return 0;
    const int64_t r = (chunk_rows + 7) / 8 * 8;
    return size_t(2) * size_t(r) * host_row_bytes(plan->n, xt, bits);
}

int bfq_forward_quant_host(bfq_plan* plan, const void* x_host, bfq_dtype xt, int64_t rows, int64_t ldx, int bits,
                           uint8_t* codes_host, uint16_t* scales_host_f16, void* workspace, size_t workspace_bytes,
                           void* stream) {
    if (plan == nullptr) return BFQ_ERR_NULL;
    if (xt != BFQ_F32 && xt != BFQ_BF16) return BFQ_ERR_DTYPE;
    if (bits != 2 && bits != 4 && bits != 8) return BFQ_ERR_BITS;
    if (rows < 0 || ldx < plan->n) return BFQ_ERR_STRIDE;
    if (rows == 0) return BFQ_OK;
    if (x_host == nullptr || codes_host == nullptr || scales_host_f16 == nullptr || workspace == nullptr) return BFQ_ERR_NULL;
    if (!aligned16(workspace)) return BFQ_ERR_ALIGN;
    if (!plan->angles_set) return BFQ_ERR_WORKSPACE;
    const int n = plan->n;
    const size_t esz = xt == BFQ_F32 ? 4 : 2, code_row = size_t(n) * bits / 8;
    // two buffers of `chunk` rows each: rows, then codes, then scales (chunk is a multiple of 8: 16-byte aligned parts)
    int64_t chunk = int64_t(workspace_bytes / (2 * host_row_bytes(n, xt, bits))) / 8 * 8;
    if (chunk < 8) return BFQ_ERR_WORKSPACE;
    if (chunk > rows) chunk = (rows + 7) / 8 * 8;
    DeviceGuard guard(plan->device);
    if (guard.err != cudaSuccess) return cuda_fail(plan, guard.err);
    cudaStream_t main = static_cast<cudaStream_t>(stream), s_in = plan->host_in, s_out = plan->host_out;
    uint8_t* base = static_cast<uint8_t*>(workspace);
    const size_t buf_bytes = size_t(chunk) * host_row_bytes(n, xt, bits);
    auto xbuf = [&](int b) { return base + b * buf_bytes; };
    auto cbuf = [&](int b) { return base + b * buf_bytes + size_t(chunk) * n * esz; };
    auto sbuf = [&](int b) { return reinterpret_cast<uint16_t*>(base + b * buf_bytes + size_t(chunk) * (n * esz + code_row)); };
    cudaEvent_t* loaded = plan->host_ev;        // [2] the rows of buffer b have arrived
    cudaEvent_t* consumed = plan->host_ev + 2;  // [2] the kernels have read the rows of buffer b
    cudaEvent_t* computed = plan->host_ev + 4;  // [2] codes and scales of buffer b are written
    cudaEvent_t* drained = plan->host_ev + 6;   // [2] codes and scales of buffer b are back on the host
    cudaError_t e = cudaEventRecord(loaded[0], main);  // the side streams start after the caller's earlier work
    if (e == cudaSuccess) e = cudaStreamWaitEvent(s_in, loaded[0], 0);
    if (e == cudaSuccess) e = cudaStreamWaitEvent(s_out, loaded[0], 0);
    int rc = BFQ_OK;
    const int64_t nchunks = (rows + chunk - 1) / chunk;
    for (int64_t c = 0; c < nchunks && e == cudaSuccess && rc == BFQ_OK; ++c) {
        const int b = int(c & 1);
        const int64_t r0 = c * chunk, r = (rows - r0 < chunk) ? rows - r0 : chunk;
        if (c >= 2) e = cudaStreamWaitEvent(s_in, consumed[b], 0);
        if (e == cudaSuccess)
            e = cudaMemcpy2DAsync(xbuf(b), size_t(n) * esz, static_cast<const uint8_t*>(x_host) + size_t(r0) * ldx * esz,
                                  size_t(ldx) * esz, size_t(n) * esz, size_t(r), cudaMemcpyHostToDevice, s_in);
        if (e == cudaSuccess) e = cudaEventRecord(loaded[b], s_in);
        if (e == cudaSuccess) e = cudaStreamWaitEvent(main, loaded[b], 0);
        if (e == cudaSuccess && c >= 2) e = cudaStreamWaitEvent(main, drained[b], 0);
        if (e != cudaSuccess) break;
        rc = forward_quant_impl(plan, xbuf(b), xt, r, n, bits, cbuf(b), sbuf(b), nullptr, BFQ_F32, main);
        if (rc != BFQ_OK) break;
        e = cudaEventRecord(consumed[b], main);
        if (e == cudaSuccess) e = cudaEventRecord(computed[b], main);
        if (e == cudaSuccess) e = cudaStreamWaitEvent(s_out, computed[b], 0);
        if (e == cudaSuccess)
            e = cudaMemcpyAsync(codes_host + size_t(r0) * code_row, cbuf(b), size_t(r) * code_row, cudaMemcpyDeviceToHost, s_out);
        if (e == cudaSuccess)
            e = cudaMemcpyAsync(scales_host_f16 + r0, sbuf(b), size_t(r) * 2, cudaMemcpyDeviceToHost, s_out);
        if (e == cudaSuccess) e = cudaEventRecord(drained[b], s_out);
    }
    // the caller's stream is done when both side streams are
    if (e == cudaSuccess) e = cudaEventRecord(loaded[0], s_in);
    if (e == cudaSuccess) e = cudaStreamWaitEvent(main, loaded[0], 0);
    if (e == cudaSuccess) e = cudaEventRecord(loaded[1], s_out);
    if (e == cudaSuccess) e = cudaStreamWaitEvent(main, loaded[1], 0);
    if (rc != BFQ_OK) return rc;
    return e == cudaSuccess ? BFQ_OK : cuda_fail(plan, e);
}

int bfq_forward_quant_stats(bfq_plan* plan, const void* x, bfq_dtype xt, int64_t rows, int64_t ldx, int bits,
                            uint8_t* codes, uint16_t* scales_f16, uint64_t* hist, float* rowstats, void* stream) {
    if (hist == nullptr || (rowstats == nullptr && rows != 0)) return BFQ_ERR_NULL;
    if ((reinterpret_cast<uintptr_t>(hist) & 7u) != 0 || (reinterpret_cast<uintptr_t>(rowstats) & 3u) != 0) return BFQ_ERR_ALIGN;
    if (bits != 2 && bits != 4 && bits != 8) return BFQ_ERR_BITS;
    if (rows == 0 && plan != nullptr) {
        DeviceGuard guard(plan->device);
        cudaError_t e = cudaMemsetAsync(hist, 0, sizeof(uint64_t) << bits, static_cast<cudaStream_t>(stream));
        if (e != cudaSuccess) return cuda_fail(plan, e);
    }
    return forward_quant_impl(plan, x, xt, rows, ldx, bits, codes, scales_f16, nullptr, BFQ_F32, stream,
                              reinterpret_cast<unsigned long long*>(hist), rowstats);
}

int bfq_fold_weights(bfq_plan* plan, const void* W, bfq_dtype wt, int64_t m, int64_t ldw, int bits, uint8_t* codes,
                     uint16_t* scales_f16, void* WQt, bfq_dtype ot, void* stream) {
    return forward_quant_impl(plan, W, wt, m, ldw, bits, codes, scales_f16, WQt, ot, stream);
}

int bfq_hadamard(bfq_plan* plan, const void* x, bfq_dtype xt, int64_t rows, int64_t ldx, void* y, bfq_dtype yt,
                 int64_t ldy, void* stream) {
    if (plan == nullptr) return BFQ_ERR_NULL;
    int rc = check_rows(x, xt, rows, ldx, plan->n);
    if (rc == BFQ_OK) rc = check_rows(y, yt, rows, ldy, plan->n);
    if (rc != BFQ_OK) return rc;
    if (rows == 0) return BFQ_OK;
    DeviceGuard guard(plan->device);
    if (guard.err != cudaSuccess) return cuda_fail(plan, guard.err);
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    cudaError_t e;
    if (xt == BFQ_BF16 && yt == BFQ_BF16 && x != y && rows < (int64_t(1) << 31) && !env_flag("BFQ_GENERIC_ONLY") &&
        fwdq4096_available(plan)) {
        e = fwdq4096_launch(plan, x, rows, ldx, true, nullptr, nullptr, y, ldy, st);
    } else if (xt == BFQ_BF16 && yt == BFQ_BF16 && x != y && rows < (int64_t(1) << 31) && !env_flag("BFQ_GENERIC_ONLY") &&
               fwdq8192_available(plan)) {
        e = fwdq8192_launch_hadamard(plan, x, rows, ldx, 0, nullptr, nullptr, y, ldy, st);
    } else {
        GenericParams p{};
        p.tw = plan->tw, p.x = x, p.xt = xt, p.ldx = ldx, p.y = y, p.yt = yt, p.ldy = ldy, p.rows = rows;
        e = launch_generic<kModeHadamard>(plan, p, st);
    }
    return e == cudaSuccess ? BFQ_OK : cuda_fail(plan, e);
}

int bfq_hadamard_quant(bfq_plan* plan, const void* x, bfq_dtype xt, int64_t rows, int64_t ldx, int bits, uint8_t* codes,
                       uint16_t* scales_f16, void* stream) {
    if (plan == nullptr) return BFQ_ERR_NULL;
    int rc = check_rows(x, xt, rows, ldx, plan->n);
    if (rc != BFQ_OK) return rc;
    if ((codes == nullptr || scales_f16 == nullptr) && rows != 0) return BFQ_ERR_NULL;
    if (bits != 2 && bits != 4 && bits != 8) return BFQ_ERR_BITS;
    if (!aligned16(codes) || (reinterpret_cast<uintptr_t>(scales_f16) & 1u) != 0) return BFQ_ERR_ALIGN;
    if (rows == 0) return BFQ_OK;
    DeviceGuard guard(plan->device);
    if (guard.err != cudaSuccess) return cuda_fail(plan, guard.err);
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    cudaError_t e;
    if (xt == BFQ_BF16 && rows < (int64_t(1) << 31) && !env_flag("BFQ_GENERIC_ONLY") && fwdq4096_available(plan)) {
        e = bits == 4 ? fwdq4096_launch(plan, x, rows, ldx, true, codes, scales_f16, nullptr, 0, st)
                      : fwdq4096_launch_bits(plan, x, rows, ldx, true, bits, codes, scales_f16, st);
    } else if (xt == BFQ_BF16 && rows < (int64_t(1) << 31) && !env_flag("BFQ_GENERIC_ONLY") && fwdq8192_available(plan)) {
        e = fwdq8192_launch_hadamard(plan, x, rows, ldx, bits, codes, scales_f16, nullptr, 0, st);
    } else {
        GenericParams p{};
        p.tw = plan->tw, p.x = x, p.xt = xt, p.ldx = ldx, p.y = nullptr, p.yt = BFQ_F32, p.ldy = plan->n;
        p.codes = codes, p.scales = scales_f16, p.bits = bits, p.rows = rows;
        e = launch_generic<kModeHadamardQuant>(plan, p, st);
    }
    return e == cudaSuccess ? BFQ_OK : cuda_fail(plan, e);
}

int bfq_inverse(bfq_plan* plan, const void* y, bfq_dtype yt, int64_t rows, int64_t ldy, void* x, bfq_dtype xt,
                int64_t ldx, void* stream) {
    if (plan == nullptr) return BFQ_ERR_NULL;
    int rc = check_rows(y, yt, rows, ldy, plan->n);
    if (rc == BFQ_OK) rc = check_rows(x, xt, rows, ldx, plan->n);
    if (rc != BFQ_OK) return rc;
    if (!plan->angles_set) return BFQ_ERR_WORKSPACE;
    if (rows == 0) return BFQ_OK;
    DeviceGuard guard(plan->device);
    if (guard.err != cudaSuccess) return cuda_fail(plan, guard.err);
    if (yt == BFQ_F32 && xt == BFQ_F32 && rows < (int64_t(1) << 31) && x != y && !env_flag("BFQ_GENERIC_ONLY") &&
        bwd4096_available(plan)) {  // fp32 rows in and out on the tuned kernel
        cudaStream_t st = static_cast<cudaStream_t>(stream);
        cudaError_t e = cudaSuccess;
        if (!plan->bwd_tables_valid) {
            e = bwd4096_build_tables(plan, st);
            plan->bwd_tables_valid = (e == cudaSuccess);
        }
        if (e == cudaSuccess) e = inv4096_launch_f32(plan, y, rows, ldy, x, ldx, st);
        return e == cudaSuccess ? BFQ_OK : cuda_fail(plan, e);
    }
    if (yt == BFQ_BF16 && rows < (int64_t(1) << 31) && x != y && !env_flag("BFQ_GENERIC_ONLY") && bwd4096_available(plan)) {
        cudaStream_t st = static_cast<cudaStream_t>(stream);
        cudaError_t e = cudaSuccess;
        if (!plan->bwd_tables_valid) {  // shared with bfq_backward: built on first use after bfq_set_angles
            e = bwd4096_build_tables(plan, st);
            plan->bwd_tables_valid = (e == cudaSuccess);
        }
        if (e == cudaSuccess) e = inv4096_launch(plan, y, rows, ldy, x, xt == BFQ_BF16, ldx, st);
        return e == cudaSuccess ? BFQ_OK : cuda_fail(plan, e);
    }
    if (yt == BFQ_BF16 && rows < (int64_t(1) << 31) && x != y && !env_flag("BFQ_GENERIC_ONLY") && bwd8192_available(plan)) {
        cudaStream_t st = static_cast<cudaStream_t>(stream);
        cudaError_t e = cudaSuccess;
        if (!plan->bwd_tables_valid) {
            e = bwd8192_build_tables(plan, st);
            plan->bwd_tables_valid = (e == cudaSuccess);
        }
        if (e == cudaSuccess) e = inv8192_launch(plan, y, rows, ldy, x, xt == BFQ_BF16, ldx, st);
        return e == cudaSuccess ? BFQ_OK : cuda_fail(plan, e);
    }
    GenericParams p{};
    p.tw = plan->tw, p.x = y, p.xt = yt, p.ldx = ldy, p.y = x, p.yt = xt, p.ldy = ldx, p.rows = rows;
    cudaError_t e = launch_generic<kModeInverse>(plan, p, static_cast<cudaStream_t>(stream));
    return e == cudaSuccess ? BFQ_OK : cuda_fail(plan, e);
}

int bfq_backward(bfq_plan* plan, const void* x, bfq_dtype xt, const void* g, bfq_dtype gt, int64_t rows, int64_t ld,
                 void* dx, bfq_dtype dxt, float* dtheta, void* stream) {
    if (plan == nullptr) return BFQ_ERR_NULL;
    int rc = check_rows(x, xt, rows, ld, plan->n);
    if (rc == BFQ_OK) rc = check_rows(g, gt, rows, ld, plan->n);
    if (rc == BFQ_OK && dx != nullptr) rc = check_rows(dx, dxt, rows, ld, plan->n);
    if (rc != BFQ_OK) return rc;
    if (dtheta == nullptr) return BFQ_ERR_NULL;
    if (!aligned16(dtheta)) return BFQ_ERR_ALIGN;
    if (!plan->angles_set) return BFQ_ERR_WORKSPACE;
    DeviceGuard guard(plan->device);
    if (guard.err != cudaSuccess) return cuda_fail(plan, guard.err);
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    if (rows == 0) {
        cudaError_t e = cudaMemsetAsync(dtheta, 0, sizeof(float) * size_t(plan->log_n) * (plan->n / 2), st);
        return e == cudaSuccess ? BFQ_OK : cuda_fail(plan, e);
    }
    if (xt == gt && (dx == nullptr || dxt == xt) && rows < (int64_t(1) << 31) - 1 && !env_flag("BFQ_GENERIC_ONLY") &&
        bwd4096_available(plan)) {  // all rows bf16, or all fp32
        cudaError_t e = cudaSuccess;
        if (!plan->bwd_tables_valid) {  // built on first use after bfq_set_angles, on the caller's stream
            e = bwd4096_build_tables(plan, st);
            plan->bwd_tables_valid = (e == cudaSuccess);
        }
        if (e == cudaSuccess) e = bwd4096_launch(plan, x, g, rows, ld, dx, dtheta, xt == BFQ_F32, st);
        return e == cudaSuccess ? BFQ_OK : cuda_fail(plan, e);
    }
    if (xt == BFQ_BF16 && gt == BFQ_BF16 && (dx == nullptr || dxt == BFQ_BF16) && rows < (int64_t(1) << 31) - 1 &&
        !env_flag("BFQ_GENERIC_ONLY") && bwd8192_available(plan)) {
        // n = 8192: the n = 4096 backward kernel on both halves of the elements, the last stage folded into its read of g
        cudaError_t e = cudaSuccess;
        if (!plan->bwd_tables_valid) {
            e = bwd8192_build_tables(plan, st);
            plan->bwd_tables_valid = (e == cudaSuccess);
        }
        if (e == cudaSuccess) e = bwd8192_launch_halves(plan, x, g, rows, ld, dx, dtheta, st);
        return e == cudaSuccess ? BFQ_OK : cuda_fail(plan, e);
    }
    BackwardParams p{};
    p.tw = plan->tw, p.x = x, p.xt = xt, p.g = g, p.gt = gt, p.ld = ld, p.dx = dx, p.dxt = dxt, p.rows = rows;
    cudaError_t e = launch_backward(plan, p, dtheta, st);
    return e == cudaSuccess ? BFQ_OK : cuda_fail(plan, e);
}

int bfq_cayley(bfq_plan* plan, const float* params, int n1, float* q1, void* stream) {
    if (plan == nullptr || params == nullptr || q1 == nullptr) return BFQ_ERR_NULL;
    if (n1 < 2 || n1 > BFQ_MAX_N1) return BFQ_ERR_UNSUPPORTED_N;
    if ((reinterpret_cast<uintptr_t>(params) & 3u) != 0 || (reinterpret_cast<uintptr_t>(q1) & 3u) != 0) return BFQ_ERR_ALIGN;
    DeviceGuard guard(plan->device);
    if (guard.err != cudaSuccess) return cuda_fail(plan, guard.err);
    cudaError_t e = cayley_launch(params, n1, q1, static_cast<cudaStream_t>(stream));
    return e == cudaSuccess ? BFQ_OK : cuda_fail(plan, e);
}

static int composite_impl(bfq_plan* plan, const float* q1, int n1, const void* x, int xt, int64_t rows, int64_t ldx,
                          void* y, int yt, int64_t ldy, int bits, uint8_t* codes, uint16_t* scales, void* stream,
                          bool inverse = false) {
    if (plan == nullptr || q1 == nullptr) return BFQ_ERR_NULL;
    if (n1 < 2 || n1 > BFQ_MAX_N1 || plan->n > 1024 || int64_t(n1) * plan->n > BFQ_COMPOSITE_MAX_D)
        return BFQ_ERR_UNSUPPORTED_N;
    const int d = n1 * plan->n;
    int rc = check_rows(x, xt, rows, ldx, d);
    if (rc != BFQ_OK) return rc;
    if ((reinterpret_cast<uintptr_t>(q1) & 3u) != 0) return BFQ_ERR_ALIGN;
    if (codes != nullptr || y == nullptr) {  // the quantizing entry point
        if ((codes == nullptr || scales == nullptr) && rows != 0) return BFQ_ERR_NULL;
        if (bits != 2 && bits != 4 && bits != 8) return BFQ_ERR_BITS;
        if (!aligned16(codes) || (reinterpret_cast<uintptr_t>(scales) & 1u) != 0) return BFQ_ERR_ALIGN;
    } else {
        rc = check_rows(y, yt, rows, ldy, d);
        if (rc != BFQ_OK) return rc;
    }
    if (!plan->angles_set) return BFQ_ERR_WORKSPACE;
    if (rows == 0) return BFQ_OK;
    DeviceGuard guard(plan->device);
    if (guard.err != cudaSuccess) return cuda_fail(plan, guard.err);
    cudaError_t e;
    if (n1 == 40 && xt == BFQ_BF16 && rows < (int64_t(1) << 31) && (y == nullptr || yt == BFQ_BF16) &&
        !env_flag("BFQ_GENERIC_ONLY")) {
        // default: both factors on the tensor cores (INT4 or INT8 codes, or bf16 rows); BFQ_COMPOSITE_FP32_BUTTERFLY=1
        // keeps Q2 as an fp32 butterfly on the CUDA cores (only the dense factor on the tensor cores; INT4 or bf16 rows)
        const bool dense_ok = codes == nullptr || bits == 4 || bits == 8, bfly_ok = codes == nullptr || bits == 4;
        if (dense_ok && (inverse || !bfly_ok || !env_flag("BFQ_COMPOSITE_FP32_BUTTERFLY")) && comp5120d_available(plan)) {
            e = comp5120d_launch(plan, q1, x, rows, ldx, bits, codes, scales, y, ldy, inverse, static_cast<cudaStream_t>(stream));
            return e == cudaSuccess ? BFQ_OK : cuda_fail(plan, e);
        }
        if (!inverse && bfly_ok && comp5120_available(plan)) {
            e = comp5120_launch(plan, q1, x, rows, ldx, codes, scales, y, ldy, static_cast<cudaStream_t>(stream));
            return e == cudaSuccess ? BFQ_OK : cuda_fail(plan, e);
        }
    }
    e = composite_generic_launch(plan, q1, n1, x, xt, rows, ldx, y, yt, ldy, bits, codes, scales, inverse,
                                 static_cast<cudaStream_t>(stream));
    return e == cudaSuccess ? BFQ_OK : cuda_fail(plan, e);
}

int bfq_composite_forward(bfq_plan* plan, const float* q1, int n1, const void* x, bfq_dtype xt, int64_t rows,
                          int64_t ldx, void* y, bfq_dtype yt, int64_t ldy, void* stream) {
    if (y == nullptr && rows != 0) return BFQ_ERR_NULL;
    return composite_impl(plan, q1, n1, x, xt, rows, ldx, y, yt, ldy, 4, nullptr, nullptr, stream);
}

int bfq_composite_inverse(bfq_plan* plan, const float* q1, int n1, const void* y, bfq_dtype yt, int64_t rows, int64_t ldy,
                          void* x, bfq_dtype xt, int64_t ldx, void* stream) {
    if (x == nullptr && rows != 0) return BFQ_ERR_NULL;
    return composite_impl(plan, q1, n1, y, yt, rows, ldy, x, xt, ldx, 4, nullptr, nullptr, stream, true);
}

int bfq_composite_forward_quant(bfq_plan* plan, const float* q1, int n1, const void* x, bfq_dtype xt, int64_t rows,
                                int64_t ldx, int bits, uint8_t* codes, uint16_t* scales_f16, void* stream) {
    return composite_impl(plan, q1, n1, x, xt, rows, ldx, nullptr, BFQ_F32, 0, bits, codes, scales_f16, stream);
}

int bfq_device_status(bfq_plan* plan) {
    if (plan == nullptr) return BFQ_ERR_NULL;
    DeviceGuard guard(plan->device);
    if (guard.err != cudaSuccess) return cuda_fail(plan, guard.err);
    cudaError_t e = cudaDeviceSynchronize();
    if (e != cudaSuccess) return cuda_fail(plan, e);
    int word = 0;
    e = cudaMemcpy(&word, plan->status_word, sizeof(int), cudaMemcpyDeviceToHost);
    if (e != cudaSuccess) return cuda_fail(plan, e);
    if (word != 0) {
        cudaMemset(plan->status_word, 0, sizeof(int));
        return BFQ_ERR_DEVICE_TIMEOUT;
    }
    return BFQ_OK;
}

int bfq_last_cuda_error(const bfq_plan* plan) { return plan == nullptr ? 0 : plan->last_cuda_error; }

int bfq_test_stuck_wait(bfq_plan* plan, int enable) {
    if (plan == nullptr) return BFQ_ERR_NULL;
    plan->test_stuck_wait = enable != 0;
    return BFQ_OK;
}

int bfq_stage_form(bfq_plan* plan) {
    if (plan == nullptr) return BFQ_ERR_NULL;
    if (plan->form_flag == nullptr || !plan->angles_set) return BFQ_ERR_WORKSPACE;
    DeviceGuard guard(plan->device);
    if (guard.err != cudaSuccess) return cuda_fail(plan, guard.err);
    cudaError_t e = cudaDeviceSynchronize();
    int words[3] = {0, 0, 0};  // forward; inverse (n = 4096, or the lower half at n = 8192); inverse, upper half at n = 8192
    if (e == cudaSuccess) e = cudaMemcpy(words, plan->form_flag, sizeof(words), cudaMemcpyDeviceToHost);
    if (e != cudaSuccess) return cuda_fail(plan, e);
    return (words[0] != 0 ? 1 : 0) | ((words[1] | words[2]) != 0 ? 2 : 0);
}

int bfq_backward_partials(const bfq_plan* plan) { return plan == nullptr ? 0 : plan->last_backward_partials; }

const char* bfq_status_string(int status) {
    switch (status) {
        case BFQ_OK: return "ok";
        case BFQ_ERR_NULL: return "null pointer";
        case BFQ_ERR_UNSUPPORTED_N: return "unsupported n (power of two in [16, 8192] required)";
        case BFQ_ERR_BITS: return "bits must be 2, 4 or 8";
        case BFQ_ERR_ALIGN: return "pointer not 16-byte aligned";
        case BFQ_ERR_STRIDE: return "bad rows / leading dimension";
        case BFQ_ERR_DTYPE: return "dtype must be BFQ_F32 or BFQ_BF16";
        case BFQ_ERR_WORKSPACE: return "angles not set or workspace too small";
        case BFQ_ERR_CUDA: return "CUDA runtime error";
        case BFQ_ERR_DEVICE_TIMEOUT: return "bounded device-side wait gave up";
        case BFQ_ERR_TOO_LARGE: return "row length exceeds the fixed scratch of the no-allocation entry point";
        default: return "unknown status";
    }
}

}  // extern "C"
