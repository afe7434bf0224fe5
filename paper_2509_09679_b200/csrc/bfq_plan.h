// Internal layout of a plan (opaque to callers of the C ABI).
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

namespace bfq {
constexpr int kMaxDevices = 64;
constexpr int kBackwardCtasPerSm = 2;  // upper bound on resident backward CTAs per SM (sizes the partial sums)
}  // namespace bfq

struct bfq_plan {
    int n = 0;
    int log_n = 0;
    int device = 0;
    int sm_count = 0;
    int cc_major = 0;
    bool angles_set = false;
    float2* tw = nullptr;        // [log_n][n/2] (cos, sin), fp32
    float* img4096 = nullptr;    // [128][416] tensor-memory image of the rotation constants (n = 4096 only)
    void* prep4096 = nullptr;    // staging for the image build: per-angle constants and negation flags (n = 4096 only)
    float* img_b4096 = nullptr;  // [128][384] constants of the backward kernel (n = 4096 only)
    float* img_i4096 = nullptr;  // [104][128][4] scaled-form constants of the inverse kernel (n = 4096 only)
    int8_t* dsign4096 = nullptr; // [12][2048] sign applied to the accumulated d-theta (n = 4096 only)
    uint32_t* gsign4096 = nullptr;  // [16 * 128] sign words applied to bf16 g rows (n = 4096 only)
    bool bwd_tables_valid = false;  // the three above match the current angles
    // n = 8192: backward tables of the two 4096-element halves (stages 0 .. 11), built on first use like the above
    float* img_b8192[2] = {nullptr, nullptr};
    float* img_i8192[2] = {nullptr, nullptr};  // scaled-form constants of the inverse kernel, per half
    int8_t* dsign8192[2] = {nullptr, nullptr};
    uint32_t* gsign8192[2] = {nullptr, nullptr};
    void* prep_half8192 = nullptr;  // staging of one half: three-shear constants and negation flags
    float* img8192 = nullptr;    // [2][128][448] constants of the n = 8192 forward kernel, one image per CTA rank
    void* prep8192 = nullptr;    // staging for that image build
    float* theta_host = nullptr;    // pinned host copy of the angles (n = 128 only: the composite kernel's constants
                                    // are kernel parameters computed on the host)
    cudaEvent_t theta_event = nullptr;  // recorded after that copy
    void* dense128 = nullptr;       // device: Q2 as a dense 128 x 128 block, two bf16 terms, in the MMA operand layout
                                    // (n = 128 only)
    void* comp5120 = nullptr;       // host: kernel parameters of the 40 x 128 composite kernel
    bool comp5120_valid = false;    // they match the current angles
    float* partial = nullptr;    // [partial_slots][log_n][n/2] d-theta partial sums
    int64_t partial_slots = 0;
    size_t partial_floats = 0;   // floats allocated behind `partial` (at n = 8192 the tuned backward may need more than the above)
    int* status_word = nullptr;  // device: non-zero when a bounded wait gave up
    int* form_flag = nullptr;    // device (status_word + 1): stage form the table build selected for the tuned kernels
    // bfq_forward_quant_host: copy-in and copy-out streams and the events that order them with the caller's stream
    cudaStream_t host_in = nullptr, host_out = nullptr;
    cudaEvent_t host_ev[8] = {nullptr, nullptr, nullptr, nullptr, nullptr, nullptr, nullptr, nullptr};
    bool test_stuck_wait = false;  // bfq_test_stuck_wait: the n = 4096 forward kernel announces bytes that never arrive
    int last_cuda_error = 0;
    int last_backward_partials = 0;
};
