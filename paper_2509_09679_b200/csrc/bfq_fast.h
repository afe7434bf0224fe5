// Entry points of the tuned kernels (host side), called by the C-ABI layer.
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

#include "bfq_plan.h"

namespace bfq {

// n = 4096, bf16 rows, INT4: tensor-memory-resident rotation constants
bool fwdq4096_available(const bfq_plan* plan);
size_t fwdq4096_image_bytes();
size_t fwdq4096_prep_bytes();
// builds the plan's (cos, sin) table and the tensor-memory image from the angles
cudaError_t fwdq4096_set_angles(const bfq_plan* plan, const float* theta, cudaStream_t st);
cudaError_t fwdq4096_launch(const bfq_plan* plan, const void* x, int64_t rows, int64_t ldx, bool hadamard,
                            uint8_t* codes, uint16_t* scales, void* y_bf16, int64_t ldy, cudaStream_t st);

// INT2 / INT8 codes from the same kernel (bits = 2 or 8)
cudaError_t fwdq4096_launch_bits(const bfq_plan* plan, const void* x, int64_t rows, int64_t ldx, bool hadamard, int bits,
                                 uint8_t* codes, uint16_t* scales, cudaStream_t st);
// codes + scales (bits = 2, 4, 8) and the rotated rows in bf16 from one pass
cudaError_t fwdq4096_launch_codes_rows(const bfq_plan* plan, const void* x, int64_t rows, int64_t ldx, int bits,
                                       uint8_t* codes, uint16_t* scales, void* y_bf16, int64_t ldy, cudaStream_t st);
// fp32 rows in: codes + scales (bits = 2, 4, 8) or, with bits = 0, the rotated rows in fp32
cudaError_t fwdq4096_launch_f32(const bfq_plan* plan, const void* x, int64_t rows, int64_t ldx, int bits, uint8_t* codes,
                                uint16_t* scales, void* y_f32, int64_t ldy, cudaStream_t st);
// the same with the statistics of bfq_forward_quant_stats (hist already zeroed on `st`)
cudaError_t fwdq4096_launch_stats(const bfq_plan* plan, const void* x, int64_t rows, int64_t ldx, uint8_t* codes,
                                  uint16_t* scales, unsigned long long* hist, float* rowstats, cudaStream_t st);

// n = 8192, bf16 rows, INT2 (INT4 / INT8 through another epilogue): two-CTA clusters, one 4096-point half per CTA
size_t fwdq8192_image_bytes();
size_t fwdq8192_prep_bytes();
bool fwdq8192_available(const bfq_plan* plan);
cudaError_t fwdq8192_set_angles(const bfq_plan* plan, const float* theta, cudaStream_t st);
cudaError_t fwdq8192_launch(const bfq_plan* plan, const void* x, int64_t rows, int64_t ldx, int bits, uint8_t* codes,
                            uint16_t* scales, cudaStream_t st);
cudaError_t fwdq8192_launch_codes_rows(const bfq_plan* plan, const void* x, int64_t rows, int64_t ldx, int bits,
                                       uint8_t* codes, uint16_t* scales, void* y_bf16, int64_t ldy, cudaStream_t st);
cudaError_t fwdq8192_launch_f32(const bfq_plan* plan, const void* x, int64_t rows, int64_t ldx, int bits, uint8_t* codes,
                                uint16_t* scales, void* y_f32, int64_t ldy, cudaStream_t st);
cudaError_t fwdq8192_launch_hadamard(const bfq_plan* plan, const void* x, int64_t rows, int64_t ldx, int bits, uint8_t* codes,
                                     uint16_t* scales, void* y_bf16, int64_t ldy, cudaStream_t st);
cudaError_t fwdq8192_launch_bf16(const bfq_plan* plan, const void* x, int64_t rows, int64_t ldx, void* y, int64_t ldy,
                                 cudaStream_t st);

// n = 4096, bf16 x / g / dx: backward with tensor-memory constants and accumulators
size_t bwd4096_image_bytes();
size_t inv4096_image_bytes();
size_t bwd4096_dsign_bytes();
size_t bwd4096_gsign_bytes();
bool bwd4096_available(const bfq_plan* plan);
// n = 8192 bf16 rows: the n = 4096 backward kernel on the two halves of the elements (one launch, even CTAs on the lower half, odd CTAs on the upper); the
// stage that joins the halves is folded into the read of g and its sums are taken there too
size_t bwd8192_prep_bytes();
size_t bwd8192_partial_floats(int sm_count);
bool bwd8192_available(const bfq_plan* plan);
cudaError_t bwd8192_build_tables(const bfq_plan* plan, cudaStream_t st);
cudaError_t inv8192_launch(bfq_plan* plan, const void* y, int64_t rows, int64_t ldy, void* x, bool x_bf16, int64_t ldx,
                           cudaStream_t st);
cudaError_t bwd8192_launch_halves(bfq_plan* plan, const void* x, const void* g, int64_t rows, int64_t ld, void* dx,
                                  float* dtheta, cudaStream_t st);
cudaError_t bwd4096_build_tables(const bfq_plan* plan, cudaStream_t st);
cudaError_t bwd4096_launch(bfq_plan* plan, const void* x, const void* g, int64_t rows, int64_t ld, void* dx,
                           float* dtheta, bool f32, cudaStream_t st);

// n = 4096, bf16 y -> bf16 / fp32 x: inverse (uses the backward tables)
cudaError_t inv4096_launch_f32(bfq_plan* plan, const void* y, int64_t rows, int64_t ldy, void* x, int64_t ldx,
                               cudaStream_t st);
cudaError_t inv4096_launch(bfq_plan* plan, const void* y, int64_t rows, int64_t ldy, void* x, bool x_bf16, int64_t ldx,
                           cudaStream_t st);

// composite transform Q1 (x) Q2 (n1 <= 64, n2 = the plan's n): Cayley solve and the kernels for every shape
cudaError_t cayley_launch(const float* params, int n1, float* q1, cudaStream_t st);
cudaError_t composite_generic_launch(const bfq_plan* plan, const float* q1, int n1, const void* x, int xt, int64_t rows,
                                     int64_t ldx, void* y, int yt, int64_t ldy, int bits, uint8_t* codes,
                                     uint16_t* scales, bool inverse, cudaStream_t st);


// composite 40 x 128 on bf16 rows: butterfly with kernel-parameter constants + tcgen05 TF32 dense factor
bool comp5120_available(const bfq_plan* plan);
size_t comp5120_param_bytes();
cudaError_t comp5120_launch(bfq_plan* plan, const float* q1, const void* x, int64_t rows, int64_t ldx, uint8_t* codes,
                            uint16_t* scales, void* y_bf16, int64_t ldy, cudaStream_t st);


// composite 40 x 128 on bf16 rows with both factors on the tensor cores (Q2 merged into a dense 128 x 128 block)
size_t comp5120d_image_bytes();
bool comp5120d_available(const bfq_plan* plan);
cudaError_t comp5120d_set_angles(const bfq_plan* plan, cudaStream_t st);
cudaError_t comp5120d_launch(bfq_plan* plan, const float* q1, const void* x, int64_t rows, int64_t ldx, int bits,
                             uint8_t* codes, uint16_t* scales, void* y_bf16, int64_t ldy, bool inverse, cudaStream_t st);

}  // namespace bfq
