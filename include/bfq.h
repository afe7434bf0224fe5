/*
 * bfq — butterfly rotation + low-bit quantization for NVIDIA B200 (sm_100a).  C ABI.
 *
 * The library computes, on one GPU, the data-parallel hot path of ButterflyQuant:
 *
 *   Q = B_L ... B_2 B_1,  L = log2 n,  B_i = n/2 Givens rotations G(theta_{i,j}) on index
 *   pairs at stride 2^{i-1}  (paper Sec. 3.2.1 "Structure and Parameterization"; the
 *   appendix example for n = 8 prints B_1, B_2, B_3 entry by entry).
 *
 * Conventions used by every entry point
 *   stage s = i - 1 = 0..L-1, stride h = 2^s; theta is stage-major [L][n/2] fp32;
 *   pair j of stage s (pairs listed by increasing low index) couples
 *       lo = ((j >> s) << (s+1)) | (j & (h-1)),   hi = lo + h
 *   and maps (a, b) = (z[lo], z[hi]) to (cos*a - sin*b, sin*a + cos*b).
 *   y = Q x applies stage 0 (stride 1) first.  There is no input or output permutation.
 *
 * Memory: every data pointer below is a DEVICE pointer owned by the caller, 16-byte
 * aligned; rows are contiguous, row-major, with a leading dimension in elements
 * (ld >= n, ld * sizeof(element) a multiple of 16).  `stream` is a cudaStream_t passed as
 * void* (NULL = the legacy default stream).  Calls validate their arguments on the host,
 * enqueue work on `stream` and return without synchronising (bfq_plan_create,
 * bfq_plan_destroy and bfq_device_status synchronise).  No compute call allocates memory.
 * The plan owns the twiddle tables, the per-CTA d-theta partial sums and a device status
 * word.  A plan may be used from one host thread at a time; calls on one plan must be
 * issued to streams that serialise them (they share the plan's workspace).
 *
 * Errors: every function returns a bfq_status (0 = OK, negative = error); nothing throws.
 * rows == 0 is a successful no-op.
 */
#ifndef BFQ_H_
#define BFQ_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct bfq_plan bfq_plan; /* opaque */

typedef enum { BFQ_F32 = 0, BFQ_BF16 = 1 } bfq_dtype;

typedef enum {
    BFQ_OK = 0,
    BFQ_ERR_NULL = -1,           /* a required pointer is NULL */
    BFQ_ERR_UNSUPPORTED_N = -2,  /* n is not a power of two in [BFQ_MIN_N, BFQ_MAX_N] */
    BFQ_ERR_BITS = -3,           /* bits not in {2, 4, 8} */
    BFQ_ERR_ALIGN = -4,          /* a pointer is not 16-byte aligned */
    BFQ_ERR_STRIDE = -5,         /* ld < n, or ld * element size not a multiple of 16, or rows < 0 */
    BFQ_ERR_DTYPE = -6,          /* dtype not BFQ_F32 / BFQ_BF16 */
    BFQ_ERR_WORKSPACE = -7,      /* angles not set yet, or plan workspace too small */
    BFQ_ERR_CUDA = -8,           /* a CUDA runtime call failed; see bfq_last_cuda_error */
    BFQ_ERR_DEVICE_TIMEOUT = -9, /* a bounded device-side wait gave up (reported by bfq_device_status) */
    BFQ_ERR_TOO_LARGE = -10      /* bfq_backward_noalloc: n exceeds BFQ_NOALLOC_MAX_N */
} bfq_status;

#define BFQ_MIN_N 16
#define BFQ_MAX_N 8192
#define BFQ_NOALLOC_MAX_N 1024 /* largest row length bfq_backward_noalloc accepts */
#define BFQ_MAX_N1 64          /* largest dense factor of the composite transform */
#define BFQ_COMPOSITE_MAX_D 16384 /* largest composite row length n1 * n2 */

/*
 * Create a plan for row length n on CUDA device `device` (allocates: twiddle tables,
 * d-theta partial sums, a status word).  max_rows is a sizing hint (>= 0, may be 0); no call
 * is limited by it.  Paper: theta is the only learnable state, n log2 n / 2 angles
 * (Sec. 3.2.1, "Parameters").
 */
int bfq_plan_create(bfq_plan** out, int n, int64_t max_rows, int device);
int bfq_plan_destroy(bfq_plan* plan);

/*
 * Load the angles: builds the per-stage twiddle tables (cos theta, sin theta) in fp32 on the
 * device (paper "Inference Efficiency": pre-computed twiddle factors in a lookup table of
 * n log2 n / 2 entries).  theta: device, fp32, [log2 n][n/2], stage 0 = stride 1.
 * Enqueued on `stream`; later calls on the same stream see the new tables.
 */
int bfq_set_angles(bfq_plan* plan, const float* theta, void* stream);

/*
 * y = Q x for every row (Sec. 3.2.1: B = prod B_i; stage order as stated at the top).
 * x: [rows][ldx] of xt; y: [rows][ldy] of yt; fp32 arithmetic.  x and y may be the same buffer
 * only if xt == yt and ldx == ldy.
 */
int bfq_forward(bfq_plan* plan, const void* x, bfq_dtype xt, int64_t rows, int64_t ldx,
                void* y, bfq_dtype yt, int64_t ldy, void* stream);

/*
 * y = Q x fused with the per-row (per-token) symmetric quantizer of Sec. 3.4:
 *     qmax = 2^(bits-1) - 1;  s = max_k |y_k| / qmax, stored as IEEE fp16 (round to nearest
 *     even, saturating at 65504);  code_k = clip(round(y_k / s), -2^(bits-1), qmax),
 *     round-half-to-even, using the fp16-rounded s.  A row whose fp16 scale is 0 gets codes 0.
 * codes: [rows][n*bits/8] bytes, two's complement; element k sits in bits
 *     [bits*(k mod 8/bits), +bits) of byte k*bits/8 (INT4: even element = low nibble).
 * scales_f16: [rows] fp16 bit patterns.  Dequant(q) = s * q.
 */
int bfq_forward_quant(bfq_plan* plan, const void* x, bfq_dtype xt, int64_t rows, int64_t ldx,
                      int bits, uint8_t* codes, uint16_t* scales_f16, void* stream);

/*
 * bfq_forward_quant plus two cheap reductions over the rotated rows y = Q x:
 *   hist     [2^bits] uint64, overwritten: how often each code occurs over all rows, index = code + 2^(bits-1).
 *            P_bins = hist / (rows * n) is the distribution whose divergence from uniform is the paper's
 *            uniformity regulariser L_uniform = D_KL(P_bins || U) (Sec. 3.4); the caller forms the value.
 *   rowstats [rows][2] fp32: sum_k y_k^2 and sum_k y_k^4 of each row (kurtosis n * s4 / s2^2, sigma^2 = s2 / n,
 *            max|y| / sigma with the row's scale: the diagnostics of the paper's kurtosis / outlier tables).
 * Counts are exact for the codes written; the sums are taken in a fixed order (bit-reproducible).
 */
int bfq_forward_quant_stats(bfq_plan* plan, const void* x, bfq_dtype xt, int64_t rows, int64_t ldx, int bits,
                            uint8_t* codes, uint16_t* scales_f16, uint64_t* hist, float* rowstats, void* stream);

/*
 * The fixed rotation the paper compares the learned butterfly with (Sec. 3.1.1, Hadamard transform; QuaRot's
 * x' = H x): y = H_n x per row, H_1 = [1], H_2n = 1/sqrt(2) [[H_n, H_n], [H_n, -H_n]].  Needs no angles
 * (bfq_set_angles may or may not have been called).  With all theta = pi/4 the butterfly is H_n diag((-1)^popcount(j)).
 * bfq_hadamard_quant fuses the same per-row quantizer as bfq_forward_quant.  Together with bfq_forward
 * (unquantized rows, the weight-only "W2A16" setting of the paper's main table) these two let one machine
 * measure what the learned rotation costs over the fixed one ("Inference Efficiency" / FLOP-comparison table).
 */
int bfq_hadamard(bfq_plan* plan, const void* x, bfq_dtype xt, int64_t rows, int64_t ldx, void* y, bfq_dtype yt,
                 int64_t ldy, void* stream);
int bfq_hadamard_quant(bfq_plan* plan, const void* x, bfq_dtype xt, int64_t rows, int64_t ldx, int bits,
                       uint8_t* codes, uint16_t* scales_f16, void* stream);

/*
 * x = Q^T y (= Q^{-1} y: Q is orthogonal by construction, Sec. 3.2.1): stages L-1..0, each
 * pair mapped by G(theta)^T.  Also dL/dx = Q^T g.
 */
int bfq_inverse(bfq_plan* plan, const void* y, bfq_dtype yt, int64_t rows, int64_t ldy,
                void* x, bfq_dtype xt, int64_t ldx, void* stream);

/*
 * Backward of y = Q x for an upstream gradient g = dL/dy (Sec. 3.5.1, dG/dtheta):
 *     dx = Q^T g  per row;   dtheta[s][j] = sum over rows of  gbar^T (dG/dtheta) z  on pair j of
 *     stage s, z the stage input and gbar the gradient at the stage output.
 * x, g: [rows][ld]; dx: [rows][ld] of dxt (may be NULL to skip); dtheta: device fp32
 * [log2 n][n/2], overwritten.  The sum over rows has a fixed order (per-CTA partial sums over a
 * static row assignment, then the CTAs' sums added in a fixed order): results are bit-identical run to run on the
 * same device.  The quantizer is not differentiated here; g is the caller's.
 */
int bfq_backward(bfq_plan* plan, const void* x, bfq_dtype xt, const void* g, bfq_dtype gt,
                 int64_t rows, int64_t ld, void* dx, bfq_dtype dxt, float* dtheta, void* stream);

/*
 * Weight folding W' = W Q^T (Sec. 3.1, computational invariance y = W x = (W Q^T)(Q x)):
 * row i of W Q^T is (Q w_i)^T, so Q is applied to each of the m rows of W, followed by
 * per-row (per-output-channel) quantization exactly as in bfq_forward_quant.
 * WQt (optional, may be NULL): the unquantized rotated rows, [m][n] of type ot, ld = n.
 */
int bfq_fold_weights(bfq_plan* plan, const void* W, bfq_dtype wt, int64_t m, int64_t ldw,
                     int bits, uint8_t* codes, uint16_t* scales_f16, void* WQt, bfq_dtype ot,
                     void* stream);

/*
 * Composite transform for row lengths d that are not a power of two (Sec. 3.3, Kronecker product construction):
 * d = n1 * n2, Q = Q1 (x) Q2, with Q2 the plan's butterfly (n2 = the plan's n, angles from bfq_set_angles) and Q1 a
 * dense orthogonal n1 x n1 factor.  With a row read as an n1 x n2 matrix X (row r = elements [r n2, (r+1) n2)),
 *     Y = Q1 (X Q2^T):  y[i n2 + j] = sum_k Q1[i][k] (Q2 x_k)[j],  x_k the k-th run of n2 elements.
 * The paper's example: d = 5120 = 40 x 128, 780 Cayley parameters + 448 angles.
 *
 * bfq_cayley builds Q1 = (I - A)(I + A)^{-1} ("Concrete Example for d = 5120"): params = the n1 (n1 - 1) / 2 entries of
 * the strict upper triangle of the skew-symmetric A, row by row (device, fp32); q1 = device fp32 [n1][n1] row-major,
 * written.  Solved in float64 on the device.  2 <= n1 <= BFQ_MAX_N1.  The plan only names the device.
 *
 * bfq_composite_forward / _quant: x: [rows][ldx] of xt with ldx >= d; y: [rows][ldy]; codes: [rows][d*bits/8] and one
 * fp16 scale per row over all d elements (the quantizer of bfq_forward_quant).  q1 is read as given: any n1 x n1
 * matrix works, the caller keeps it orthogonal.  Needs 16 <= n2 <= 1024 and d <= BFQ_COMPOSITE_MAX_D, else
 * BFQ_ERR_UNSUPPORTED_N.  For n1 = 40, n2 = 128 and bf16 rows (INT4 / INT8 codes or bf16 rows out) both factors run on the
 * tensor cores: Q2 merged into a dense 128 x 128 block held as two bf16 terms, Q1 in TF32 (10 mantissa bits) applied to
 * the fp32 intermediate read as TF32, fp32 accumulation: |error| <= 2^-9 sum_k |Q1[i][k]| |(Q2 x_k)[j]| there.  With the
 * environment variable BFQ_COMPOSITE_FP32_BUTTERFLY=1 Q2 stays an fp32 butterfly on the CUDA cores and only Q1 uses the
 * tensor cores (TF32, |error| <= 2^-10 of the same sum); in that mode the first call after bfq_set_angles waits on the
 * host for a copy of the angles (the rotation constants become kernel parameters), so it must not be made during stream
 * capture.  fp32 arithmetic everywhere else.  x and y must not overlap.
 */
int bfq_cayley(bfq_plan* plan, const float* params, int n1, float* q1, void* stream);
int bfq_composite_forward(bfq_plan* plan, const float* q1, int n1, const void* x, bfq_dtype xt, int64_t rows,
                          int64_t ldx, void* y, bfq_dtype yt, int64_t ldy, void* stream);
int bfq_composite_forward_quant(bfq_plan* plan, const float* q1, int n1, const void* x, bfq_dtype xt, int64_t rows,
                                int64_t ldx, int bits, uint8_t* codes, uint16_t* scales_f16, void* stream);
/* x = (Q1 (x) Q2)^T y per row, the inverse of bfq_composite_forward (both factors are orthogonal, Sec. 3.3, "Proof of
 * orthogonality"): X = (Q1^T Y) Q2, i.e. Q1^T across the runs and the inverse butterfly on every run.  Also dL/dx of the
 * composite for an upstream gradient y.  Same shapes, limits and arithmetic as bfq_composite_forward (for n1 = 40,
 * n2 = 128, bf16 in and out: both factors on the tensor cores). */
int bfq_composite_inverse(bfq_plan* plan, const float* q1, int n1, const void* y, bfq_dtype yt, int64_t rows, int64_t ldy,
                          void* x, bfq_dtype xt, int64_t ldx, void* stream);

/*
 * bfq_backward without any device-memory allocation.  (No counterpart in the paper: this exists for
 * the library's hosts, not for the method.)
 *
 * For callers that must not allocate on the GPU -- a process whose device memory belongs entirely to
 * a framework's caching allocator, or a latency-critical loop that cannot take the device-wide
 * synchronisation of cudaMalloc / cudaFree -- and therefore cannot create a plan.  Same result as
 * bfq_set_angles + bfq_backward (d-theta may differ in rounding: the rows are summed over a different
 * number of CTAs), same argument meaning, but no plan: theta (device, fp32 [log2 n][n/2]) is passed
 * directly and the work runs on the CURRENT device.  The cos/sin table and the partial sums live in
 * an 8 MiB array in the library's device data segment, which every GPU that loads the library holds
 * until the process exits.  Limits and rules that follow from that:
 *   - n <= BFQ_NOALLOC_MAX_N (power of two >= BFQ_MIN_N), else BFQ_ERR_TOO_LARGE; rows is unlimited;
 *   - all calls share the one array: calls that may overlap on a GPU (different streams, different
 *     threads) race with each other -- serialise them; contents left by an earlier call are harmless
 *     (each call rewrites the table and overwrites the partial sums it reads);
 *   - the first call on each device resolves the array's address (cudaGetSymbolAddress) and sets a
 *     kernel attribute; make that first call before any stream capture begins.
 * It calls no cudaMalloc, cudaFree or other allocating routine.  d-theta is bit-reproducible from call
 * to call on the same device.
 */
int bfq_backward_noalloc(int n, const float* theta, const void* x, bfq_dtype xt, const void* g, bfq_dtype gt,
                         int64_t rows, int64_t ld, void* dx, bfq_dtype dxt, float* dtheta, void* stream);

/* Synchronises the device and returns BFQ_OK, or BFQ_ERR_DEVICE_TIMEOUT if a kernel of this plan
 * reported a bounded wait that ran out, or BFQ_ERR_CUDA.  (No counterpart in the paper.) */
int bfq_device_status(bfq_plan* plan);

/* Last cudaError_t seen by this plan (0 = cudaSuccess).  (No counterpart in the paper.) */
int bfq_last_cuda_error(const bfq_plan* plan);

/*
 * Which rotation form the tuned kernels (n = 4096, n = 8192) run with the current angles.  They use the scaled two-FMA
 * form (paper Sec. "Inference Efficiency": two FMAs per pair) in which every element carries the product of the
 * cosines it has been through; when such a product leaves [2^-64, 1] (an angle within ~1e-19 .. of an odd multiple of
 * pi/2 along some path, e.g. angles that are exact multiples of pi/2) the table build selects the three-shear form
 * instead, which has no such limit.  Returns bit 0 = forward tables use the fallback, bit 1 = inverse tables (built by
 * the first bfq_inverse / bfq_backward after bfq_set_angles; at n = 8192 the tables of either half of the row) use the
 * fallback; or a negative bfq_status.  Synchronises
 * the device.  With the scaled form, inputs must stay below about 2^56 in magnitude (intermediate values are the true
 * values divided by the factor).  (No counterpart in the paper; informational.)
 */
int bfq_stage_form(bfq_plan* plan);

/*
 * Test hook (no counterpart in the paper): while enabled, the tuned n = 4096 forward kernels of this plan announce 16
 * bytes more per row load than the load delivers and bound their waits at 4096 polls, so that every wait runs out:
 * the kernels return normally with meaningless outputs (inside their buffers) and bfq_device_status reports
 * BFQ_ERR_DEVICE_TIMEOUT once.  Exercises the bounded-wait path without hanging or faulting the GPU.
 */
int bfq_test_stuck_wait(bfq_plan* plan, int enable);

/* Static string for a status code. */
const char* bfq_status_string(int status);

/*
 * Dense product with on-the-fly dequantization, for the reconstruction loss of the calibration step (paper Sec. 3.4:
 * || W x - Dequant(Quant(W B^T)) Dequant(Quant(B x)) ||^2) and its gradients:
 *     C[i][j] = alpha * sum_{k < K} A(i, k) * B(j, k),   i < m, j < n;   C fp32, row-major, leading dimension ldc >= n.
 * Each operand is described by (data, kind, transposed, ld, scales):
 *   kind        BFQ_OP_F32 / BFQ_OP_BF16: rows of numbers;  BFQ_OP_CODES2 / 4 / 8: packed two's-complement codes in
 *               the layout bfq_forward_quant writes, value = code * scale of its stored row (scales: fp16 bits, device);
 *   transposed  0: stored [m or n][K] (the contraction runs along a stored row);  1: stored [K][m or n];
 *   ld          leading dimension in elements (codes: in codes) >= the stored row's length; ld * element bits must be
 *               a multiple of 128 and data 16-byte aligned.
 * K must be a multiple of 64; m, n are arbitrary.  All pointers are device pointers.  The products run on the tensor
 * cores in bf16 with fp32 accumulation: codes are exact, fp32 numbers are split into two bf16 terms (relative error
 * 2^-17 per element), bf16 numbers are exact.  Asynchronous on `stream`; allocates nothing; a bounded device-side
 * wait that runs out is reported by bfq_device_status.  Returns BFQ_OK, BFQ_ERR_NULL, BFQ_ERR_STRIDE (sizes, leading
 * dimensions, K not a multiple of 64), BFQ_ERR_ALIGN, BFQ_ERR_DTYPE (kind) or BFQ_ERR_CUDA.
 */
#define BFQ_OP_F32 0
#define BFQ_OP_BF16 1
#define BFQ_OP_CODES2 2
#define BFQ_OP_CODES4 4
#define BFQ_OP_CODES8 8
int bfq_dequant_gemm(bfq_plan* plan, int64_t m, int64_t n, int64_t k, float alpha, const void* a, int a_kind,
                     int a_transposed, int64_t lda, const uint16_t* a_scales, const void* b, int b_kind, int b_transposed,
                     int64_t ldb, const uint16_t* b_scales, float* c, int64_t ldc, void* stream);

/*
 * bfq_forward_quant for rows that live in HOST memory (paper Sec. 3.4 quantizer on y = Q x, as bfq_forward_quant): the
 * same result, with the host -> device copy of the rows, the kernels and the device -> host copy of codes and scales
 * overlapped chunk by chunk on two streams the plan owns.
 *   x_host          HOST pointer, [rows][ldx] of type xt; pinned (page-locked) memory for the copies to be asynchronous
 *   codes_host      HOST pointer, [rows][n*bits/8] packed codes; scales_host_f16: HOST pointer, [rows] fp16 bits
 *   workspace       DEVICE pointer, 16-byte aligned, owned by the caller, workspace_bytes long: holds two chunks of rows
 *                   with their codes and scales; bfq_forward_quant_host_workspace(plan, xt, bits, chunk_rows) gives the
 *                   size for a wanted chunk (rows are processed in chunks of a multiple of 8 rows that fit twice)
 * Enqueued on `stream` and the plan's two copy streams; when the work enqueued on `stream` by this call is done, the
 * host buffers hold the results.  The host buffers must stay valid until then.  Allocates nothing.  The paper has no
 * counterpart of this call (it is the end-to-end form of the online activation path).
 * Returns BFQ_OK, BFQ_ERR_NULL, BFQ_ERR_DTYPE, BFQ_ERR_BITS, BFQ_ERR_STRIDE, BFQ_ERR_ALIGN, BFQ_ERR_WORKSPACE (no angles
 * set, or a workspace too small for 8 rows twice) or BFQ_ERR_CUDA.
 */
int bfq_forward_quant_host(bfq_plan* plan, const void* x_host, bfq_dtype xt, int64_t rows, int64_t ldx, int bits,
                           uint8_t* codes_host, uint16_t* scales_host_f16, void* workspace, size_t workspace_bytes,
                           void* stream);
/* Bytes of device workspace that let bfq_forward_quant_host work in chunks of chunk_rows rows (0 on bad arguments). */
size_t bfq_forward_quant_host_workspace(const bfq_plan* plan, bfq_dtype xt, int bits, int64_t chunk_rows);

/*
 * Measures, on the current device, how many SM cycles one warp scheduler needs per FP32 FMA instruction with register
 * operands only (no memory traffic in the timed loops): out[0] packed fma.rn.f32x2 with three distinct register
 * operands (the pattern of a rotation with per-pair constants), out[1] packed with two distinct operands, out[2] /
 * out[3] the same for scalar FMAs.  `cycles_per_instruction` is a HOST array of 4 floats.  Synchronous: allocates and
 * frees a few hundred bytes of device memory and synchronises the device; meant for benchmarks, which print the
 * measured issue rate beside the nominal peak of one FMA per lane per cycle (the paper counts FLOPs, appendix table
 * "FLOP comparison"; it has no counterpart of this call).  Returns BFQ_OK, BFQ_ERR_NULL or BFQ_ERR_CUDA.
 */
int bfq_measure_fma_rates(float* cycles_per_instruction);

/*
 * Measures, on the current device, the SM cycles one tcgen05.mma (bf16 x bf16 -> fp32, M = 128, K = 16, operands in
 * shared memory, issued back to back by one thread) takes for N = 16, 64, 128 and 256: `cycles_per_mma` is a HOST
 * array of 4 floats in that order.  It prices running merged butterfly stages as small dense blocks on the tensor
 * cores (one 2^k x 2^k block per MMA; the paper's Sec. 3.2.1 structure has a different block for every group of
 * columns) against the FP32 path; no counterpart in the paper.  Synchronous, allocates and frees a few bytes of device
 * memory.  Returns BFQ_OK, BFQ_ERR_NULL, BFQ_ERR_CUDA or BFQ_ERR_DEVICE_TIMEOUT (a bounded wait ran out).
 */
int bfq_measure_mma_rates(float* cycles_per_mma);

/* Number of CTAs the backward pass uses (= number of d-theta partial sums); informational. */
int bfq_backward_partials(const bfq_plan* plan);

#ifdef __cplusplus
}
#endif
#endif /* BFQ_H_ */
