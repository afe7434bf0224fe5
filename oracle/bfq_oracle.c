/*
 * CPU oracle for the butterfly-rotation + low-bit quantization path of ButterflyQuant.
 *
 * TEST INFRASTRUCTURE ONLY.  This file is the plain, slow, obviously-correct statement
 * of what the path computes; the tests, the smoke check and the benchmark's CPU-baseline
 * leg call it, and nothing else may.  It shares no code, header, table or constant with
 * the CUDA library and never calls it.
 *
 * All arithmetic is IEEE double (compile with -ffp-contract=off, no fast-math).  Rows are
 * independent; the only parallelism is an OpenMP loop over rows.
 *
 * Notation (paper, Sec. 3.2.1 "Structure and Parameterization" and the n = 8 appendix
 * example): n = 2^L; layer i = 1..L of the paper is stage s = i - 1 here; stage s pairs
 * indices at stride h = 2^s; theta[s][j] is the angle of the j-th pair of the stage when
 * pairs are listed by increasing low index (appendix: layer 2 pairs (0,2),(1,3),(4,6),(5,7)
 * carry theta_{2,1..4}).  The low index of a pair gets  cos*a - sin*b,  the high index
 * sin*a + cos*b  (Givens matrix G(theta), Sec. 3.2.1).
 *
 * Readings taken where the paper leaves a choice (all listed in the design notes):
 *  - y = Q x applies stride 1 first:  Q = B_L ... B_2 B_1  (Sec. "Inference Efficiency":
 *    sequential stages, stride 2^{i-1} at stage i; the appendix diagram runs layer 1 first).
 *  - no global permutation: B_i is exactly the printed stride-2^{i-1} matrix.
 *  - quantizer (Sec. 3.4): per row, s = max|y| / (2^{b-1}-1), stored as IEEE fp16
 *    (round to nearest even, saturating at 65504); codes = clip(round(y / s16)) with the
 *    fp16-rounded scale, round-half-even, decided on the fp32 value of y / s16.
 *    A row whose fp16 scale is 0 gets all-zero codes.
 *
 * Pins (tests/test_oracle_pins.py): printed n = 8 layer matrices; Q^T Q = I and norm
 * preservation; theta = 0 gives I; theta = pi/4 gives H_n D with |entries| = 1/sqrt(n);
 * Kronecker closed form for stage-uniform angles; stage-by-stage == dense product;
 * inverse(forward(x)) = x; d theta == central finite differences; adjoint identity;
 * quantizer closed-form properties and a hand-worked example; fold invariance
 * (W Q^T)(Q x) = W x; fp16 rounding against numpy's float16; the Hadamard transform against the
 * Kronecker power of H_2, |entries| = 1/sqrt(n) and the theta = pi/4 butterfly (Q = H_n D).
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

static int ilog2_exact(int64_t n) {
    int L = 0;
    if (n < 2) return -1;
    while (((int64_t)1 << L) < n) ++L;
    return (((int64_t)1 << L) == n) ? L : -1;
}

/* ---- fp16 (IEEE binary16) from float, round-to-nearest-even, saturating to 65504 ---- */
uint16_t orc_f32_to_f16_sat(float f) {
    uint32_t u;
    memcpy(&u, &f, 4);
    uint16_t sign = (uint16_t)((u >> 16) & 0x8000u);
    uint32_t mag = u & 0x7FFFFFFFu;
    if (mag > 0x7F800000u) return (uint16_t)(sign | 0x7E00u); /* NaN */
    double a = fabs((double)f);
    if (a >= 65520.0) return (uint16_t)(sign | 0x7BFFu);      /* would round to inf: saturate */
    if (a == 0.0) return sign;
    int e;
    double m = frexp(a, &e);          /* a = m * 2^e, m in [0.5, 1) */
    int exp16 = e - 1;                /* a = (2m) * 2^(e-1), 2m in [1, 2) */
    double q;                         /* a expressed in units of the target ulp */
    int biased;
    if (exp16 < -14) {                /* subnormal: ulp = 2^-24 */
        q = ldexp(a, 24);
        biased = 0;
    } else {                          /* normal: ulp = 2^(exp16-10) */
        q = ldexp(m, 11);             /* in [1024, 2048) */
        biased = exp16 + 15;
    }
    double fl = floor(q);
    double r = q - fl;
    uint32_t n = (uint32_t)fl;
    if (r > 0.5 || (r == 0.5 && (n & 1u))) n += 1;
    uint32_t bits;
    if (biased == 0) {
        bits = n;                     /* n == 1024 becomes the smallest normal: same encoding */
    } else {
        bits = ((uint32_t)biased << 10) + (n - 1024u); /* n == 2048 carries into the exponent */
    }
    return (uint16_t)(sign | (uint16_t)bits);
}

double orc_f16_to_f64(uint16_t h) {
    int sign = (h >> 15) & 1;
    int e = (h >> 10) & 0x1F;
    int m = h & 0x3FF;
    double v;
    if (e == 0) v = ldexp((double)m, -24);
    else if (e == 31) v = m ? NAN : INFINITY;
    else v = ldexp((double)(m + 1024), e - 25);
    return sign ? -v : v;
}

/* ---- one stage, in place on one row (Sec. 3.2.1; appendix n = 8 matrices) ---- */
static void stage_forward(int64_t n, int s, const double* th, double* z) {
    int64_t h = (int64_t)1 << s;
    int64_t j = 0;                                   /* pairs in order of increasing low index */
    for (int64_t base = 0; base < n; base += 2 * h) {
        for (int64_t k = 0; k < h; ++k, ++j) {
            int64_t lo = base + k, hi = lo + h;
            double c = cos(th[j]), sn = sin(th[j]);
            double a = z[lo], b = z[hi];
            z[lo] = c * a - sn * b;
            z[hi] = sn * a + c * b;
        }
    }
}

/* transpose of the stage: G(theta)^T on every pair */
static void stage_transpose(int64_t n, int s, const double* th, double* z) {
    int64_t h = (int64_t)1 << s;
    int64_t j = 0;
    for (int64_t base = 0; base < n; base += 2 * h) {
        for (int64_t k = 0; k < h; ++k, ++j) {
            int64_t lo = base + k, hi = lo + h;
            double c = cos(th[j]), sn = sin(th[j]);
            double a = z[lo], b = z[hi];
            z[lo] = c * a + sn * b;
            z[hi] = -sn * a + c * b;
        }
    }
}

/* Dense n x n matrix of one layer, row-major: the printed B_{s+1}. */
int orc_dense_stage(int64_t n, int s, const double* theta_s, double* M) {
    int L = ilog2_exact(n);
    if (L < 0 || s < 0 || s >= L) return -1;
    memset(M, 0, sizeof(double) * (size_t)(n * n));
    int64_t h = (int64_t)1 << s;
    int64_t j = 0;
    for (int64_t base = 0; base < n; base += 2 * h) {
        for (int64_t k = 0; k < h; ++k, ++j) {
            int64_t lo = base + k, hi = lo + h;
            double c = cos(theta_s[j]), sn = sin(theta_s[j]);
            M[lo * n + lo] = c;
            M[lo * n + hi] = -sn;
            M[hi * n + lo] = sn;
            M[hi * n + hi] = c;
        }
    }
    return 0;
}

/* y = Q x, stage s = 0 .. L-1 in that order.  theta: [L][n/2]. */
int orc_forward(int64_t n, const double* theta, const double* x, int64_t rows, int64_t ldx,
                double* y, int64_t ldy) {
    int L = ilog2_exact(n);
    if (L < 0) return -1;
    int64_t r;
#pragma omp parallel for schedule(static)
    for (r = 0; r < rows; ++r) {
        double* z = y + r * ldy;
        memmove(z, x + r * ldx, sizeof(double) * (size_t)n);
        for (int s = 0; s < L; ++s) stage_forward(n, s, theta + (int64_t)s * (n / 2), z);
    }
    return 0;
}

/* x = Q^T y, stage s = L-1 .. 0 with G^T. */
int orc_inverse(int64_t n, const double* theta, const double* y, int64_t rows, int64_t ldy,
                double* x, int64_t ldx) {
    int L = ilog2_exact(n);
    if (L < 0) return -1;
    int64_t r;
#pragma omp parallel for schedule(static)
    for (r = 0; r < rows; ++r) {
        double* z = x + r * ldx;
        memmove(z, y + r * ldy, sizeof(double) * (size_t)n);
        for (int s = L - 1; s >= 0; --s) stage_transpose(n, s, theta + (int64_t)s * (n / 2), z);
    }
    return 0;
}

/*
 * Normalised Walsh-Hadamard transform y = H_n x, the fixed rotation the paper compares against
 * (Sec. 3.1.1): H_1 = [1], H_2n = 1/sqrt(2) [[H_n, H_n], [H_n, -H_n]].  Written as that recursion:
 * the first and second halves of x are transformed by H_{n/2}, then combined.
 */
static void hadamard_rec(int64_t n, double* z, double* tmp) {
    if (n == 1) return;
    const int64_t h = n / 2;
    hadamard_rec(h, z, tmp);
    hadamard_rec(h, z + h, tmp);
    const double r = 1.0 / sqrt(2.0);
    for (int64_t i = 0; i < h; ++i) {
        const double a = z[i], b = z[h + i];
        tmp[i] = r * (a + b);
        tmp[h + i] = r * (a - b);
    }
    memcpy(z, tmp, sizeof(double) * (size_t)n);
}

int orc_hadamard(int64_t n, const double* x, int64_t rows, int64_t ldx, double* y, int64_t ldy) {
    if (ilog2_exact(n) < 0) return -1;
    int64_t r;
    int fail = 0;
#pragma omp parallel for schedule(static)
    for (r = 0; r < rows; ++r) {
        double* tmp = (double*)malloc(sizeof(double) * (size_t)n);
        if (!tmp) {
            fail = 1;
            continue;
        }
        double* z = y + r * ldy;
        memmove(z, x + r * ldx, sizeof(double) * (size_t)n);
        hadamard_rec(n, z, tmp);
        free(tmp);
    }
    return fail ? -8 : 0;
}

/*
 * Per-row symmetric absmax quantizer (Sec. 3.4, Quant / Dequant).
 *   qmax = 2^(b-1) - 1;  s16 = fp16(float(max|y|) / qmax);
 *   code_k = clip(rint_f32(y_k / s16), -2^(b-1), qmax).
 * scale_in (optional): use these fp16 scales instead of computing them (the checker's
 * re-quantisation rule for rows whose scale differs by one fp16 ulp).
 * prequant (optional): the double value y_k / s16 before rounding, for boundary analysis.
 */
int orc_quantize(int64_t n, int bits, const double* y, int64_t rows, int64_t ldy,
                 int8_t* codes /*[rows][n]*/, uint16_t* scale_f16 /*[rows]*/,
                 const uint16_t* scale_in /*or NULL*/, double* prequant /*[rows][n] or NULL*/) {
    if (bits != 2 && bits != 4 && bits != 8) return -3;
    int qmax = (1 << (bits - 1)) - 1, qmin = -(1 << (bits - 1));
    int64_t r;
#pragma omp parallel for schedule(static)
    for (r = 0; r < rows; ++r) {
        const double* yr = y + r * ldy;
        uint16_t s16;
        if (scale_in) {
            s16 = scale_in[r];
        } else {
            double amax = 0.0;
            for (int64_t k = 0; k < n; ++k) {
                double a = fabs(yr[k]);
                if (a > amax) amax = a;
            }
            float sf = (float)amax / (float)qmax;
            s16 = orc_f32_to_f16_sat(sf);
        }
        scale_f16[r] = s16;
        double sd = orc_f16_to_f64(s16);
        for (int64_t k = 0; k < n; ++k) {
            int q = 0;
            double v = 0.0;
            if (sd > 0.0) {
                v = yr[k] / sd;
                float vf = (float)v;
                float rf = rintf(vf);              /* round half to even (default mode) */
                if (rf > (float)qmax) rf = (float)qmax;
                if (rf < (float)qmin) rf = (float)qmin;
                q = (int)rf;
            }
            codes[r * n + k] = (int8_t)q;
            if (prequant) prequant[r * n + k] = v;
        }
    }
    return 0;
}

/* Two's-complement packing: element k occupies bits [b*(k mod 8/b), +b) of byte k*b/8. */
int orc_pack(int64_t n, int bits, const int8_t* codes, int64_t rows, uint8_t* packed) {
    if (bits != 2 && bits != 4 && bits != 8) return -3;
    int per = 8 / bits;
    int mask = (1 << bits) - 1;
    int64_t nb = n * bits / 8;
    for (int64_t r = 0; r < rows; ++r) {
        for (int64_t B = 0; B < nb; ++B) {
            unsigned v = 0;
            for (int e = 0; e < per; ++e) {
                int q = codes[r * n + B * per + e];
                v |= ((unsigned)q & (unsigned)mask) << (bits * e);
            }
            packed[r * nb + B] = (uint8_t)v;
        }
    }
    return 0;
}

int orc_unpack(int64_t n, int bits, const uint8_t* packed, int64_t rows, int8_t* codes) {
    if (bits != 2 && bits != 4 && bits != 8) return -3;
    int per = 8 / bits;
    int mask = (1 << bits) - 1;
    int signbit = 1 << (bits - 1);
    int64_t nb = n * bits / 8;
    for (int64_t r = 0; r < rows; ++r) {
        for (int64_t B = 0; B < nb; ++B) {
            unsigned v = packed[r * nb + B];
            for (int e = 0; e < per; ++e) {
                int q = (int)((v >> (bits * e)) & (unsigned)mask);
                if (q & signbit) q -= (1 << bits);
                codes[r * n + B * per + e] = (int8_t)q;
            }
        }
    }
    return 0;
}

/*
 * Backward of y = Q x for upstream gradient g = dL/dy (Sec. 3.5.1, dG/dtheta).
 * Keeps every stage input z^0..z^L, then walks s = L-1..0:
 *   dtheta[s][j] += gbar^T (dG/dtheta) z^s  on the pair,   gbar <- G^T gbar.
 * dtheta [L][n/2] is the sum over all rows (accumulated in row order).
 */
int orc_backward(int64_t n, const double* theta, const double* x, const double* g, int64_t rows,
                 int64_t ld, double* dx, int64_t lddx, double* dtheta) {
    int L = ilog2_exact(n);
    if (L < 0) return -1;
    int64_t half = n / 2;
    memset(dtheta, 0, sizeof(double) * (size_t)(L * half));
    int nthreads = 1;
#ifdef _OPENMP
    extern int omp_get_max_threads(void);
    extern int omp_get_thread_num(void);
    nthreads = omp_get_max_threads();
#endif
    /* fixed row blocks, one partial per block, summed in block order: result does not
       depend on the thread count */
    int64_t block = 64;
    int64_t nblocks = (rows + block - 1) / block;
    double* partial = (double*)calloc((size_t)(nblocks > 0 ? nblocks : 1) * L * half, sizeof(double));
    if (!partial) return -8;
    (void)nthreads;
    int64_t bidx;
#pragma omp parallel for schedule(dynamic, 1)
    for (bidx = 0; bidx < nblocks; ++bidx) {
        double* zs = (double*)malloc(sizeof(double) * (size_t)((L + 1) * n));
        double* gb = (double*)malloc(sizeof(double) * (size_t)n);
        double* dth = partial + bidx * L * half;
        int64_t r0 = bidx * block, r1 = r0 + block < rows ? r0 + block : rows;
        for (int64_t r = r0; r < r1; ++r) {
            memcpy(zs, x + r * ld, sizeof(double) * (size_t)n);
            for (int s = 0; s < L; ++s) {
                memcpy(zs + (int64_t)(s + 1) * n, zs + (int64_t)s * n, sizeof(double) * (size_t)n);
                stage_forward(n, s, theta + (int64_t)s * half, zs + (int64_t)(s + 1) * n);
            }
            memcpy(gb, g + r * ld, sizeof(double) * (size_t)n);
            for (int s = L - 1; s >= 0; --s) {
                const double* th = theta + (int64_t)s * half;
                const double* z = zs + (int64_t)s * n;      /* stage input */
                int64_t h = (int64_t)1 << s;
                int64_t j = 0;
                for (int64_t base = 0; base < n; base += 2 * h) {
                    for (int64_t k = 0; k < h; ++k, ++j) {
                        int64_t lo = base + k, hi = lo + h;
                        double c = cos(th[j]), sn = sin(th[j]);
                        double a = z[lo], b = z[hi];
                        double ga = gb[lo], gbv = gb[hi];
                        /* [ga gb] * [[-sin, -cos],[cos, -sin]] * [a b]^T */
                        dth[(int64_t)s * half + j] += ga * (-sn * a - c * b) + gbv * (c * a - sn * b);
                        gb[lo] = c * ga + sn * gbv;
                        gb[hi] = -sn * ga + c * gbv;
                    }
                }
            }
            memcpy(dx + r * lddx, gb, sizeof(double) * (size_t)n);
        }
        free(zs);
        free(gb);
    }
    for (int64_t b = 0; b < nblocks; ++b)
        for (int64_t k = 0; k < L * half; ++k) dtheta[k] += partial[b * L * half + k];
    free(partial);
    return 0;
}

/* forward + quantize + pack in one call (what bfq_forward_quant / bfq_fold_weights compute:
   folding W Q^T applies Q to every row of W, Sec. 3.1 computational invariance). */
int orc_forward_quant(int64_t n, const double* theta, const double* x, int64_t rows, int64_t ldx,
                      int bits, uint8_t* packed, uint16_t* scale_f16, double* y_out /*or NULL*/) {
    int L = ilog2_exact(n);
    if (L < 0) return -1;
    if (bits != 2 && bits != 4 && bits != 8) return -3;
    int64_t nb = n * bits / 8;
    int64_t chunk = 256;
    for (int64_t r0 = 0; r0 < rows; r0 += chunk) {
        int64_t rc = rows - r0 < chunk ? rows - r0 : chunk;
        double* y = y_out ? y_out + r0 * n : (double*)malloc(sizeof(double) * (size_t)(rc * n));
        int8_t* codes = (int8_t*)malloc((size_t)(rc * n));
        if (!y || !codes) return -8;
        orc_forward(n, theta, x + r0 * ldx, rc, ldx, y, n);
        orc_quantize(n, bits, y, rc, n, codes, scale_f16 + r0, NULL, NULL);
        orc_pack(n, bits, codes, rc, packed + r0 * nb);
        free(codes);
        if (!y_out) free(y);
    }
    return 0;
}

int orc_num_threads(void) {
#ifdef _OPENMP
    extern int omp_get_max_threads(void);
    return omp_get_max_threads();
#else
    return 1;
#endif
}
