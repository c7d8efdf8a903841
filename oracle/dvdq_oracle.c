/*
 * dvdq_oracle.c -- TEST INFRASTRUCTURE ONLY.
 *
 * A plain, slow, fp64 CPU statement of the quantized-linear path of DVD-Quant
 * (Sec. 3.2 "Auto-scaling Rotated Quantization", Eq. 10; Sec. 3.1 Quant/DeQuant
 * definitions).  It exists so that the CUDA library can be checked against
 * something written directly from the paper.  Only tests, the smoke check and
 * the benchmark's cpu-baseline leg may call it; the product path never does,
 * and this file shares no code, header, table or helper with the CUDA sources.
 *
 * Everything is the textbook definition: dense matrix products, no fast
 * transform, no blocking, no fusion.  OpenMP only spreads independent rows over
 * cores; each row is computed exactly as a single thread would.
 *
 * bf16 values travel as their 16 raw bits (uint16_t).
 *
 * Readings adopted where the paper is silent (each also listed in the design
 * notes of the repository):
 *   - the rotation for K not a power of two is block diagonal, I (x) H_B / sqrt(B)
 *     with H_B the Sylvester Hadamard matrix (Sec. 3.2 names a Hadamard matrix and
 *     a fast Hadamard transform but gives no construction);
 *   - one scale per token: s_i = max_k |x~_ik| / qmax  (Sec. 3.2 says the deployed
 *     kernels use a block-wise variant of Eq. 10's scaling; one block per token row
 *     is the variant that keeps the product an integer GEMM);
 *   - the activation quantizer Q of Eq. 10 is symmetric, qmax = 2^(b-1) - 1;
 *   - round half to even wherever the paper writes the nearest-integer bracket.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

/* ---------------------------------------------------------------- bf16 <-> fp64 */

/* A bf16 is the upper half of an IEEE binary32. */
double oracle_bf16_to_double(uint16_t h) {
    uint32_t u = ((uint32_t)h) << 16;
    float f;
    memcpy(&f, &u, sizeof f);
    return (double)f;
}

/* Round a double to the nearest bf16 (8 significand bits, binary32 exponent range),
 * ties to even, in ONE rounding step (no intermediate binary32 rounding). */
uint16_t oracle_double_to_bf16(double v) {
    if (isnan(v)) return 0x7FC0;
    uint16_t sign = signbit(v) ? 0x8000 : 0;
    double a = fabs(v);
    if (a == 0.0) return sign;
    if (isinf(a)) return (uint16_t)(sign | 0x7F80);
    int e;
    double m = frexp(a, &e);            /* a = m * 2^e, 0.5 <= m < 1 */
    int ulp_exp = e - 8;                /* 8 significant bits -> ulp = 2^(e-8) */
    if (ulp_exp < -133) ulp_exp = -133; /* subnormal bf16: fixed ulp 2^-133 */
    (void)m;
    double q = nearbyint(ldexp(a, -ulp_exp)); /* default rounding mode: ties to even */
    double r = ldexp(q, ulp_exp);             /* exactly representable in binary32 */
    if (r >= ldexp(1.0, 128)) return (uint16_t)(sign | 0x7F80);
    float f = (float)r;                       /* exact */
    uint32_t u;
    memcpy(&u, &f, sizeof u);
    return (uint16_t)(sign | (uint16_t)(u >> 16));
}

/* ---------------------------------------------------------------- rotation */

static int popcount64(uint64_t x) {
    int c = 0;
    while (x) { c += (int)(x & 1u); x >>= 1; }
    return c;
}

/* Sylvester Hadamard matrix of order B (a power of two), orthonormal:
 * H[i][j] = (-1)^{popcount(i AND j)} / sqrt(B).   (Sec. 3.2: rotation Q with Q Q^T = I.) */
void oracle_hadamard_matrix(int64_t B, double* H) {
    double inv = 1.0 / sqrt((double)B);
    for (int64_t i = 0; i < B; ++i)
        for (int64_t j = 0; j < B; ++j)
            H[i * B + j] = (popcount64((uint64_t)(i & j)) & 1) ? -inv : inv;
}

/* X~ = X R with R = I_{K/B} (x) H_B  (Sec. 3.2, "X~ = XH"), by the dense definition
 * x~_ik = sum_j x_ij R_jk.  B == 0 means no rotation (R = I).
 * x: rows x K bf16 bits with leading dimension ld; xt: rows x K doubles, dense. */
int oracle_rotate_rows(const uint16_t* x, int64_t rows, int64_t K, int64_t ld, int64_t B, double* xt) {
    if (B == 0) {
        for (int64_t i = 0; i < rows; ++i)
            for (int64_t k = 0; k < K; ++k) xt[i * K + k] = oracle_bf16_to_double(x[i * ld + k]);
        return 0;
    }
    if (B < 1 || (B & (B - 1)) != 0 || K % B != 0) return 1;
    double* H = (double*)malloc(sizeof(double) * (size_t)B * (size_t)B);
    if (!H) return 2;
    oracle_hadamard_matrix(B, H);
#pragma omp parallel for schedule(static)
    for (int64_t i = 0; i < rows; ++i) {
        for (int64_t blk = 0; blk < K / B; ++blk) {
            const uint16_t* xr = x + i * ld + blk * B;
            double* out = xt + i * K + blk * B;
            for (int64_t k = 0; k < B; ++k) out[k] = 0.0;
            for (int64_t j = 0; j < B; ++j) {
                double xj = oracle_bf16_to_double(xr[j]);
                const double* Hj = H + j * B;
                for (int64_t k = 0; k < B; ++k) out[k] += xj * Hj[k];
            }
        }
    }
    free(H);
    return 0;
}

/* ---------------------------------------------------------------- activation quantizer */

/* Per token i (Sec. 3.2, Eq. 10 with one scale per token row):
 *   a_i = max_k |x~_ik|,  s_i = a_i / qmax,  qmax = 2^(bits-1) - 1,
 *   c_ik = clamp(round_half_even(x~_ik / s_i), -2^(bits-1), qmax).
 * An all-zero token gets s_i = 0 and all codes 0.
 * scale32 is s_i rounded to binary32, the type the scale is stored in. */
int oracle_act_quantize(const double* xt, int64_t rows, int64_t K, int bits,
                        int32_t* codes, double* scale64, float* scale32) {
    if (bits < 2 || bits > 16) return 1;
    const double qmax = (double)((1 << (bits - 1)) - 1);
    const double qmin = -(double)(1 << (bits - 1));
#pragma omp parallel for schedule(static)
    for (int64_t i = 0; i < rows; ++i) {
        const double* r = xt + i * K;
        double a = 0.0;
        for (int64_t k = 0; k < K; ++k) { double v = fabs(r[k]); if (v > a) a = v; }
        double s = a / qmax;
        scale64[i] = s;
        scale32[i] = (float)s;
        for (int64_t k = 0; k < K; ++k) {
            double q = 0.0;
            if (s > 0.0) {
                q = nearbyint(r[k] / s);
                if (q > qmax) q = qmax;
                if (q < qmin) q = qmin;
            }
            codes[i * K + k] = (int32_t)q;
        }
    }
    return 0;
}

/* ---------------------------------------------------------------- weight quantizers (Sec. 3.1) */

/* Quant:   W_q = clamp(round(W / Delta) + z, 0, 2^b - 1)
 * DeQuant: W^  = Delta * (W_q - z)                                  (Sec. 3.1, b = 4)
 * MinMax per output channel (row): Delta = (max - min) / (2^b - 1), z = -round(min / Delta).
 * z is kept inside [0, 2^b - 1] so that it is a valid code offset. */
void oracle_weight_quantize_minmax(const double* wt, int64_t N, int64_t K,
                                   uint8_t* u, float* delta, int32_t* zero) {
    const double levels = 15.0;
#pragma omp parallel for schedule(static)
    for (int64_t n = 0; n < N; ++n) {
        const double* r = wt + n * K;
        double lo = r[0], hi = r[0];
        for (int64_t k = 1; k < K; ++k) { if (r[k] < lo) lo = r[k]; if (r[k] > hi) hi = r[k]; }
        double d = (hi - lo) / levels;
        if (!(d > 0.0)) { /* constant row: any step works, codes sit at the zero point */
            d = (fabs(hi) > 0.0) ? fabs(hi) : 1.0;
        }
        double z = -nearbyint(lo / d);
        if (z < 0.0) z = 0.0;
        if (z > levels) z = levels;
        delta[n] = (float)d;
        zero[n] = (int32_t)z;
        for (int64_t k = 0; k < K; ++k) {
            double q = nearbyint(r[k] / d) + z;
            if (q < 0.0) q = 0.0;
            if (q > levels) q = levels;
            u[n * K + k] = (uint8_t)q;
        }
    }
}

/* "Symmetric per-output-channel 4-bit": the Quant/DeQuant format above with the zero
 * point pinned at z = 8 and Delta = max|w| / 7, so that (W_q - z) lies in [-7, 7]. */
void oracle_weight_quantize_symmetric(const double* wt, int64_t N, int64_t K,
                                      uint8_t* u, float* delta, int32_t* zero) {
#pragma omp parallel for schedule(static)
    for (int64_t n = 0; n < N; ++n) {
        const double* r = wt + n * K;
        double a = 0.0;
        for (int64_t k = 0; k < K; ++k) { double v = fabs(r[k]); if (v > a) a = v; }
        double d = a / 7.0;
        if (!(d > 0.0)) d = 1.0;
        delta[n] = (float)d;
        zero[n] = 8;
        for (int64_t k = 0; k < K; ++k) {
            double q = nearbyint(r[k] / d);
            if (q < -8.0) q = -8.0;
            if (q > 7.0) q = 7.0;
            u[n * K + k] = (uint8_t)(q + 8.0);
        }
    }
}

/* ---------------------------------------------------------------- Bounded-init Grid Refinement (Alg. 1, Sec. 3.1) */

/* Quant of Sec. 3.1 for one row with a given grid (Delta, z); returns the squared error
 * || w - Delta (W_q - z) ||^2 and, if the pointers are not NULL, the three row sums the
 * refinement formulas need:  <W_q - z, w>,  <W_q - z, W_q - z>,  sum of W_q. */
static double bgr_row_quantize(const double* w, int64_t K, double levels, double d, double z,
                               uint8_t* u_or_null, double* s_qw, double* s_qq, double* s_q) {
    double e2 = 0.0, qw = 0.0, qq = 0.0, sq = 0.0;
    for (int64_t k = 0; k < K; ++k) {
        double c = nearbyint(w[k] / d) + z;
        if (c < 0.0) c = 0.0;
        if (c > levels) c = levels;
        double q = c - z;
        double r = w[k] - d * q;
        e2 += r * r; qw += q * w[k]; qq += q * q; sq += c;
        if (u_or_null) u_or_null[k] = (uint8_t)c;
    }
    if (s_qw) *s_qw = qw;
    if (s_qq) *s_qq = qq;
    if (s_q) *s_q = sq;
    return e2;
}

/* Alg. 1 for every row (output channel) on its own: the objective of Sec. 3.1,
 * || W - Delta (W_q - z) ||_F with one (Delta, z) per row, separates over rows.
 *
 *   for i = 1, 2, ... (shrink steps, delta_l = delta_u = (max - min) / n_steps):
 *       clip the row to [min + i delta_l, max - i delta_u]; MinMax grid of the clipped row
 *       (Delta(0), z(0)); quantize the UNclipped row on it; then repeat
 *           Delta' = <W_q - z, w> / <W_q - z, W_q - z>                  (least squares, z and W_q fixed)
 *           z'     = clamp(round(mean(W_q) - mean(w) / Delta'), 0, 2^b - 1)  (relax, then round)
 *           W_q'   = clamp(round(w / Delta') + z', 0, 2^b - 1)
 *       until the error stops falling by at least eps; keep the best grid seen.
 *
 * Readings where Alg. 1 cannot be taken literally:
 *   - it uses one letter for the number of rows and for the number of shrink steps: n_steps here;
 *   - its bounds cross once 2 i >= n_steps, so i stops before that;
 *   - its stopping test, E(j-1) - E(j-2) < eps, holds at once for any falling error: the loop
 *     here stops when the improvement E(j-1) - E(j) drops below eps (or after max_iter rounds);
 *   - the text says z is rounded after the relaxation, the formula omits the rounding: rounded here;
 *   - the candidate of a shrink step is its lowest-error iterate, and a z(0) outside [0, 2^b - 1]
 *     is pulled into that range (the code format has no other zero points).
 * bits is a parameter so that a 2-bit example can be worked by hand; the method uses b = 4.
 * Outputs: u [N,K] codes, delta [N] (double), zero [N], err [N] = final row error (not squared). */
void oracle_bgr_quantize(const double* wt, int64_t N, int64_t K, int bits, int n_steps, double eps, int max_iter,
                         uint8_t* u, double* delta, int32_t* zero, double* err) {
    const double levels = (double)((1 << bits) - 1);
#pragma omp parallel for schedule(static)
    for (int64_t n = 0; n < N; ++n) {
        const double* w = wt + n * K;
        double lo = w[0], hi = w[0], mean = 0.0;
        for (int64_t k = 0; k < K; ++k) { if (w[k] < lo) lo = w[k]; if (w[k] > hi) hi = w[k]; mean += w[k]; }
        mean /= (double)K;
        double best_e2 = INFINITY, best_d = 1.0, best_z = 0.0;
        const double step = (hi - lo) / (double)n_steps;
        for (int i = 1; 2 * i < n_steps && hi > lo; ++i) {
            const double lo_c = lo + i * step, hi_c = hi - i * step;   /* min and max of the clipped row */
            double d = (hi_c - lo_c) / levels;
            double z = -nearbyint(lo_c / d);
            if (z < 0.0) z = 0.0;
            if (z > levels) z = levels;
            double qw, qq, sq;
            double e2 = bgr_row_quantize(w, K, levels, d, z, NULL, &qw, &qq, &sq);
            if (e2 < best_e2) { best_e2 = e2; best_d = d; best_z = z; }
            for (int j = 1; j <= max_iter; ++j) {
                if (!(qq > 0.0) || !(qw > 0.0)) break;      /* no usable least-squares step */
                const double d1 = qw / qq;
                double z1 = nearbyint(sq / (double)K - mean / d1);
                if (z1 < 0.0) z1 = 0.0;
                if (z1 > levels) z1 = levels;
                const double e2_1 = bgr_row_quantize(w, K, levels, d1, z1, NULL, &qw, &qq, &sq);
                const double improvement = sqrt(e2) - sqrt(e2_1);
                d = d1; z = z1; e2 = e2_1;
                if (e2 < best_e2) { best_e2 = e2; best_d = d; best_z = z; }
                if (improvement < eps) break;
            }
        }
        if (!(best_e2 < INFINITY)) {                            /* constant row, or n_steps < 3 */
            best_d = (fabs(hi) > 0.0) ? fabs(hi) : 1.0;
            best_z = 0.0;
            if (hi > lo) { best_d = (hi - lo) / levels; best_z = -nearbyint(lo / best_d); if (best_z < 0.0) best_z = 0.0; if (best_z > levels) best_z = levels; }
            best_e2 = bgr_row_quantize(w, K, levels, best_d, best_z, NULL, NULL, NULL, NULL);
        }
        best_e2 = bgr_row_quantize(w, K, levels, best_d, best_z, u + n * K, NULL, NULL, NULL);
        delta[n] = best_d;
        zero[n] = (int32_t)best_z;
        err[n] = sqrt(best_e2);
    }
}

/* The error of the plain MinMax grid of Sec. 3.1 for every row, for comparisons with the above. */
void oracle_minmax_row_error(const double* wt, int64_t N, int64_t K, int bits, double* err) {
    const double levels = (double)((1 << bits) - 1);
#pragma omp parallel for schedule(static)
    for (int64_t n = 0; n < N; ++n) {
        const double* w = wt + n * K;
        double lo = w[0], hi = w[0];
        for (int64_t k = 1; k < K; ++k) { if (w[k] < lo) lo = w[k]; if (w[k] > hi) hi = w[k]; }
        double d = (hi - lo) / levels;
        if (!(d > 0.0)) { err[n] = 0.0; continue; }
        double z = -nearbyint(lo / d);
        if (z < 0.0) z = 0.0;
        if (z > levels) z = levels;
        err[n] = sqrt(bgr_row_quantize(w, K, levels, d, z, NULL, NULL, NULL, NULL));
    }
}

/* ---------------------------------------------------------------- integer GEMM */

/* acc_in = sum_k c_ik * (u_nk - z_n)   (the integer core of Y = X^ Lambda W^^T, Eq. 10).
 * Accumulated in 64 bits; returns the number of results that do not fit in int32
 * (0 for every shape this method allows). */
int64_t oracle_int_gemm(const int32_t* c, const uint8_t* u, const int32_t* zero,
                        int64_t M, int64_t N, int64_t K, int32_t* acc) {
    int64_t overflow = 0;
#pragma omp parallel for schedule(static) reduction(+ : overflow)
    for (int64_t i = 0; i < M; ++i) {
        for (int64_t n = 0; n < N; ++n) {
            int64_t s = 0;
            for (int64_t k = 0; k < K; ++k)
                s += (int64_t)c[i * K + k] * ((int64_t)u[n * K + k] - (int64_t)zero[n]);
            if (s > INT32_MAX || s < INT32_MIN) overflow += 1;
            acc[i * N + n] = (int32_t)s;
        }
    }
    return overflow;
}

/* ---------------------------------------------------------------- dequantizing epilogue */

/* tanh-form GELU: 0.5 y (1 + tanh( sqrt(2/pi) (y + 0.044715 y^3) )). */
double oracle_gelu_tanh(double y) {
    const double c = 0.79788456080286535588; /* sqrt(2/pi) */
    return 0.5 * y * (1.0 + tanh(c * (y + 0.044715 * y * y * y)));
}

/* y_in = bf16( acc_in * s_i * Delta_n + bias_n )   (DeQuant of Sec. 3.1 applied to
 * both factors of Eq. 10's product; s_i and Delta_n are the stored binary32 values).
 * act == 1: the rounded value then goes through GELU-tanh (evaluated in fp64 on the
 * bf16 value) and is rounded to bf16 again, i.e. "GELU in bf16" on the layer output. */
void oracle_epilogue(const int32_t* acc, const float* scale, const float* delta,
                     const uint16_t* bias_or_null, int act, int64_t M, int64_t N, uint16_t* y) {
#pragma omp parallel for schedule(static)
    for (int64_t i = 0; i < M; ++i) {
        for (int64_t n = 0; n < N; ++n) {
            double v = (double)acc[i * N + n] * (double)scale[i] * (double)delta[n];
            if (bias_or_null) v += oracle_bf16_to_double(bias_or_null[n]);
            uint16_t h = oracle_double_to_bf16(v);
            if (act == 1) h = oracle_double_to_bf16(oracle_gelu_tanh(oracle_bf16_to_double(h)));
            y[i * N + n] = h;
        }
    }
}

/* The tail of the epilogue for values already dequantized in fp64 (used by the block-wise
 * variant, whose sum over blocks is formed before): y = bf16(v + bias) [GELU, bf16 again]. */
void oracle_round_output(const double* v, const uint16_t* bias_or_null, int act, int64_t M, int64_t N, uint16_t* y) {
#pragma omp parallel for schedule(static)
    for (int64_t i = 0; i < M; ++i)
        for (int64_t n = 0; n < N; ++n) {
            double t = v[i * N + n];
            if (bias_or_null) t += oracle_bf16_to_double(bias_or_null[n]);
            uint16_t h = oracle_double_to_bf16(t);
            if (act == 1) h = oracle_double_to_bf16(oracle_gelu_tanh(oracle_bf16_to_double(h)));
            y[i * N + n] = h;
        }
}

/* The exact product the method approximates, Y = X W^T in fp64 (Sec. 3.2), for the
 * invariance and convergence checks. */
void oracle_exact_linear(const double* x, const double* w, int64_t M, int64_t N, int64_t K, double* y) {
#pragma omp parallel for schedule(static)
    for (int64_t i = 0; i < M; ++i)
        for (int64_t n = 0; n < N; ++n) {
            double s = 0.0;
            for (int64_t k = 0; k < K; ++k) s += x[i * K + k] * w[n * K + k];
            y[i * N + n] = s;
        }
}
