/*
 * CPU oracle for the BWLA W1AX linear layer.  TEST INFRASTRUCTURE ONLY.
 *
 * A plain, slow, step-by-step statement of what the layer computes, in fp64 and
 * int64, written from the paper.  It shares no code with the CUDA library and is
 * never called from the product path: only tests, the smoke check and the CPU
 * baseline leg of the benchmark load it.
 *
 * The paper never prints the inference-time forward of the quantised layer; it
 * is assembled from:
 *   - the weight format, Eq. 1-4 (row-wise mu_i, delta_i, Sign, W_deq);
 *   - the Kronecker evaluation of R = R1 (x) R2 on a reshaped vector
 *     (Sec. 3.1 "Orthogonal-Kronecker Transformation"; App. A.2 "Matrix
 *     Formulation and Kronecker Structure");
 *   - forward equivalence under orthogonal R (Sec. 1, Sec. 3.1): W x = (W R)(R^T x);
 *   - the PSP residual M = A B with W_res = W - M (Sec. 3.2; App. A.2 "Residual
 *     Modeling"), hence W x = (W - M) x + A (B x);
 *   - per-token activation quantisation (Sec. 4.1 "Implementation Details").
 *
 * Parity pins: every function below is pinned by tests/test_oracle_pins.py against
 * brute-force Kronecker products, closed forms and exact special cases.  The
 * absolute output values on the seeded configurations are "parity unpinned":
 * the paper prints no worked input/output example of a linear layer.
 *
 * Layouts (all row-major): x bf16 bits [M][ldx]; P1 [n1][n1], P2 [n2][n2] fp32;
 * packed uint32 [N][K/32], weight k of row n is bit (k & 31) of word k >> 5,
 * bit 1 <=> +1; alpha, mu fp32 [N]; U bf16 [N][r]; V bf16 [r][K].
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

static double bf16_to_f64(uint16_t b) {
    uint32_t u = (uint32_t)b << 16;
    float f;
    memcpy(&f, &u, 4);
    return (double)f;
}

/* fp64 -> bf16, round to nearest, ties to even, straight from the double (no fp32 detour). */
static uint16_t f64_to_bf16(double d) {
    if (isnan(d)) return 0x7FC0;
    if (d == 0.0) return signbit(d) ? 0x8000 : 0x0000;
    if (isinf(d)) return signbit(d) ? 0xFF80 : 0x7F80;
    int e;
    (void)frexp(d, &e);          /* |d| = m * 2^e, m in [0.5, 1) */
    int q = e - 8;               /* 8 significant bits -> quantum 2^(e-8) */
    if (q < -133) q = -133;      /* bf16 subnormal quantum */
    double r = nearbyint(ldexp(d, -q)); /* default rounding mode: ties to even */
    double v = ldexp(r, q);
    if (fabs(v) >= ldexp(1.0, 128)) return signbit(d) ? 0xFF80 : 0x7F80;
    float f = (float)v;          /* exact: v has <= 8 significant bits */
    uint32_t u;
    memcpy(&u, &f, 4);
    return (uint16_t)(u >> 16);
}

void bwla_oracle_bf16_round(const double* in, int64_t n, uint16_t* out) {
    for (int64_t i = 0; i < n; ++i) out[i] = f64_to_bf16(in[i]);
}

/* Alg. 1 (Kronecker dimension factorisation): largest divisor a <= floor(sqrt(n)); n2 = a, n1 = n / a. */
void bwla_oracle_kron_factor(int64_t n, int64_t* n1, int64_t* n2) {
    int64_t a = (int64_t)floor(sqrt((double)n));
    while ((a + 1) * (a + 1) <= n) ++a;  /* guard the floating sqrt */
    while (a * a > n) --a;
    while (a > 1 && n % a != 0) --a;
    *n2 = a;
    *n1 = n / a;
}

/* Eq. 1: mu_i = mean_j W_ij, delta_i = mean_j |W_ij - mu_i| (centre = 0 skips the shift). */
void bwla_oracle_row_stats(const float* W, int64_t N, int64_t K, int centre, double* mu, double* delta) {
    for (int64_t n = 0; n < N; ++n) {
        double m = 0.0;
        if (centre) {
            for (int64_t k = 0; k < K; ++k) m += (double)W[n * K + k];
            m /= (double)K;
        }
        double d = 0.0;
        for (int64_t k = 0; k < K; ++k) d += fabs((double)W[n * K + k] - m);
        mu[n] = m;
        delta[n] = d / (double)K;
    }
}

/* Eq. 2-3: Sign(x) = +1 iff x > 0 (so 0, -0.0 and NaN give -1); bit 1 <=> +1, LSB-first in each word. */
void bwla_oracle_pack_signs(const float* W, int64_t N, int64_t K, int64_t ldw, uint32_t* packed) {
    int64_t words = K / 32;
    for (int64_t n = 0; n < N; ++n) {
        for (int64_t w = 0; w < words; ++w) packed[n * words + w] = 0u;
        for (int64_t k = 0; k < K; ++k)
            if (W[n * ldw + k] > 0.0f) packed[n * words + (k >> 5)] |= (1u << (k & 31));
    }
}

/* Same rule on bf16 input. */
void bwla_oracle_pack_signs_bf16(const uint16_t* W, int64_t N, int64_t K, int64_t ldw, uint32_t* packed) {
    int64_t words = K / 32;
    for (int64_t n = 0; n < N; ++n) {
        for (int64_t w = 0; w < words; ++w) packed[n * words + w] = 0u;
        for (int64_t k = 0; k < K; ++k)
            if (bf16_to_f64(W[n * ldw + k]) > 0.0) packed[n * words + (k >> 5)] |= (1u << (k & 31));
    }
}

void bwla_oracle_unpack_signs(const uint32_t* packed, int64_t N, int64_t K, int8_t* s) {
    int64_t words = K / 32;
    for (int64_t n = 0; n < N; ++n)
        for (int64_t k = 0; k < K; ++k)
            s[n * K + k] = ((packed[n * words + (k >> 5)] >> (k & 31)) & 1u) ? 1 : -1;
}

/*
 * OKT applied to an activation row (Sec. 3.1; App. A.2 Kronecker identity):
 * X = reshape(x_t, n1 x n2) row-major, Y = P1^T X P2, y_t = flatten(Y) row-major.
 * Evaluated as Z = X P2, then Y = P1^T Z, all in fp64.
 */
void bwla_oracle_rotate(const uint16_t* x, int64_t M, int64_t K, int64_t ldx,
                        const float* P1, int64_t n1, const float* P2, int64_t n2, double* Y) {
#pragma omp parallel for schedule(dynamic, 1)
    for (int64_t t = 0; t < M; ++t) {
        double* Z = (double*)malloc(sizeof(double) * (size_t)K);
        double* X = (double*)malloc(sizeof(double) * (size_t)K);
        for (int64_t k = 0; k < K; ++k) X[k] = bf16_to_f64(x[t * ldx + k]);
        for (int64_t a = 0; a < n1; ++a)
            for (int64_t d = 0; d < n2; ++d) {
                double s = 0.0;
                for (int64_t b = 0; b < n2; ++b) s += X[a * n2 + b] * (double)P2[b * n2 + d];
                Z[a * n2 + d] = s;
            }
        for (int64_t c = 0; c < n1; ++c)
            for (int64_t d = 0; d < n2; ++d) {
                double s = 0.0;
                for (int64_t a = 0; a < n1; ++a) s += (double)P1[a * n1 + c] * Z[a * n2 + d];
                Y[t * K + c * n2 + d] = s;
            }
        free(Z);
        free(X);
    }
}

/*
 * Final binarisation in the rotated coordinates (Alg. 2, last step, with Eq. 1-3): X = W_res R with R = P1 (x) P2,
 * i.e. every row of W_res = W - M goes through the same map as an activation row, X_n = flatten(P1^T reshape(w_n) P2);
 * then per output row n: mu_n = mean_k X_nk, alpha_n = mean_k |X_nk - mu_n|, bit_nk = (X_nk - mu_n > 0).
 * (The centring matrix H of Alg. 2 is the subtraction of the row mean; the mean is kept as the row shift of Eq. 4.)
 * W_res is fp32 [N][K], widened exactly.  X (fp64 [N][K]) is returned for the tests' near-zero window.
 */
void bwla_oracle_binarize(const float* W, int64_t N, int64_t K, const float* P1, int64_t n1, const float* P2, int64_t n2,
                          double* X, double* mu, double* alpha, uint32_t* packed) {
    int64_t words = K / 32;
#pragma omp parallel for schedule(dynamic, 1)
    for (int64_t n = 0; n < N; ++n) {
        double* Z = (double*)malloc(sizeof(double) * (size_t)K);
        const float* w = W + n * K;
        for (int64_t a = 0; a < n1; ++a)
            for (int64_t d = 0; d < n2; ++d) {
                double s = 0.0;
                for (int64_t b = 0; b < n2; ++b) s += (double)w[a * n2 + b] * (double)P2[b * n2 + d];
                Z[a * n2 + d] = s;
            }
        double* x = X + n * K;
        for (int64_t c = 0; c < n1; ++c)
            for (int64_t d = 0; d < n2; ++d) {
                double s = 0.0;
                for (int64_t a = 0; a < n1; ++a) s += (double)P1[a * n1 + c] * Z[a * n2 + d];
                x[c * n2 + d] = s;
            }
        free(Z);
        double m = 0.0;
        for (int64_t k = 0; k < K; ++k) m += x[k];
        m /= (double)K;
        double dsum = 0.0;
        for (int64_t k = 0; k < K; ++k) dsum += fabs(x[k] - m);
        mu[n] = m;
        alpha[n] = dsum / (double)K;
        for (int64_t wd = 0; wd < words; ++wd) packed[n * words + wd] = 0u;
        for (int64_t k = 0; k < K; ++k)
            if (x[k] - m > 0.0) packed[n * words + (k >> 5)] |= (1u << (k & 31));
    }
}

static double round_half_even(double t) {
    double f = floor(t);
    double d = t - f;
    if (d > 0.5) return f + 1.0;
    if (d < 0.5) return f;
    return (fmod(f, 2.0) == 0.0) ? f : f + 1.0;
}

/*
 * Per-token symmetric INT-b quantiser (Sec. 4.1 says per-token; symmetric, restricted range
 * and round-half-to-even are this build's reading).  qmax = 2^(b-1) - 1.
 *   amax = max_k |y_k|;  amax == 0: scale = 1, codes 0.
 *   decision == 0 (definition, fp64): scale = amax / qmax, t_k = y_k / scale.
 *   decision == 1 (fp32 arithmetic, the precision a float kernel decides in):
 *       amax, y_k taken as float; inv = fl32(qmax / amax); t_k = fl32(y_k * inv);
 *       emitted scale = fl32(amax / qmax).
 *   q_k = clamp(rne(t_k), -qmax, qmax).
 * dist[k] (optional) = | t_k - (floor(t_k) + 1/2) |, the distance to the nearest rounding boundary.
 * qsum[t] (optional) = sum_k q_k.
 */
void bwla_oracle_quantize(const double* Y, int64_t M, int64_t K, int bits, int decision,
                          int8_t* codes, float* scales, double* dist, int64_t* qsum) {
    const double qmax = (double)((1 << (bits - 1)) - 1);
    for (int64_t t = 0; t < M; ++t) {
        const double* y = Y + t * K;
        double amax = 0.0;
        for (int64_t k = 0; k < K; ++k) {
            double a = fabs(y[k]);
            if (a > amax) amax = a;
        }
        int64_t s = 0;
        if (amax == 0.0) {
            scales[t] = 1.0f;
            for (int64_t k = 0; k < K; ++k) {
                codes[t * K + k] = 0;
                if (dist) dist[t * K + k] = 0.5;
            }
            if (qsum) qsum[t] = 0;
            continue;
        }
        double scale64 = amax / qmax;
        volatile float amax32 = (float)amax;
        volatile float inv32 = (float)qmax / amax32;
        volatile float scale32 = amax32 / (float)qmax;
        scales[t] = decision ? scale32 : (float)scale64;
        for (int64_t k = 0; k < K; ++k) {
            double tk;
            if (decision) {
                volatile float yf = (float)y[k];
                volatile float tf = yf * inv32;
                tk = (double)tf;
            } else {
                tk = y[k] / scale64;
            }
            double q = round_half_even(tk);
            if (q > qmax) q = qmax;
            if (q < -qmax) q = -qmax;
            codes[t * K + k] = (int8_t)q;
            s += (int64_t)q;
            if (dist) dist[t * K + k] = fabs(tk - (floor(tk) + 0.5));
        }
        if (qsum) qsum[t] = s;
    }
}

/*
 * Per-token asymmetric INT-b quantiser: Sec. 4.1 states "per-token asymmetric quantization for activations" and gives no
 * constants; this is the common definition with an integer zero point, and zero kept representable:
 *   lo = min(0, min_k y_k), hi = max(0, max_k y_k), L = 2^b - 1 levels above code 0
 *   lo == hi (an all-zero row): scale = 1, zero = 0, all codes 0
 *   scale = (hi - lo) / L;  zero = clamp(rne(-lo / scale), 0, L);  u_k = clamp(rne(y_k / scale) + zero, 0, L)
 *   the value a code stands for is scale * (u_k - zero); y = 0 maps to u = zero exactly.
 *   decision == 1 (the precision a float kernel decides in): range = fl32(hi - lo), inv = fl32(L / range),
 *   scale = fl32(range / L), zero = rne(fl32(-lo * inv)), u_k = rne(fl32(y_k * inv)) + zero.
 * dist[k] (optional) = distance of y_k / scale to the nearest rounding boundary; dist_zero[t] the same for -lo / scale.
 */
void bwla_oracle_quantize_asym(const double* Y, int64_t M, int64_t K, int bits, int decision,
                               uint8_t* codes, float* scales, int32_t* zeros, double* dist, double* dist_zero) {
    const double L = (double)((1 << bits) - 1);
    for (int64_t t = 0; t < M; ++t) {
        const double* y = Y + t * K;
        double lo = 0.0, hi = 0.0;
        for (int64_t k = 0; k < K; ++k) {
            if (y[k] < lo) lo = y[k];
            if (y[k] > hi) hi = y[k];
        }
        if (lo == hi) {
            scales[t] = 1.0f;
            zeros[t] = 0;
            if (dist_zero) dist_zero[t] = 0.5;
            for (int64_t k = 0; k < K; ++k) {
                codes[t * K + k] = 0;
                if (dist) dist[t * K + k] = 0.5;
            }
            continue;
        }
        double scale64 = (hi - lo) / L;
        volatile float lo32 = (float)lo, hi32 = (float)hi;
        volatile float range32 = hi32 - lo32;
        volatile float inv32 = (float)L / range32;
        volatile float scale32 = range32 / (float)L;
        double tz;
        if (decision) {
            volatile float zf = -lo32 * inv32;
            tz = (double)zf;
        } else {
            tz = -lo / scale64;
        }
        double z = round_half_even(tz);
        if (z < 0.0) z = 0.0;
        if (z > L) z = L;
        zeros[t] = (int32_t)z;
        scales[t] = decision ? scale32 : (float)scale64;
        if (dist_zero) dist_zero[t] = fabs(tz - (floor(tz) + 0.5));
        for (int64_t k = 0; k < K; ++k) {
            double tk;
            if (decision) {
                volatile float yf = (float)y[k];
                volatile float tf = yf * inv32;
                tk = (double)tf;
            } else {
                tk = y[k] / scale64;
            }
            double u = round_half_even(tk) + z;
            if (u < 0.0) u = 0.0;
            if (u > L) u = L;
            codes[t * K + k] = (uint8_t)u;
            if (dist) dist[t * K + k] = fabs(tk - (floor(tk) + 0.5));
        }
    }
}

/* acc[t][n] = sum_k s[n][k] * (u[t][k] - zero[t]) for unsigned codes with a per-token zero point, int64; and
 * rsum[t] = sum_k (u[t][k] - zero[t]). */
void bwla_oracle_gemm_asym(const uint8_t* codes, const int32_t* zeros, const uint32_t* packed, int64_t M, int64_t N,
                           int64_t K, int64_t* acc, int64_t* rsum) {
    int64_t words = K / 32;
    for (int64_t t = 0; t < M; ++t) {
        int64_t s = 0;
        for (int64_t k = 0; k < K; ++k) s += (int64_t)codes[t * K + k] - (int64_t)zeros[t];
        rsum[t] = s;
    }
#pragma omp parallel for schedule(static)
    for (int64_t n = 0; n < N; ++n)
        for (int64_t t = 0; t < M; ++t) {
            int64_t a = 0;
            for (int64_t k = 0; k < K; ++k) {
                int64_t r = (int64_t)codes[t * K + k] - (int64_t)zeros[t];
                a += ((packed[n * words + (k >> 5)] >> (k & 31)) & 1u) ? r : -r;
            }
            acc[t * N + n] = a;
        }
}

/* acc[t][n] = sum_k s[n][k] * q[t][k], s = +-1 read from the packed bits, int64. */
void bwla_oracle_gemm(const int8_t* codes, const uint32_t* packed, int64_t M, int64_t N, int64_t K,
                      int64_t* acc) {
    int64_t words = K / 32;
#pragma omp parallel for schedule(static)
    for (int64_t n = 0; n < N; ++n)
        for (int64_t t = 0; t < M; ++t) {
            int64_t a = 0;
            for (int64_t k = 0; k < K; ++k) {
                int64_t s = ((packed[n * words + (k >> 5)] >> (k & 31)) & 1u) ? 1 : -1;
                a += s * (int64_t)codes[t * K + k];
            }
            acc[t * N + n] = a;
        }
}

/* PSP branch (Sec. 3.2; App. A.2): T = V x_t (r values), L = U T, on the un-rotated activation, fp64. */
void bwla_oracle_lowrank(const uint16_t* x, int64_t M, int64_t K, int64_t ldx,
                         const uint16_t* U, const uint16_t* V, int64_t N, int64_t r, double* L) {
#pragma omp parallel for schedule(static)
    for (int64_t t = 0; t < M; ++t) {
        double* T = (double*)malloc(sizeof(double) * (size_t)(r > 0 ? r : 1));
        for (int64_t j = 0; j < r; ++j) {
            double s = 0.0;
            for (int64_t k = 0; k < K; ++k) s += bf16_to_f64(V[j * K + k]) * bf16_to_f64(x[t * ldx + k]);
            T[j] = s;
        }
        for (int64_t n = 0; n < N; ++n) {
            double s = 0.0;
            for (int64_t j = 0; j < r; ++j) s += bf16_to_f64(U[n * r + j]) * T[j];
            L[t * N + n] = s;
        }
        free(T);
    }
}

/*
 * Dequantisation and sum (Eq. 4 applied to the integer accumulator):
 * y[t][n] = alpha[n] * scale[t] * acc[t][n] + L[t][n] (+ mu[n] * scale[t] * qsum[t] when mu is given).
 */
void bwla_oracle_epilogue(const int64_t* acc, const float* scales, const float* alpha, const float* mu,
                          const int64_t* qsum, const double* L, int64_t M, int64_t N,
                          double* y, uint16_t* y_bf16) {
    for (int64_t t = 0; t < M; ++t)
        for (int64_t n = 0; n < N; ++n) {
            double v = (double)alpha[n] * (double)scales[t] * (double)acc[t * N + n];
            if (L) v += L[t * N + n];
            if (mu) v += (double)mu[n] * (double)scales[t] * (double)qsum[t];
            y[t * N + n] = v;
            if (y_bf16) y_bf16[t * N + n] = f64_to_bf16(v);
        }
}

/*
 * The weight-only operating point, W1A16 (Table 1, upper half: binarised weights, 16-bit activations): the rotated
 * activation is not quantised to integers but kept as a 16-bit value, here bf16 (round to nearest even of the fp64
 * rotation), and meets the signs directly:
 *   yhat = bf16(Y),  acc[t][n] = sum_k s[n][k] * yhat[t][k],  y[t][n] = alpha[n] * acc[t][n] + L[t][n] (+ mu[n] * sum_k yhat[t][k]).
 * Y (fp64 [M][K]) comes from bwla_oracle_rotate, L (fp64 [M][N], may be NULL) from bwla_oracle_lowrank.
 */
void bwla_oracle_a16(const double* Y, int64_t M, int64_t K, const uint32_t* packed, const float* alpha, const float* mu,
                     const double* L, int64_t N, uint16_t* yhat, double* acc, double* y) {
    int64_t words = K / 32;
    for (int64_t i = 0; i < M * K; ++i) yhat[i] = f64_to_bf16(Y[i]);
#pragma omp parallel for schedule(static)
    for (int64_t n = 0; n < N; ++n)
        for (int64_t t = 0; t < M; ++t) {
            double a = 0.0, sum = 0.0;
            for (int64_t k = 0; k < K; ++k) {
                double v = bf16_to_f64(yhat[t * K + k]);
                a += ((packed[n * words + (k >> 5)] >> (k & 31)) & 1u) ? v : -v;
                sum += v;
            }
            acc[t * N + n] = a;
            double out = (double)alpha[n] * a;
            if (L) out += L[t * N + n];
            if (mu) out += (double)mu[n] * sum;
            y[t * N + n] = out;
        }
}

/* The whole layer, steps in order.  Optional outputs may be NULL.  Returns 0, or 1 if an accumulator leaves int32. */
int bwla_oracle_linear(const uint16_t* x, int64_t M, int64_t K, int64_t ldx,
                       const float* P1, int64_t n1, const float* P2, int64_t n2, int bits, int decision,
                       const uint32_t* packed, const float* alpha, const float* mu,
                       const uint16_t* U, const uint16_t* V, int64_t r, int64_t N,
                       double* y, uint16_t* y_bf16,
                       double* Y_out, int8_t* codes_out, float* scales_out, int64_t* acc_out) {
    double* Y = Y_out ? Y_out : (double*)malloc(sizeof(double) * (size_t)(M * K));
    int8_t* codes = codes_out ? codes_out : (int8_t*)malloc((size_t)(M * K));
    float* scales = scales_out ? scales_out : (float*)malloc(sizeof(float) * (size_t)M);
    int64_t* acc = acc_out ? acc_out : (int64_t*)malloc(sizeof(int64_t) * (size_t)(M * N));
    int64_t* qsum = (int64_t*)malloc(sizeof(int64_t) * (size_t)M);
    double* L = NULL;
    int overflow = 0;

    bwla_oracle_rotate(x, M, K, ldx, P1, n1, P2, n2, Y);
    bwla_oracle_quantize(Y, M, K, bits, decision, codes, scales, NULL, qsum);
    bwla_oracle_gemm(codes, packed, M, N, K, acc);
    for (int64_t i = 0; i < M * N; ++i)
        if (acc[i] > INT32_MAX || acc[i] < INT32_MIN) overflow = 1;
    if (r > 0) {
        L = (double*)malloc(sizeof(double) * (size_t)(M * N));
        bwla_oracle_lowrank(x, M, K, ldx, U, V, N, r, L);
    }
    bwla_oracle_epilogue(acc, scales, alpha, mu, qsum, L, M, N, y, y_bf16);

    if (L) free(L);
    free(qsum);
    if (!acc_out) free(acc);
    if (!scales_out) free(scales);
    if (!codes_out) free(codes);
    if (!Y_out) free(Y);
    return overflow;
}

int bwla_oracle_num_threads(void) {
#ifdef _OPENMP
    extern int omp_get_max_threads(void);
    return omp_get_max_threads();
#else
    return 1;
#endif
}
