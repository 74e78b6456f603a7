/*
 * DiRotQ rotation-aware W4A4 linear layer -- plain CPU oracle (TEST INFRASTRUCTURE).
 *
 * This file is a checker, not a product path: only the tests, the smoke check and
 * the benchmark's CPU-baseline leg may call it.  It shares no code with the CUDA
 * library.  Everything is written as the definition reads: fp64 arithmetic,
 * scalar quantizer, naive triple-loop integer GEMM, no blocking, no fusion.
 *
 * Method (paper Sec. 4.2, Eq. 5):  Y ~= [X U_h , Q4(X~_l)] [W~_h ; Q4(W~_l)]
 *   with  V = [U_h , U_l R]  (called Q here),  W~ = V^T W  folded offline,
 *   Q4 = symmetric 4-bit per-group quantizer of Eq. 1 with z = 0,
 *   s = max|.|/q_max, q_max = 2^(4-1)-1 = 7  (Sec. 3), groups along K (Sec. 5.1:
 *   group size 64, 16-bit scales).
 *
 * "Deployed" rounding points (where the product stores a narrow type, the oracle
 * rounds at the same point; everything in between is fp64):
 *   - x and the online rotation matrix are bf16 values,
 *   - the r high-precision coefficients and the r high rows of W~ are bf16,
 *   - every scale is a bf16 value and the rounded scale is used to divide,
 *   - the output is bf16.
 * Readings taken where the paper is silent:
 *   groups are counted from the first low-precision column; the last group may be
 *   ragged; rounding is half-to-even; codes are clipped to [-7, 7]; a group whose
 *   absmax is zero has scale 0 and codes 0; bias is added before the final rounding.
 *
 * Parity pins: see tests/test_oracle_*.py (orthogonality, Eq. 4 identity, brute
 * force nearest-level search, exhaustive integer products, textbook RTN special
 * case, integer path == dequantized path).  The choices above that no printed
 * value fixes (group axis/alignment, bf16 scales, tie rule, clip range) are
 * "parity unpinned" against the authors' implementation.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

/* ---------- bf16 <-> double ------------------------------------------------- */

double dq_bf16_to_double(uint16_t h) {
    uint32_t u = ((uint32_t)h) << 16;
    float f;
    memcpy(&f, &u, sizeof f);
    return (double)f;
}

/* Round an fp64 value straight to bf16 (8 significant bits), nearest, ties to even. */
uint16_t dq_double_to_bf16(double v) {
    if (v != v) return 0x7FC0;
    uint16_t sign = signbit(v) ? 0x8000 : 0;
    double a = fabs(v);
    if (a == 0.0) return sign;
    if (isinf(a)) return sign | 0x7F80;
    int e = ilogb(a);                 /* 2^e <= a < 2^(e+1) */
    if (e < -126) e = -126;           /* subnormal bf16: fixed quantum 2^-133 */
    double quantum = ldexp(1.0, e - 7);
    double m = rint(a / quantum);     /* default rounding mode: ties to even */
    double r = m * quantum;           /* exactly representable in float */
    float f = (float)r;
    if (isinf(f) || r > 3.3895313892515355e38) return sign | 0x7F80;
    uint32_t u;
    memcpy(&u, &f, sizeof u);
    return sign | (uint16_t)(u >> 16);
}

void dq_round_bf16(const double* src, uint16_t* dst, int64_t n) {
#pragma omp parallel for schedule(static)
    for (int64_t i = 0; i < n; ++i) dst[i] = dq_double_to_bf16(src[i]);
}

/* ---------- Eq. 1, symmetric, one group -------------------------------------- */

/* v[0..n): the group's real elements (stride in elements).  Writes the bf16 scale,
 * the codes, and (if t != NULL) the pre-rounding quotients v/s. */
void dq_quantize_group(const double* v, int n, int64_t stride, uint16_t* scale_bits, int8_t* codes,
                       int64_t code_stride, double* t, int64_t t_stride) {
    double a = 0.0;
    for (int i = 0; i < n; ++i) {
        double x = fabs(v[i * stride]);
        if (x > a) a = x;
    }
    uint16_t sb = (a == 0.0) ? 0 : dq_double_to_bf16(a / 7.0);   /* s = max|X| / q_max */
    double s = dq_bf16_to_double(sb);
    *scale_bits = sb;
    for (int i = 0; i < n; ++i) {
        double q = 0.0, ti = 0.0;
        if (s != 0.0) {
            ti = v[i * stride] / s;
            q = rint(ti);                 /* half to even */
            if (q > 7.0) q = 7.0;         /* clip to [q_min, q_max] */
            if (q < -7.0) q = -7.0;
        }
        codes[i * code_stride] = (int8_t)q;
        if (t) t[i * t_stride] = ti;
    }
}

/* ---------- offline: fold and weight quantization (Eq. 5, left factor) -------- */

/* Wt[K,N] = Q^T W   (Q[K,K] column j = basis vector j; W[K,N]) */
void dq_fold(const double* Q, const double* W, double* Wt, int K, int N) {
#pragma omp parallel for schedule(static)
    for (int i = 0; i < K; ++i) {
        double* out = Wt + (int64_t)i * N;
        for (int n = 0; n < N; ++n) out[n] = 0.0;
        for (int k = 0; k < K; ++k) {
            double q = Q[(int64_t)k * K + i];
            const double* w = W + (int64_t)k * N;
            for (int n = 0; n < N; ++n) out[n] += q * w[n];
        }
    }
}

/* Rows < r of Wt -> bf16 Wh[r,N].  Rows >= r: per (group, column) scale + codes.
 * wcodes[K_l,N], wscales[n_g,N], wt (optional) [K_l,N] pre-rounding quotients. */
void dq_prepare_weights(const double* Wt, int K, int N, int r, int G, uint16_t* Wh, int8_t* wcodes,
                        uint16_t* wscales, double* wt) {
    int K_l = K - r;
    int n_g = (K_l + G - 1) / G;
    dq_round_bf16(Wt, Wh, (int64_t)r * N);
#pragma omp parallel for schedule(static)
    for (int n = 0; n < N; ++n) {
        for (int g = 0; g < n_g; ++g) {
            int j0 = g * G;
            int len = (j0 + G <= K_l) ? G : (K_l - j0);
            dq_quantize_group(Wt + (int64_t)(r + j0) * N + n, len, N, wscales + (int64_t)g * N + n,
                              wcodes + (int64_t)j0 * N + n, N, wt ? wt + (int64_t)j0 * N + n : NULL, N);
        }
    }
}

/* ---------- online step 1: rotation  x~ = x Q_b  (Sec. 4.2) -------------------- */

void dq_rotate(const uint16_t* x_bits, const uint16_t* Qb_bits, double* xt, int M, int K) {
    double* Qd = (double*)malloc(sizeof(double) * (size_t)K * K);
    for (int64_t i = 0; i < (int64_t)K * K; ++i) Qd[i] = dq_bf16_to_double(Qb_bits[i]);
#pragma omp parallel for schedule(static)
    for (int m = 0; m < M; ++m) {
        double* out = xt + (int64_t)m * K;
        for (int c = 0; c < K; ++c) out[c] = 0.0;
        for (int k = 0; k < K; ++k) {
            double xv = dq_bf16_to_double(x_bits[(int64_t)m * K + k]);
            const double* q = Qd + (int64_t)k * K;
            for (int c = 0; c < K; ++c) out[c] += xv * q[c];
        }
    }
    free(Qd);
}

/* ---------- online steps 2-3: split, per-token per-group quantization ---------- */

/* xt[M,K] -> xh bf16 [M,r]; codes [M,K_l]; scales bf16 [M,n_g]; t (optional) [M,K_l] */
void dq_split_quantize(const double* xt, int M, int K, int r, int G, uint16_t* xh, int8_t* codes,
                       uint16_t* scales, double* t) {
    int K_l = K - r;
    int n_g = (K_l + G - 1) / G;
#pragma omp parallel for schedule(static)
    for (int m = 0; m < M; ++m) {
        const double* row = xt + (int64_t)m * K;
        for (int i = 0; i < r; ++i) xh[(int64_t)m * r + i] = dq_double_to_bf16(row[i]);
        for (int g = 0; g < n_g; ++g) {
            int j0 = g * G;
            int len = (j0 + G <= K_l) ? G : (K_l - j0);
            dq_quantize_group(row + r + j0, len, 1, scales + (int64_t)m * n_g + g,
                              codes + (int64_t)m * K_l + j0, 1, t ? t + (int64_t)m * K_l + j0 : NULL, 1);
        }
    }
}

/* ---------- online step 4: integer GEMM per group ------------------------------ */

/* P[g,m,n] = sum_{j in group g} qx[m,j] * qw[j,n]   (int32, naive triple loop) */
void dq_int_gemm(const int8_t* qx, const int8_t* qw, int32_t* P, int M, int K_l, int N, int G) {
    int n_g = (K_l + G - 1) / G;
#pragma omp parallel for schedule(static)
    for (int m = 0; m < M; ++m) {
        for (int g = 0; g < n_g; ++g) {
            int j0 = g * G;
            int j1 = (j0 + G <= K_l) ? j0 + G : K_l;
            for (int n = 0; n < N; ++n) {
                int32_t acc = 0;
                for (int j = j0; j < j1; ++j)
                    acc += (int32_t)qx[(int64_t)m * K_l + j] * (int32_t)qw[(int64_t)j * N + n];
                P[((int64_t)g * M + m) * N + n] = acc;
            }
        }
    }
}

/* ---------- online step 5: dequantize, add the 16-bit branch and the bias ------- */

/* y[m,n] = sum_g sx[m,g] sw[g,n] P[g,m,n] + sum_{i<r} xh[m,i] Wh[i,n] + bias[n]
 * y64 (optional): value before the final rounding; ybits: bf16 result. */
void dq_combine(const int32_t* P, const uint16_t* sx, const uint16_t* sw, const uint16_t* xh,
                const uint16_t* Wh, const uint16_t* bias, int M, int N, int r, int n_g, double* y64,
                uint16_t* ybits) {
#pragma omp parallel for schedule(static)
    for (int m = 0; m < M; ++m) {
        for (int n = 0; n < N; ++n) {
            double acc = 0.0;
            for (int g = 0; g < n_g; ++g)
                acc += dq_bf16_to_double(sx[(int64_t)m * n_g + g]) * dq_bf16_to_double(sw[(int64_t)g * N + n]) *
                       (double)P[((int64_t)g * M + m) * N + n];
            double lr = 0.0;
            for (int i = 0; i < r; ++i)
                lr += dq_bf16_to_double(xh[(int64_t)m * r + i]) * dq_bf16_to_double(Wh[(int64_t)i * N + n]);
            double v = acc + lr + (bias ? dq_bf16_to_double(bias[n]) : 0.0);
            if (y64) y64[(int64_t)m * N + n] = v;
            ybits[(int64_t)m * N + n] = dq_double_to_bf16(v);
        }
    }
}

/* =====================================================================================
 * Asymmetric activation quantization (paper Sec. 3, Eq. 1 with z = min X,
 * s = (max X - min X) / (q_max - q_min), q_min = 0, q_max = 2^4 - 1 = 15; Sec. 5.1: the 4-bit INT
 * setting quantizes activations asymmetrically, weights symmetrically).
 * Readings: both the scale and the zero-point are kept in 16 bits (bf16) and the ROUNDED values
 * are the ones that divide and dequantize; the range max - min is taken before any rounding; a
 * group whose elements are all equal has scale 0 and codes 0 (it dequantizes to z).
 * "Parity unpinned" against the authors' implementation.
 * ===================================================================================== */

/* One group: codes u in 0..15 with x ~ s*u + z.  t (optional): pre-rounding quotients (x - z)/s. */
void dq_quantize_group_asym(const double* v, int n, int64_t stride, uint16_t* scale_bits, uint16_t* zero_bits,
                            uint8_t* codes, int64_t code_stride, double* t, int64_t t_stride) {
    double lo = v[0], hi = v[0];
    for (int i = 1; i < n; ++i) {
        double x = v[i * stride];
        if (x < lo) lo = x;
        if (x > hi) hi = x;
    }
    uint16_t zb = dq_double_to_bf16(lo);                          /* z = min X */
    uint16_t sb = (hi == lo) ? 0 : dq_double_to_bf16((hi - lo) / 15.0);   /* s = (max - min)/(q_max - q_min) */
    double z = dq_bf16_to_double(zb), s = dq_bf16_to_double(sb);
    *scale_bits = sb;
    *zero_bits = zb;
    for (int i = 0; i < n; ++i) {
        double q = 0.0, ti = 0.0;
        if (s != 0.0) {
            ti = (v[i * stride] - z) / s;
            q = rint(ti);                  /* half to even */
            if (q > 15.0) q = 15.0;        /* clip to [q_min, q_max] */
            if (q < 0.0) q = 0.0;
        }
        codes[i * code_stride] = (uint8_t)q;
        if (t) t[i * t_stride] = ti;
    }
}

/* xt[M,K] -> xh bf16 [M,r]; codes u8 [M,K_l]; scales, zeros bf16 [M,n_g]; t (optional) [M,K_l] */
void dq_split_quantize_asym(const double* xt, int M, int K, int r, int G, uint16_t* xh, uint8_t* codes,
                            uint16_t* scales, uint16_t* zeros, double* t) {
    int K_l = K - r;
    int n_g = (K_l + G - 1) / G;
#pragma omp parallel for schedule(static)
    for (int m = 0; m < M; ++m) {
        const double* row = xt + (int64_t)m * K;
        for (int i = 0; i < r; ++i) xh[(int64_t)m * r + i] = dq_double_to_bf16(row[i]);
        for (int g = 0; g < n_g; ++g) {
            int j0 = g * G;
            int len = (j0 + G <= K_l) ? G : (K_l - j0);
            dq_quantize_group_asym(row + r + j0, len, 1, scales + (int64_t)m * n_g + g, zeros + (int64_t)m * n_g + g,
                                   codes + (int64_t)m * K_l + j0, 1, t ? t + (int64_t)m * K_l + j0 : NULL, 1);
        }
    }
}

/* Integer products with unsigned activation codes: P[g,m,n] = sum_{j in g} u[m,j] qw[j,n]. */
void dq_int_gemm_u(const uint8_t* ux, const int8_t* qw, int32_t* P, int M, int K_l, int N, int G) {
    int n_g = (K_l + G - 1) / G;
#pragma omp parallel for schedule(static)
    for (int m = 0; m < M; ++m) {
        for (int g = 0; g < n_g; ++g) {
            int j0 = g * G;
            int j1 = (j0 + G <= K_l) ? j0 + G : K_l;
            for (int n = 0; n < N; ++n) {
                int32_t acc = 0;
                for (int j = j0; j < j1; ++j)
                    acc += (int32_t)ux[(int64_t)m * K_l + j] * (int32_t)qw[(int64_t)j * N + n];
                P[((int64_t)g * M + m) * N + n] = acc;
            }
        }
    }
}

/* y[m,n] = sum_g sw[g,n] ( sx[m,g] P[g,m,n] + zx[m,g] C[g,n] ) + sum_{i<r} xh[m,i] Wh[i,n] + bias[n],
 * C[g,n] = sum_{j in g} qw[j,n]: the "additional z term" of the asymmetric case -- dequantizing
 * x^ = s u + z inside the product gives s * (u . qw) + z * (1 . qw) per group. */
void dq_combine_asym(const int32_t* P, const uint16_t* sx, const uint16_t* zx, const uint16_t* sw, const int8_t* qw,
                     const uint16_t* xh, const uint16_t* Wh, const uint16_t* bias, int M, int N, int K_l, int r, int G,
                     double* y64, uint16_t* ybits) {
    int n_g = (K_l + G - 1) / G;
#pragma omp parallel for schedule(static)
    for (int m = 0; m < M; ++m) {
        for (int n = 0; n < N; ++n) {
            double acc = 0.0;
            for (int g = 0; g < n_g; ++g) {
                int j0 = g * G;
                int j1 = (j0 + G <= K_l) ? j0 + G : K_l;
                int32_t c = 0;
                for (int j = j0; j < j1; ++j) c += (int32_t)qw[(int64_t)j * N + n];
                acc += dq_bf16_to_double(sw[(int64_t)g * N + n]) *
                       (dq_bf16_to_double(sx[(int64_t)m * n_g + g]) * (double)P[((int64_t)g * M + m) * N + n] +
                        dq_bf16_to_double(zx[(int64_t)m * n_g + g]) * (double)c);
            }
            double lr = 0.0;
            for (int i = 0; i < r; ++i)
                lr += dq_bf16_to_double(xh[(int64_t)m * r + i]) * dq_bf16_to_double(Wh[(int64_t)i * N + n]);
            double v = acc + lr + (bias ? dq_bf16_to_double(bias[n]) : 0.0);
            if (y64) y64[(int64_t)m * N + n] = v;
            ybits[(int64_t)m * N + n] = dq_double_to_bf16(v);
        }
    }
}

/* =====================================================================================
 * W4A8 (paper Sec. 5.1, "INT W4A8" rows of Table 1): 8-bit activations with one dynamic scale per
 * token, 4-bit weights with one static scale per output channel (Sec. 5.1 gives these two granularities
 * for its 8-bit settings).
 * Readings: symmetric on both sides (Eq. 1 with z = 0, q_max = 2^7 - 1 = 127 for the activations);
 * the token's scale covers its K - r low-precision coefficients and is kept as bf16, the rounded
 * value dividing and dequantizing; the weight side is Eq. 1 with one group spanning the whole
 * column, i.e. dq_prepare_weights with G = K - r.  "Parity unpinned" against the authors' code.
 * ===================================================================================== */

/* xt[M,K] -> xh bf16 [M,r]; codes int8 [M,K_l]; scales bf16 [M]; t (optional) [M,K_l] */
void dq_split_quantize_a8(const double* xt, int M, int K, int r, uint16_t* xh, int8_t* codes, uint16_t* scales, double* t) {
    int K_l = K - r;
#pragma omp parallel for schedule(static)
    for (int m = 0; m < M; ++m) {
        const double* row = xt + (int64_t)m * K;
        for (int i = 0; i < r; ++i) xh[(int64_t)m * r + i] = dq_double_to_bf16(row[i]);
        double a = 0.0;
        for (int j = 0; j < K_l; ++j) {
            double x = fabs(row[r + j]);
            if (x > a) a = x;
        }
        uint16_t sb = (a == 0.0) ? 0 : dq_double_to_bf16(a / 127.0);      /* s = max|X| / q_max */
        double s = dq_bf16_to_double(sb);
        scales[m] = sb;
        for (int j = 0; j < K_l; ++j) {
            double q = 0.0, tj = 0.0;
            if (s != 0.0) {
                tj = row[r + j] / s;
                q = rint(tj);
                if (q > 127.0) q = 127.0;
                if (q < -127.0) q = -127.0;
            }
            codes[(int64_t)m * K_l + j] = (int8_t)q;
            if (t) t[(int64_t)m * K_l + j] = tj;
        }
    }
}

/* ---------- plain fp64 product, used by the ideal (nothing quantized) mode ------ */

void dq_matmul(const double* A, const double* B, double* C, int M, int K, int N) {
#pragma omp parallel for schedule(static)
    for (int m = 0; m < M; ++m) {
        double* out = C + (int64_t)m * N;
        for (int n = 0; n < N; ++n) out[n] = 0.0;
        for (int k = 0; k < K; ++k) {
            double a = A[(int64_t)m * K + k];
            const double* b = B + (int64_t)k * N;
            for (int n = 0; n < N; ++n) out[n] += a * b[n];
        }
    }
}

int dq_num_threads(void) {
    int n = 1;
#ifdef _OPENMP
#pragma omp parallel
    {
#pragma omp master
        n = omp_get_num_threads();
    }
#endif
    return n;
}

/* =====================================================================================
 * NVFP4 variant (paper Sec. 5.1: the 4-bit float setting is NVFP4, blocks of 16 with an FP8 scale each;
 * Sec. 3: a 4-bit float with 1 mantissa and 2 exponent bits has q_max = 6).
 *
 *   element format E2M1: sign, 2 exponent bits, 1 mantissa bit; magnitudes {0, .5, 1, 1.5, 2, 3, 4, 6}
 *   block of 16 consecutive low-precision coefficients shares one FP8 E4M3 scale (used unsigned)
 *   Q(X) = e2m1_rne(X / s) * s,   s = e4m3_rne(max|X| / 6 / 2^e) * 2^e          (Eq. 1 with z = 0)
 *
 * Reading where the paper is silent: NVFP4 is a two-level format; the second level here is one
 * power-of-two scale 2^e per tensor, fixed offline (activations: from the calibration batch;
 * weights: from the folded weight), chosen so that the largest block scale lands at <= 256 in
 * E4M3 (max finite 448).  Rounding is to nearest, ties to the even code; the scale saturates at
 * 448, the element at +-6.  "Parity unpinned" against the authors' implementation.
 * ===================================================================================== */

/* E4M3 (4 exponent bits, bias 7, 3 mantissa bits, no infinities, max finite 448), unsigned use. */
double dq_e4m3_to_double(uint8_t b) {
    int e = (b >> 3) & 0xF, m = b & 7;
    double v = (e == 0) ? ldexp((double)m, -9) : ldexp(1.0 + m / 8.0, e - 7);
    return (b & 0x80) ? -v : v;
}

/* Round a non-negative fp64 value to E4M3, nearest, ties to even, saturating at 448. */
uint8_t dq_e4m3_round(double v) {
    if (!(v > 0.0)) return 0;
    if (v >= 448.0) return 0x7E;                       /* 1111 110 = 448 */
    int e = ilogb(v);
    if (e < -6) e = -6;                                /* subnormals: fixed quantum 2^-9 */
    double quantum = ldexp(1.0, e - 3);
    double m = rint(v / quantum);                      /* ties to even */
    double r = m * quantum;
    if (r >= 448.0) return 0x7E;
    if (r == 0.0) return 0;
    int er = ilogb(r);
    if (er < -6) return (uint8_t)(int)(r / ldexp(1.0, -9));            /* subnormal: mantissa only */
    int mant = (int)((r / ldexp(1.0, er) - 1.0) * 8.0);
    return (uint8_t)(((er + 7) << 3) | mant);
}

static const double kE2M1[8] = {0.0, 0.5, 1.0, 1.5, 2.0, 3.0, 4.0, 6.0};

double dq_e2m1_to_double(uint8_t code) {
    double v = kE2M1[code & 7];
    return (code & 8) ? -v : v;
}

/* Nearest E2M1 value, ties to the even code (mantissa bit 0), saturating at 6. */
uint8_t dq_e2m1_round(double t) {
    uint8_t sign = (t < 0.0 || (t == 0.0 && signbit(t))) ? 8 : 0;
    double a = fabs(t);
    int best = 0;
    double bd = fabs(a - kE2M1[0]);
    for (int c = 1; c < 8; ++c) {
        double d = fabs(a - kE2M1[c]);
        if (d < bd || (d == bd && (c & 1) == 0)) { bd = d; best = c; }
    }
    return (uint8_t)(sign | best);
}

/* Exponent of the per-tensor power-of-two scale for a tensor whose absolute maximum is amax. */
int dq_nvfp4_global_exponent(double amax) {
    if (!(amax > 0.0)) return 0;
    return (int)ceil(log2(amax / (6.0 * 256.0)));
}

/* One block (n <= 16 real elements).  Writes the E4M3 scale byte, the E2M1 codes and, if t != NULL,
 * the pre-rounding quotients. */
void dq_nvfp4_quantize_block(const double* v, int n, int64_t stride, int e_global, uint8_t* sf, uint8_t* codes,
                             int64_t code_stride, double* t, int64_t t_stride) {
    double a = 0.0;
    for (int i = 0; i < n; ++i) {
        double x = fabs(v[i * stride]);
        if (x > a) a = x;
    }
    uint8_t sb = dq_e4m3_round(ldexp(a / 6.0, -e_global));
    double s = ldexp(dq_e4m3_to_double(sb), e_global);
    *sf = sb;
    for (int i = 0; i < n; ++i) {
        double ti = (s != 0.0) ? v[i * stride] / s : 0.0;
        codes[i * code_stride] = (s != 0.0) ? dq_e2m1_round(ti) : 0;
        if (t) t[i * t_stride] = ti;
    }
}

/* Weights: rows < r -> bf16 Wh; rows >= r -> blocks of 16 along K per output column.
 * wcodes[K_l,N] (E2M1 codes 0..15), wsf[ceil(K_l/16),N] (E4M3 bytes); returns the global exponent. */
int dq_nvfp4_prepare_weights(const double* Wt, int K, int N, int r, uint16_t* Wh, uint8_t* wcodes, uint8_t* wsf,
                             double* wt) {
    int K_l = K - r;
    int nb = (K_l + 15) / 16;
    dq_round_bf16(Wt, Wh, (int64_t)r * N);
    double amax = 0.0;
    for (int64_t i = (int64_t)r * N; i < (int64_t)K * N; ++i) {
        double x = fabs(Wt[i]);
        if (x > amax) amax = x;
    }
    int e = dq_nvfp4_global_exponent(amax);
#pragma omp parallel for schedule(static)
    for (int n = 0; n < N; ++n) {
        for (int b = 0; b < nb; ++b) {
            int j0 = b * 16;
            int len = (j0 + 16 <= K_l) ? 16 : (K_l - j0);
            dq_nvfp4_quantize_block(Wt + (int64_t)(r + j0) * N + n, len, N, e, wsf + (int64_t)b * N + n,
                                    wcodes + (int64_t)j0 * N + n, N, wt ? wt + (int64_t)j0 * N + n : NULL, N);
        }
    }
    return e;
}

/* Activations: xt[M,K] -> xh bf16 [M,r]; codes [M,K_l]; sf [M,ceil(K_l/16)]; t (optional) [M,K_l]. */
void dq_nvfp4_split_quantize(const double* xt, int M, int K, int r, int e_global, uint16_t* xh, uint8_t* codes,
                             uint8_t* sf, double* t) {
    int K_l = K - r;
    int nb = (K_l + 15) / 16;
#pragma omp parallel for schedule(static)
    for (int m = 0; m < M; ++m) {
        const double* row = xt + (int64_t)m * K;
        for (int i = 0; i < r; ++i) xh[(int64_t)m * r + i] = dq_double_to_bf16(row[i]);
        for (int b = 0; b < nb; ++b) {
            int j0 = b * 16;
            int len = (j0 + 16 <= K_l) ? 16 : (K_l - j0);
            dq_nvfp4_quantize_block(row + r + j0, len, 1, e_global, sf + (int64_t)m * nb + b,
                                    codes + (int64_t)m * K_l + j0, 1, t ? t + (int64_t)m * K_l + j0 : NULL, 1);
        }
    }
}

/* y = sum_k (sfx 2^ex vx)(sfw 2^ew vw) + sum_{i<r} xh Wh + bias, fp64, then bf16. */
void dq_nvfp4_combine(const uint8_t* xcodes, const uint8_t* xsf, int ex, const uint8_t* wcodes, const uint8_t* wsf,
                      int ew, const uint16_t* xh, const uint16_t* Wh, const uint16_t* bias, int M, int N, int K_l,
                      int r, double* y64, uint16_t* ybits) {
    int nb = (K_l + 15) / 16;
#pragma omp parallel for schedule(static)
    for (int m = 0; m < M; ++m) {
        for (int n = 0; n < N; ++n) {
            double acc = 0.0;
            for (int b = 0; b < nb; ++b) {
                int j1 = (b * 16 + 16 <= K_l) ? b * 16 + 16 : K_l;
                double part = 0.0;
                for (int j = b * 16; j < j1; ++j)
                    part += dq_e2m1_to_double(xcodes[(int64_t)m * K_l + j]) * dq_e2m1_to_double(wcodes[(int64_t)j * N + n]);
                acc += part * dq_e4m3_to_double(xsf[(int64_t)m * nb + b]) * dq_e4m3_to_double(wsf[(int64_t)b * N + n]);
            }
            acc = ldexp(acc, ex + ew);
            double lr = 0.0;
            for (int i = 0; i < r; ++i)
                lr += dq_bf16_to_double(xh[(int64_t)m * r + i]) * dq_bf16_to_double(Wh[(int64_t)i * N + n]);
            double v = acc + lr + (bias ? dq_bf16_to_double(bias[n]) : 0.0);
            if (y64) y64[(int64_t)m * N + n] = v;
            ybits[(int64_t)m * N + n] = dq_double_to_bf16(v);
        }
    }
}
