/*
 * CPU ORACLE — TEST INFRASTRUCTURE, NOT PART OF THE PRODUCT.
 *
 * A plain, slow, obviously-correct definition of the BF16 attention output
 * projection with residual addition,
 *
 *     ref[m,n] = sum_{k=0..K-1} X[m,k] * W[n,k]  (+ bias[n])  (+ R[m,n]),
 *
 * which is the row-major form of the paper's residual GEMM epilogue
 * D = alpha * W^T A + beta * C with C = D, alpha = beta = 1 (Appendix A,
 * "L1-030: attention output projection with residual", Algorithm 3, last two
 * steps: the output is aliased onto the residual and O <- W^T A + O), and,
 * with bias = R = NULL, the plain BF16 matrix product of the paper's
 * fixed-shape GEMM study (Section 4.1).
 *
 * Arithmetic: every BF16 input is widened exactly to double; each product of
 * two BF16 values is exact in double (8 x 8 significant bits); the sum runs
 * over k in increasing order, one output element at a time; bias and residual
 * are added last, in that order; the result is kept as an unrounded double.
 * The four outputs handled per inner loop are independent elements: nothing
 * is blocked, fused or reordered inside one element's sum.
 *
 * Only tests, the smoke check and the benchmark's CPU-baseline leg may call
 * this.  It shares no code, header, table or helper with the CUDA path.
 *
 * Pins (tests that run without a GPU): exact rational brute force on tiny
 * shapes, agreement with a float64 library matmul, closed forms (constant
 * operands, one-hot selectors), the invariants W=0, W=I and linearity in X,
 * and a hand-computed fixture.  The paper prints no worked numerical example
 * for this operation, so no fixture carries paper-printed values.
 */
#include <fenv.h>
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

/* BF16 bit pattern -> double (exact): BF16 is the upper half of an FP32. */
static inline double bf16_widen(uint16_t b) {
    uint32_t u = (uint32_t)b << 16;
    float f;
    memcpy(&f, &u, sizeof f);
    return (double)f;
}

int kx_oracle_max_threads(void) {
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}

void kx_oracle_widen_bf16(const uint16_t* in, double* out, int64_t n) {
    for (int64_t i = 0; i < n; ++i) out[i] = bf16_widen(in[i]);
}

/*
 * double -> BF16 bits, ONE round-to-nearest-even from the exact value.
 * BF16 has 8 significant bits (1 implicit + 7 stored) and FP32's exponent
 * range: normal binades 2^-126 .. 2^127, subnormal quantum 2^-133.
 * For |x| in [2^e, 2^(e+1)) the representable grid has spacing q = 2^(e-7);
 * x/q is exact (q is a power of two) and nearbyint() under the default
 * rounding mode rounds half-way cases to the even integer, i.e. to the BF16
 * value whose last stored bit is zero.
 */
static uint16_t bf16_round_one(double x) {
    if (isnan(x)) return 0x7FC0;
    uint16_t sign = signbit(x) ? 0x8000 : 0;
    double a = fabs(x);
    if (isinf(a)) return (uint16_t)(sign | 0x7F80);
    if (a == 0.0) return sign;
    int ex;
    (void)frexp(a, &ex);           /* a = f * 2^ex, f in [0.5,1)  => 2^(ex-1) <= a */
    int e = ex - 1;
    if (e < -126) e = -126;        /* subnormal range shares the 2^-126 binade's grid */
    double q = ldexp(1.0, e - 7);
    double r = nearbyint(a / q) * q;   /* exact: integer < 2^9 times a power of two */
    if (r >= ldexp(1.0, 128)) return (uint16_t)(sign | 0x7F80);
    float f = (float)r;            /* exact: r has <= 8 significant bits */
    uint32_t u;
    memcpy(&u, &f, sizeof u);
    return (uint16_t)(sign | (uint16_t)(u >> 16));
}

void kx_oracle_round_bf16(const double* in, uint16_t* out, int64_t n) {
    fesetround(FE_TONEAREST);
    for (int64_t i = 0; i < n; ++i) out[i] = bf16_round_one(in[i]);
}

/*
 * Reference for a set of rows.
 *   X    [M,K]  BF16 bits, row-major (host)
 *   W    [N,K]  BF16 bits, row-major (host)
 *   bias [N]    BF16 bits or NULL
 *   R    [M,N]  BF16 bits or NULL
 *   rows [nrows] row indices into X / R, or NULL meaning rows 0..nrows-1
 *   ref    [nrows,N] out: unrounded double
 *   absref [nrows,N] out or NULL: sum_k |X||W| + |bias| + |R|
 * Returns 0, or -1 on a bad argument / failed allocation.
 */
int kx_oracle_outproj_rows(const uint16_t* X, const uint16_t* W, const uint16_t* bias,
                           const uint16_t* R, const int64_t* rows, int64_t nrows,
                           double* ref, double* absref,
                           int64_t M, int64_t N, int64_t K, int threads) {
    if (M < 0 || N < 0 || K < 0 || nrows < 0) return -1;
    if (nrows == 0 || N == 0) return 0;
    if (!ref || (K > 0 && (!X || !W))) return -1;
    for (int64_t i = 0; rows && i < nrows; ++i)
        if (rows[i] < 0 || rows[i] >= M) return -1;
    if (!rows && nrows > M) return -1;

    double* Wd = (double*)malloc(sizeof(double) * (size_t)(N * K > 0 ? N * K : 1));
    double* Xd = (double*)malloc(sizeof(double) * (size_t)(nrows * K > 0 ? nrows * K : 1));
    if (!Wd || !Xd) { free(Wd); free(Xd); return -1; }
#ifdef _OPENMP
    if (threads <= 0) threads = omp_get_max_threads();
#else
    threads = 1;
#endif

#pragma omp parallel for schedule(static) num_threads(threads)
    for (int64_t n = 0; n < N; ++n)
        for (int64_t k = 0; k < K; ++k) Wd[n * K + k] = bf16_widen(W[n * K + k]);
#pragma omp parallel for schedule(static) num_threads(threads)
    for (int64_t i = 0; i < nrows; ++i) {
        int64_t m = rows ? rows[i] : i;
        for (int64_t k = 0; k < K; ++k) Xd[i * K + k] = bf16_widen(X[m * K + k]);
    }

    const int64_t nblk = (N + 3) / 4;
#pragma omp parallel for collapse(2) schedule(static) num_threads(threads)
    for (int64_t i = 0; i < nrows; ++i) {
        for (int64_t nb = 0; nb < nblk; ++nb) {
            const int64_t m = rows ? rows[i] : i;
            const int64_t n0 = nb * 4;
            const int cnt = (int)((N - n0) < 4 ? (N - n0) : 4);
            const double* x = Xd + i * K;
            const double* w[4];
            for (int j = 0; j < 4; ++j) w[j] = Wd + (n0 + (j < cnt ? j : 0)) * K;
            /* four independent output elements; each sums k = 0,1,2,... in order */
            double s0 = 0.0, s1 = 0.0, s2 = 0.0, s3 = 0.0;
            for (int64_t k = 0; k < K; ++k) {
                const double xv = x[k];
                s0 += xv * w[0][k];
                s1 += xv * w[1][k];
                s2 += xv * w[2][k];
                s3 += xv * w[3][k];
            }
            double s[4] = {s0, s1, s2, s3};
            for (int j = 0; j < cnt; ++j) {
                double v = s[j];
                if (bias) v += bf16_widen(bias[n0 + j]);
                if (R) v += bf16_widen(R[m * N + n0 + j]);
                ref[i * N + n0 + j] = v;
            }
            if (absref) {
                for (int j = 0; j < cnt; ++j) {
                    double a = 0.0;
                    for (int64_t k = 0; k < K; ++k) a += fabs(x[k]) * fabs(w[j][k]);
                    if (bias) a += fabs(bf16_widen(bias[n0 + j]));
                    if (R) a += fabs(bf16_widen(R[m * N + n0 + j]));
                    absref[i * N + n0 + j] = a;
                }
            }
        }
    }
    free(Wd);
    free(Xd);
    return 0;
}

/* Reference for the whole [M,N] output. */
int kx_oracle_outproj(const uint16_t* X, const uint16_t* W, const uint16_t* bias,
                      const uint16_t* R, double* ref, double* absref,
                      int64_t M, int64_t N, int64_t K, int threads) {
    return kx_oracle_outproj_rows(X, W, bias, R, NULL, M, ref, absref, M, N, K, threads);
}

/* Reference for one output element (used for spot checks at full sizes). */
double kx_oracle_element(const uint16_t* X, const uint16_t* W, const uint16_t* bias,
                         const uint16_t* R, int64_t m, int64_t n, int64_t N, int64_t K) {
    double s = 0.0;
    for (int64_t k = 0; k < K; ++k) s += bf16_widen(X[m * K + k]) * bf16_widen(W[n * K + k]);
    if (bias) s += bf16_widen(bias[n]);
    if (R) s += bf16_widen(R[m * N + n]);
    return s;
}

/*
 * RMSNorm of rows of a BF16 matrix (the step that follows the output projection and
 * first residual in the paper's decoder-layer case study, Appendix A, Algorithm 7: "run
 * fused add+RMSNorm ..."; the paper prints no formula, so this is the textbook
 * definition):
 *
 *     z[m,n] = h[m,n] / sqrt( (1/N) * sum_j h[m,j]^2 + eps ) * gamma[n]
 *
 * h and gamma are BF16 bit patterns widened exactly to double; the sum of squares runs
 * over j in increasing order in double; the result is kept unrounded.
 *   H [M,N], gamma [N], rows [nrows] (NULL = rows 0..nrows-1), out [nrows,N].
 */
int kx_oracle_rmsnorm_rows(const uint16_t* H, const uint16_t* gamma, double eps, const int64_t* rows,
                           int64_t nrows, double* out, int64_t M, int64_t N) {
    if (M < 0 || N <= 0 || nrows < 0 || !H || !gamma || !out) return -1;
    for (int64_t i = 0; rows && i < nrows; ++i)
        if (rows[i] < 0 || rows[i] >= M) return -1;
    if (!rows && nrows > M) return -1;
#pragma omp parallel for schedule(static)
    for (int64_t i = 0; i < nrows; ++i) {
        const int64_t m = rows ? rows[i] : i;
        double ss = 0.0;
        for (int64_t j = 0; j < N; ++j) {
            const double h = bf16_widen(H[m * N + j]);
            ss += h * h;
        }
        const double inv = 1.0 / sqrt(ss / (double)N + eps);
        for (int64_t j = 0; j < N; ++j)
            out[i * N + j] = bf16_widen(H[m * N + j]) * inv * bf16_widen(gamma[j]);
    }
    return 0;
}

/*
 * Gate/up projections with the SwiGLU product (the MLP's first half in the paper's
 * decoder-layer case study, Appendix A, Algorithm 7: "compute BF16 gate/up projections
 * and a ... SiLU-multiply", fused there as a "SwiGLU epilogue"):
 *
 *     g[m,i] = sum_k X[m,k] * Wg[i,k],   u[m,i] = sum_k X[m,k] * Wu[i,k]
 *     z[m,i] = silu(g[m,i]) * u[m,i],    silu(t) = t / (1 + exp(-t))
 *
 * Both sums run over k in increasing order in double (products of BF16 values are exact);
 * the result is kept unrounded.  X [M,K], Wg and Wu [I,K] BF16 bits; rows [nrows] or NULL;
 * out [nrows,I]; gate_out / up_out [nrows,I] optional (NULL to skip).
 */
int kx_oracle_swiglu_rows(const uint16_t* X, const uint16_t* Wg, const uint16_t* Wu, const int64_t* rows,
                          int64_t nrows, double* out, double* gate_out, double* up_out,
                          int64_t M, int64_t I, int64_t K) {
    if (M < 0 || I < 0 || K < 0 || nrows < 0 || !out) return -1;
    if (K > 0 && (!X || !Wg || !Wu)) return -1;
    for (int64_t r = 0; rows && r < nrows; ++r)
        if (rows[r] < 0 || rows[r] >= M) return -1;
    if (!rows && nrows > M) return -1;
#pragma omp parallel for collapse(2) schedule(static)
    for (int64_t r = 0; r < nrows; ++r) {
        for (int64_t i = 0; i < I; ++i) {
            const int64_t m = rows ? rows[r] : r;
            double g = 0.0, u = 0.0;
            for (int64_t k = 0; k < K; ++k) {
                const double x = bf16_widen(X[m * K + k]);
                g += x * bf16_widen(Wg[i * K + k]);
                u += x * bf16_widen(Wu[i * K + k]);
            }
            out[r * I + i] = g / (1.0 + exp(-g)) * u;
            if (gate_out) gate_out[r * I + i] = g;
            if (up_out) up_out[r * I + i] = u;
        }
    }
    return 0;
}


/*
 * INT8 branch of the decoder layer (Appendix A, Algorithm 7: "fused add+RMSNorm+activation
 * quantization", "quantize gate/up weights", "gate/up GEMM with fused dequantization and
 * SwiGLU epilogue").  The paper names the steps but not the code book; the reading taken here
 * is the common symmetric one, per row (per token for activations, per output channel for
 * weights):
 *
 *     a      = max_j |z[j]|                        (exact: the inputs are BF16)
 *     scale  = a / 127,   inv = 127 / a            (each ONE binary32 division; a == 0: 1, 0)
 *     q[j]   = clamp(rint(z[j] * inv), -127, 127)  (binary32 product, round half to even)
 *
 * The code is an integer decided by floating point, so the decision is taken in binary32,
 * the precision the CUDA path uses, with exactly these operations in this order; nothing
 * here runs in double.  Z [rows, cols] BF16 bits -> Q [rows, cols] int8, S [rows] float.
 */
int kx_oracle_quantize_rows(const uint16_t* Z, int64_t rows, int64_t cols, int8_t* Q, float* S) {
    if (rows < 0 || cols < 0 || (rows > 0 && (!S || (cols > 0 && (!Z || !Q))))) return -1;
#pragma omp parallel for schedule(static)
    for (int64_t r = 0; r < rows; ++r) {
        float a = 0.0f;
        for (int64_t j = 0; j < cols; ++j) {
            const float v = fabsf((float)bf16_widen(Z[r * cols + j]));
            if (v > a) a = v;
        }
        const float scale = (a > 0.0f) ? a / 127.0f : 1.0f;
        const float inv = (a > 0.0f) ? 127.0f / a : 0.0f;
        S[r] = scale;
        for (int64_t j = 0; j < cols; ++j) {
            const float z = (float)bf16_widen(Z[r * cols + j]);
            float t = rintf(z * inv);
            if (t > 127.0f) t = 127.0f;
            if (t < -127.0f) t = -127.0f;
            Q[r * cols + j] = (int8_t)t;
        }
    }
    return 0;
}

/*
 * Integer contraction with dequantisation: acc[m,n] = sum_k Xq[m,k] * Wq[n,k] (exact, int64),
 * value = acc * sx[m] * sw[n] in double.  Used by the two functions below.
 */
static double dq_dot(const int8_t* x, const int8_t* w, int64_t K, float sx, float sw, int64_t* acc_out) {
    int64_t acc = 0;
    for (int64_t k = 0; k < K; ++k) acc += (int64_t)x[k] * (int64_t)w[k];
    if (acc_out) *acc_out = acc;
    return (double)acc * (double)sx * (double)sw;
}

/*
 * Gate/up GEMM on INT8 codes with fused dequantisation and SwiGLU (Appendix A, Algorithm 7):
 *     g = (Xq Wgq^T)[m,i] * sx[m] * sg[i],  u = (Xq Wuq^T)[m,i] * sx[m] * su[i],
 *     z = g / (1 + exp(-g)) * u              (double, unrounded)
 * Xq [M,K], Wgq / Wuq [I,K] int8; sx [M], sg / su [I] float; rows [nrows] or NULL;
 * out [nrows, I]; gate_acc / up_acc [nrows, I] optional exact integer sums.
 */
int kx_oracle_swiglu_int8_rows(const int8_t* Xq, const float* sx, const int8_t* Wgq, const float* sg,
                               const int8_t* Wuq, const float* su, const int64_t* rows, int64_t nrows,
                               double* out, int64_t* gate_acc, int64_t* up_acc, int64_t M, int64_t I, int64_t K) {
    if (M < 0 || I < 0 || K < 0 || nrows < 0 || !out || !sx || !sg || !su) return -1;
    if (K > 0 && (!Xq || !Wgq || !Wuq)) return -1;
    for (int64_t r = 0; rows && r < nrows; ++r)
        if (rows[r] < 0 || rows[r] >= M) return -1;
    if (!rows && nrows > M) return -1;
#pragma omp parallel for collapse(2) schedule(static)
    for (int64_t r = 0; r < nrows; ++r) {
        for (int64_t i = 0; i < I; ++i) {
            const int64_t m = rows ? rows[r] : r;
            int64_t ga = 0, ua = 0;
            const double g = dq_dot(Xq + m * K, Wgq + i * K, K, sx[m], sg[i], &ga);
            const double u = dq_dot(Xq + m * K, Wuq + i * K, K, sx[m], su[i], &ua);
            out[r * I + i] = g / (1.0 + exp(-g)) * u;
            if (gate_acc) gate_acc[r * I + i] = ga;
            if (up_acc) up_acc[r * I + i] = ua;
        }
    }
    return 0;
}

/*
 * The output projection with residual on INT8 codes (the precision axis of the paper's strategy
 * space, Section 3.2, applied to the operator of Appendix A, Algorithm 3):
 *     y[m,n] = (Xq Wq^T)[m,n] * sx[m] * sw[n] + bias[n] + R[m,n]     (double, unrounded)
 * bias [N] / R [M,N] BF16 bits or NULL.
 */
int kx_oracle_outproj_int8_rows(const int8_t* Xq, const float* sx, const int8_t* Wq, const float* sw,
                                const uint16_t* bias, const uint16_t* R, const int64_t* rows, int64_t nrows,
                                double* out, int64_t M, int64_t N, int64_t K) {
    if (M < 0 || N < 0 || K < 0 || nrows < 0 || !out || !sx || !sw) return -1;
    if (K > 0 && (!Xq || !Wq)) return -1;
    for (int64_t r = 0; rows && r < nrows; ++r)
        if (rows[r] < 0 || rows[r] >= M) return -1;
    if (!rows && nrows > M) return -1;
#pragma omp parallel for collapse(2) schedule(static)
    for (int64_t r = 0; r < nrows; ++r) {
        for (int64_t n = 0; n < N; ++n) {
            const int64_t m = rows ? rows[r] : r;
            double y = dq_dot(Xq + m * K, Wq + n * K, K, sx[m], sw[n], 0);
            if (bias) y += bf16_widen(bias[n]);
            if (R) y += bf16_widen(R[m * N + n]);
            out[r * N + n] = y;
        }
    }
    return 0;
}

/*
 * FP8 (E4M3, the "FN" flavour: bias 7, no infinities, 0x7F / 0xFF = NaN, largest finite 448)
 * variants of the same three steps, the other low-precision operand type of the paper's
 * precision axis (Section 3.2).  Decoding is exact; encoding rounds a binary32 value to the
 * nearest code, ties to the even mantissa, and saturates to +-448 ("satfinite"); NaN -> 0x7F.
 */
static double e4m3_decode(uint8_t c) {
    const int s = c >> 7, e = (c >> 3) & 15, m = c & 7;
    double v;
    if (e == 15 && m == 7) return NAN;
    if (e == 0) v = ldexp((double)m, -9);              /* subnormal: m/8 * 2^-6 */
    else v = ldexp(1.0 + m / 8.0, e - 7);
    return s ? -v : v;
}

static uint8_t e4m3_encode(float x) {
    const uint8_t s = signbit(x) ? 0x80 : 0;
    if (isnan(x)) return 0x7F;
    const float ax = fabsf(x);
    if (ax > 448.0f) {
        /* above the largest finite code: everything that would round past 448 saturates */
        return s | 0x7E;
    }
    if (ax < 0.015625f) {                               /* below 2^-6: fixed step 2^-9 */
        const int q = (int)rintf(ax * 512.0f);          /* exact product; 8 means 2^-6 = code 0x08 */
        return s | (uint8_t)q;
    }
    int e;
    const float mant = frexpf(ax, &e) * 2.0f;           /* ax = mant * 2^(e-1), mant in [1, 2) */
    e -= 1;
    int q = (int)rintf((mant - 1.0f) * 8.0f);           /* exact; ties to even */
    if (q == 8) { q = 0; e += 1; }
    int code = ((e + 7) << 3) | q;
    if (code > 0x7E) code = 0x7E;
    return s | (uint8_t)code;
}

int kx_oracle_e4m3_decode(const uint8_t* in, double* out, int64_t n) {
    if (n < 0 || (n > 0 && (!in || !out))) return -1;
    for (int64_t i = 0; i < n; ++i) out[i] = e4m3_decode(in[i]);
    return 0;
}

int kx_oracle_e4m3_encode(const float* in, uint8_t* out, int64_t n) {
    if (n < 0 || (n > 0 && (!in || !out))) return -1;
    for (int64_t i = 0; i < n; ++i) out[i] = e4m3_encode(in[i]);
    return 0;
}

/*
 * Per-row FP8 code book: a = max|z|, scale = a / 448, q = e4m3(z * (448 / a)), every operation
 * in binary32 as for the INT8 code book above (zero row: scale 1, codes 0).
 */
int kx_oracle_quantize_rows_fp8(const uint16_t* Z, int64_t rows, int64_t cols, uint8_t* Q, float* S) {
    if (rows < 0 || cols < 0 || (rows > 0 && (!S || (cols > 0 && (!Z || !Q))))) return -1;
#pragma omp parallel for schedule(static)
    for (int64_t r = 0; r < rows; ++r) {
        float a = 0.0f;
        for (int64_t j = 0; j < cols; ++j) {
            const float v = fabsf((float)bf16_widen(Z[r * cols + j]));
            if (v > a) a = v;
        }
        const float inv = (a > 0.0f) ? 448.0f / a : 0.0f;
        S[r] = (a > 0.0f) ? a / 448.0f : 1.0f;
        for (int64_t j = 0; j < cols; ++j) {
            const float z = (float)bf16_widen(Z[r * cols + j]);
            Q[r * cols + j] = e4m3_encode(z * inv);
        }
    }
    return 0;
}

static double dq_dot_fp8(const uint8_t* x, const uint8_t* w, int64_t K, float sx, float sw) {
    double acc = 0.0;                                   /* products of two E4M3 values are exact in double */
    for (int64_t k = 0; k < K; ++k) acc += e4m3_decode(x[k]) * e4m3_decode(w[k]);
    return acc * (double)sx * (double)sw;
}

/* z = silu(g) * u, g = (Xq Wgq^T) sx sg, u = (Xq Wuq^T) sx su on E4M3 codes; double, unrounded. */
int kx_oracle_swiglu_fp8_rows(const uint8_t* Xq, const float* sx, const uint8_t* Wgq, const float* sg,
                              const uint8_t* Wuq, const float* su, const int64_t* rows, int64_t nrows,
                              double* out, int64_t M, int64_t I, int64_t K) {
    if (M < 0 || I < 0 || K < 0 || nrows < 0 || !out || !sx || !sg || !su) return -1;
    if (K > 0 && (!Xq || !Wgq || !Wuq)) return -1;
    for (int64_t r = 0; rows && r < nrows; ++r)
        if (rows[r] < 0 || rows[r] >= M) return -1;
    if (!rows && nrows > M) return -1;
#pragma omp parallel for collapse(2) schedule(static)
    for (int64_t r = 0; r < nrows; ++r) {
        for (int64_t i = 0; i < I; ++i) {
            const int64_t m = rows ? rows[r] : r;
            const double g = dq_dot_fp8(Xq + m * K, Wgq + i * K, K, sx[m], sg[i]);
            const double u = dq_dot_fp8(Xq + m * K, Wuq + i * K, K, sx[m], su[i]);
            out[r * I + i] = g / (1.0 + exp(-g)) * u;
        }
    }
    return 0;
}

/* y = (Xq Wq^T) sx sw + bias + R on E4M3 codes; double, unrounded. */
int kx_oracle_outproj_fp8_rows(const uint8_t* Xq, const float* sx, const uint8_t* Wq, const float* sw,
                               const uint16_t* bias, const uint16_t* R, const int64_t* rows, int64_t nrows,
                               double* out, int64_t M, int64_t N, int64_t K) {
    if (M < 0 || N < 0 || K < 0 || nrows < 0 || !out || !sx || !sw) return -1;
    if (K > 0 && (!Xq || !Wq)) return -1;
    for (int64_t r = 0; rows && r < nrows; ++r)
        if (rows[r] < 0 || rows[r] >= M) return -1;
    if (!rows && nrows > M) return -1;
#pragma omp parallel for collapse(2) schedule(static)
    for (int64_t r = 0; r < nrows; ++r) {
        for (int64_t n = 0; n < N; ++n) {
            const int64_t m = rows ? rows[r] : r;
            double y = dq_dot_fp8(Xq + m * K, Wq + n * K, K, sx[m], sw[n]);
            if (bias) y += bf16_widen(bias[n]);
            if (R) y += bf16_widen(R[m * N + n]);
            out[r * N + n] = y;
        }
    }
    return 0;
}

/*
 * Block-scaled FP8 ("MXFP8": E4M3 elements, one power-of-two scale per 32 consecutive elements
 * of a row, stored as an E8M0 byte e meaning 2^(e-127); 0xFF is NaN), the block-scaled member of
 * the paper's precision axis (Section 3.2; Section 4.3 names the block-scaled tensor-core kinds).
 * The paper prints no conversion, so this follows the open Microscaling-formats definition:
 *   shared exponent  se = floor(log2(max|v|)) - 8        (8 = exponent of E4M3's largest binade)
 *   scale byte       e  = clamp(se + 127, 0, 254)        (an all-zero block takes e = 127)
 *   element          q  = e4m3(v / 2^(e-127))            (nearest, ties to even, saturating)
 * The quotient is exact (a power-of-two scaling), so the only rounding is E4M3's.
 */
static double e8m0_decode(uint8_t e) {
    return e == 0xFF ? NAN : ldexp(1.0, (int)e - 127);
}

int kx_oracle_e8m0_decode(const uint8_t* in, double* out, int64_t n) {
    if (n < 0 || (n > 0 && (!in || !out))) return -1;
    for (int64_t i = 0; i < n; ++i) out[i] = e8m0_decode(in[i]);
    return 0;
}

/* Z [rows, cols] BF16 -> Q [rows, cols] E4M3 codes, E [rows, ceil(cols/32)] E8M0 bytes (row-major). */
int kx_oracle_quantize_rows_mx(const uint16_t* Z, int64_t rows, int64_t cols, uint8_t* Q, uint8_t* E) {
    if (rows < 0 || cols < 0 || (rows > 0 && cols > 0 && (!Z || !Q || !E))) return -1;
    const int64_t nb = (cols + 31) / 32;
#pragma omp parallel for schedule(static)
    for (int64_t r = 0; r < rows; ++r) {
        for (int64_t j = 0; j < nb; ++j) {
            const int64_t k0 = j * 32, k1 = (k0 + 32 < cols) ? k0 + 32 : cols;
            double a = 0.0;
            for (int64_t k = k0; k < k1; ++k) {
                const double v = fabs(bf16_widen(Z[r * cols + k]));
                if (v > a) a = v;                       /* NaN never wins the comparison */
            }
            int e = 127;
            if (a > 0.0) {
                int ex;
                if (isinf(a)) ex = 129;                 /* treated as the binade above the largest finite one */
                else (void)frexp(a, &ex);               /* a = f * 2^ex, f in [0.5, 1): floor(log2 a) = ex - 1 */
                e = (ex - 1) - 8 + 127;
                if (e < 0) e = 0;
                if (e > 254) e = 254;
            }
            E[r * nb + j] = (uint8_t)e;
            for (int64_t k = k0; k < k1; ++k) {
                const double t = ldexp(bf16_widen(Z[r * cols + k]), 127 - e);   /* exact */
                Q[r * cols + k] = e4m3_encode((float)t);
            }
        }
    }
    return 0;
}

/* y = sum over 32-element blocks j of 2^(ex[m,j]-127) 2^(ew[n,j]-127) (xq . wq over the block)
 *     + bias + R; double, unrounded. */
int kx_oracle_outproj_mx_rows(const uint8_t* Xq, const uint8_t* ex, const uint8_t* Wq, const uint8_t* ew,
                              const uint16_t* bias, const uint16_t* R, const int64_t* rows, int64_t nrows,
                              double* out, int64_t M, int64_t N, int64_t K) {
    if (M < 0 || N < 0 || K < 0 || nrows < 0 || !out) return -1;
    if (K > 0 && (!Xq || !Wq || !ex || !ew)) return -1;
    for (int64_t r = 0; rows && r < nrows; ++r)
        if (rows[r] < 0 || rows[r] >= M) return -1;
    if (!rows && nrows > M) return -1;
    const int64_t nb = (K + 31) / 32;
#pragma omp parallel for collapse(2) schedule(static)
    for (int64_t r = 0; r < nrows; ++r) {
        for (int64_t n = 0; n < N; ++n) {
            const int64_t m = rows ? rows[r] : r;
            double y = 0.0;
            for (int64_t j = 0; j < nb; ++j) {
                const int64_t k1 = (j * 32 + 32 < K) ? j * 32 + 32 : K;
                double acc = 0.0;
                for (int64_t k = j * 32; k < k1; ++k) acc += e4m3_decode(Xq[m * K + k]) * e4m3_decode(Wq[n * K + k]);
                y += acc * e8m0_decode(ex[m * nb + j]) * e8m0_decode(ew[n * nb + j]);
            }
            if (bias) y += bf16_widen(bias[n]);
            if (R) y += bf16_widen(R[m * N + n]);
            out[r * N + n] = y;
        }
    }
    return 0;
}

/*
 * 4-bit block-scaled format ("NVFP4", the format of the paper's Section 4.3 task): E2M1 elements
 * (sign, 2 exponent bits with bias 1, 1 mantissa bit: magnitudes 0, 0.5, 1, 1.5, 2, 3, 4, 6), two per
 * byte (the element with the even k index in the low nibble), one E4M3 scale byte per 16 consecutive
 * elements of a row, and one binary32 scale gs for the whole tensor:
 *     value = e2m1(q) * e4m3(s) * gs.
 * The paper prints no conversion; the code book below is this build's reading, every step in binary32:
 *     a  = max |z| over the block
 *     s  = e4m3( a / (6 gs) )                  (nearest, ties to even, saturating at 448)
 *     r  = 1 / (e4m3_value(s) * gs)            (codes are all zero when s decodes to zero)
 *     q  = e2m1( z * r )                       (nearest, ties to the even code, saturating at 6)
 */
static double e2m1_decode(uint8_t nib) {
    const int s = (nib >> 3) & 1, e = (nib >> 1) & 3, m = nib & 1;
    const double v = (e == 0) ? 0.5 * m : ldexp(1.0 + 0.5 * m, e - 1);
    return s ? -v : v;
}

static uint8_t e2m1_encode(float x) {
    static const float grid[8] = {0.0f, 0.5f, 1.0f, 1.5f, 2.0f, 3.0f, 4.0f, 6.0f};
    const uint8_t s = signbit(x) ? 8 : 0;
    if (isnan(x)) return 7;                               /* no NaN code: the largest magnitude */
    const float ax = fabsf(x);
    if (ax >= 6.0f) return s | 7;
    int best = 0;
    for (int c = 1; c < 8; ++c) {
        const float dc = fabsf(grid[c] - ax), db = fabsf(grid[best] - ax);      /* exact differences */
        if (dc < db || (dc == db && (c & 1) == 0)) best = c;
    }
    return s | (uint8_t)best;
}

int kx_oracle_e2m1_decode(const uint8_t* in, double* out, int64_t n) {
    if (n < 0 || (n > 0 && (!in || !out))) return -1;
    for (int64_t i = 0; i < n; ++i) out[i] = e2m1_decode(in[i] & 15);
    return 0;
}

int kx_oracle_e2m1_encode(const float* in, uint8_t* out, int64_t n) {
    if (n < 0 || (n > 0 && (!in || !out))) return -1;
    for (int64_t i = 0; i < n; ++i) out[i] = e2m1_encode(in[i]);
    return 0;
}

/* Z [rows, cols] BF16 (cols even) -> Q [rows, cols / 2] packed nibbles, S [rows, ceil(cols / 16)] E4M3 bytes. */
int kx_oracle_quantize_rows_nvfp4(const uint16_t* Z, int64_t rows, int64_t cols, float gs, uint8_t* Q, uint8_t* S) {
    if (rows < 0 || cols < 0 || (cols & 1) || !(gs > 0.0f) || (rows > 0 && cols > 0 && (!Z || !Q || !S))) return -1;
    const int64_t nb = (cols + 15) / 16;
#pragma omp parallel for schedule(static)
    for (int64_t r = 0; r < rows; ++r) {
        for (int64_t j = 0; j < nb; ++j) {
            const int64_t k0 = j * 16, k1 = (k0 + 16 < cols) ? k0 + 16 : cols;
            float a = 0.0f;
            for (int64_t k = k0; k < k1; ++k) {
                const float v = fabsf((float)bf16_widen(Z[r * cols + k]));
                if (v > a) a = v;
            }
            const float d6 = 6.0f * gs;                    /* one binary32 product */
            const uint8_t sb = e4m3_encode(a / d6);        /* one binary32 division, then the E4M3 rounding */
            S[r * nb + j] = sb;
            const float sd = (float)e4m3_decode(sb);
            const float dq = sd * gs;                      /* binary32 product */
            const float rcp = (dq > 0.0f) ? 1.0f / dq : 0.0f;
            for (int64_t k = k0; k < k1; k += 2) {
                const float z0 = (float)bf16_widen(Z[r * cols + k]), z1 = (float)bf16_widen(Z[r * cols + k + 1]);
                const uint8_t q0 = (dq > 0.0f) ? e2m1_encode(z0 * rcp) : 0;
                const uint8_t q1 = (dq > 0.0f) ? e2m1_encode(z1 * rcp) : 0;
                Q[(r * cols + k) / 2] = (uint8_t)(q0 | (q1 << 4));
            }
        }
    }
    return 0;
}

/* y = alpha * sum over 16-element blocks j of e4m3(sx[m,j]) e4m3(sw[n,j]) (xq . wq over the block)
 *     + bias + R; double, unrounded.  Xq [M, K/2], Wq [N, K/2] packed nibbles. */
int kx_oracle_outproj_nvfp4_rows(const uint8_t* Xq, const uint8_t* sx, const uint8_t* Wq, const uint8_t* sw,
                                 double alpha, const uint16_t* bias, const uint16_t* R, const int64_t* rows,
                                 int64_t nrows, double* out, int64_t M, int64_t N, int64_t K) {
    if (M < 0 || N < 0 || K < 0 || (K & 1) || nrows < 0 || !out) return -1;
    if (K > 0 && (!Xq || !Wq || !sx || !sw)) return -1;
    for (int64_t r = 0; rows && r < nrows; ++r)
        if (rows[r] < 0 || rows[r] >= M) return -1;
    if (!rows && nrows > M) return -1;
    const int64_t nb = (K + 15) / 16, kb = K / 2;
#pragma omp parallel for collapse(2) schedule(static)
    for (int64_t r = 0; r < nrows; ++r) {
        for (int64_t n = 0; n < N; ++n) {
            const int64_t m = rows ? rows[r] : r;
            double y = 0.0;
            for (int64_t j = 0; j < nb; ++j) {
                const int64_t k1 = (j * 16 + 16 < K) ? j * 16 + 16 : K;
                double acc = 0.0;
                for (int64_t k = j * 16; k < k1; ++k) {
                    const uint8_t xb = Xq[m * kb + k / 2], wb = Wq[n * kb + k / 2];
                    acc += e2m1_decode((k & 1) ? xb >> 4 : xb & 15) * e2m1_decode((k & 1) ? wb >> 4 : wb & 15);
                }
                y += acc * e4m3_decode(sx[m * nb + j]) * e4m3_decode(sw[n * nb + j]);
            }
            y *= alpha;
            if (bias) y += bf16_widen(bias[n]);
            if (R) y += bf16_widen(R[m * N + n]);
            out[r * N + n] = y;
        }
    }
    return 0;
}
