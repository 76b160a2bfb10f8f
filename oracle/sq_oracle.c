/*
 * SmoothQuant W8A8 hot path -- CPU ORACLE (test infrastructure, not product code).
 *
 * A plain, slow, loop-by-loop restatement of what the paper's method computes,
 * used only to check the CUDA library and to be timed as a CPU baseline.  It
 * shares no code, header, table or helper with the CUDA path and must never be
 * called from it.  Build:  gcc -O2 -ffp-contract=off -fno-fast-math -fopenmp.
 * With contraction off, every fused multiply-add below is an explicit fmaf().
 *
 * Notation follows the paper: X in R^{T x C_i} (tokens x input channels),
 * stored W is [C_o, C_i] row-major (the transpose of the paper's W in
 * R^{C_i x C_o}), Delta is a quantisation step size, s in R^{C_i} is the
 * smoothing factor, alpha the migration strength.
 *
 * Two kinds of function live here:
 *   - the NORMATIVE fp32 path: the one rounding sequence that "bit-exact"
 *     refers to (Eq. 1 quantiser, Eq. 2 dequantisation, Eq. 3 folding);
 *   - fp64 TRUTH helpers (plain definitions) used to pin the normative path.
 *
 * Activation-typed (fp16 / bf16) tensors arrive as float arrays whose values
 * are exactly representable in that type; rounding a result back to fp16/bf16
 * is done by the Python wrapper with a library cast (round-to-nearest-even).
 *
 * Parity unpinned: nothing in this file.  (The paper's accuracy tables and the
 * alpha sweet spot need trained weights and datasets; they are out of scope.)
 */
#include <math.h>
#include <stddef.h>
#include <stdint.h>
#ifdef _OPENMP
#include <omp.h>
#endif

/* Smallest absolute maximum ever used as a divisor.  The paper is silent on an
 * all-zero row or channel (Delta = 0, s_j = 0 or infinity); this floor is the
 * reading taken. */
#define SQO_ABSMAX_FLOOR 1e-5f

int sqo_num_threads(void) {
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}

/* ------------------------------------------------------------------------- */
/* Section 4, "s_j = max(|X_j|)": per-input-channel absolute maximum, taken  */
/* over every token of every calibration sample (a running maximum; the      */
/* caller initialises a[] to 0 and may call this once per batch).  The same  */
/* routine on the stored W[C_o, C_i] gives max(|W_j|) of Eq. 4.              */
/* ------------------------------------------------------------------------- */
void sqo_col_absmax(const float *X, int64_t rows, int64_t cols, int64_t ld, float *a) {
    for (int64_t t = 0; t < rows; ++t)
        for (int64_t j = 0; j < cols; ++j) {
            float v = fabsf(X[t * ld + j]);
            if (v > a[j]) a[j] = v;
        }
}

/* Row-wise absolute maximum (per-token statistic of Section 2 / Fig. 3). */
void sqo_row_absmax(const float *X, int64_t rows, int64_t cols, int64_t ld, float *m) {
    for (int64_t t = 0; t < rows; ++t) {
        float r = 0.0f;
        for (int64_t j = 0; j < cols; ++j) {
            float v = fabsf(X[t * ld + j]);
            if (v > r) r = v;
        }
        m[t] = r;
    }
}

/* ------------------------------------------------------------------------- */
/* Eq. 4: s_j = max|X_j|^alpha / max|W_j|^(1-alpha).  Both maxima are floored */
/* (see SQO_ABSMAX_FLOOR); the powers and the quotient are evaluated in fp64  */
/* and rounded once to fp32.                                                  */
/* ------------------------------------------------------------------------- */
void sqo_smooth_scales(const float *act_absmax, const float *w_absmax, int64_t C, float alpha,
                       float *s) {
    double a = (double)alpha;
    for (int64_t j = 0; j < C; ++j) {
        float ax = act_absmax[j] > SQO_ABSMAX_FLOOR ? act_absmax[j] : SQO_ABSMAX_FLOOR;
        float aw = w_absmax[j] > SQO_ABSMAX_FLOOR ? w_absmax[j] : SQO_ABSMAX_FLOOR;
        s[j] = (float)(pow((double)ax, a) / pow((double)aw, 1.0 - a));
    }
}

/* Eq. 3, activation side, folded offline into the producer's parameters
 * (Section 4: "fuse the smoothing factor into previous layers' parameters"):
 * out_j = p_j / s_j in fp32.  The wrapper rounds the result to the parameter
 * dtype, as a checkpoint would store it. */
void sqo_div_by_s(const float *p, const float *s, int64_t C, float *out) {
    for (int64_t j = 0; j < C; ++j) out[j] = p[j] / s[j];
}

/* Eq. 3, weight side: W_hat[o, j] = W[o, j] * s_j (fp32 product, not rounded
 * back to fp16/bf16).  s == NULL means no smoothing (s_j = 1). */
void sqo_scale_weight_cols(const float *W, int64_t N, int64_t K, const float *s, float *What) {
    for (int64_t o = 0; o < N; ++o)
        for (int64_t j = 0; j < K; ++j)
            What[o * K + j] = s ? W[o * K + j] * s[j] : W[o * K + j];
}

/* ------------------------------------------------------------------------- */
/* Eq. 1: Delta = max|X| / (2^(N-1) - 1), N = 8.                              */
/* ------------------------------------------------------------------------- */
float sqo_step_size(float absmax) {
    float m = absmax > SQO_ABSMAX_FLOOR ? absmax : SQO_ABSMAX_FLOOR;
    return m / 127.0f;
}

/* Eq. 1: X_bar = round(X / Delta), evaluated as round(X * inv) with one fp32
 * reciprocal inv = 1/Delta per step size.  The product is NOT rounded before
 * the rounding function is applied: the product of two floats is exact in
 * double, so rint() below sees x * inv itself.  Round-half-to-even, clamped to
 * [-127, 127] (the symmetric range 2^(N-1)-1 of Eq. 1; -128 is never produced). */
static inline int8_t sqo_q(float v, float inv) {
    double r = rint((double)v * (double)inv);
    if (r > 127.0) r = 127.0;
    if (r < -127.0) r = -127.0;
    return (int8_t)r;
}

/* Quantise a [rows, cols] tensor.  delta has one entry per row (per-token /
 * per-output-channel) when per_row != 0, else a single entry (per-tensor). */
void sqo_quantize(const float *V, int64_t rows, int64_t cols, int64_t ld, const float *delta,
                  int per_row, int8_t *Q) {
    for (int64_t t = 0; t < rows; ++t) {
        float inv = 1.0f / delta[per_row ? t : 0];
        for (int64_t j = 0; j < cols; ++j) Q[t * cols + j] = sqo_q(V[t * ld + j], inv);
    }
}

/* Literal Eq. 1 in fp64 (true division, round-half-to-even): diagnostic used
 * to count how often the reciprocal-multiply reading differs from it. */
void sqo_quantize_f64_literal(const float *V, int64_t rows, int64_t cols, int64_t ld,
                              const float *delta, int per_row, int8_t *Q) {
    for (int64_t t = 0; t < rows; ++t) {
        double d = (double)delta[per_row ? t : 0];
        for (int64_t j = 0; j < cols; ++j) {
            double r = rint((double)V[t * ld + j] / d);
            if (r > 127.0) r = 127.0;
            if (r < -127.0) r = -127.0;
            Q[t * cols + j] = (int8_t)r;
        }
    }
}

/* Optional explicit per-channel multiplier (1/s for a producer that is not a
 * LayerNorm): y = x * col_mul_j in fp32. */
void sqo_mul_cols(const float *X, int64_t rows, int64_t cols, int64_t ld, const float *col_mul,
                  float *Y) {
    for (int64_t t = 0; t < rows; ++t)
        for (int64_t j = 0; j < cols; ++j) Y[t * cols + j] = X[t * ld + j] * col_mul[j];
}

/* ------------------------------------------------------------------------- */
/* LayerNorm (Fig. 6 keeps it in floating point; the paper gives no formula, */
/* so the textbook one is used): biased variance, two passes, fp64.          */
/* ------------------------------------------------------------------------- */
void sqo_ln_stats_f64(const float *X, int64_t M, int64_t C, int64_t ld, double eps, double *mu,
                      double *rstd) {
    for (int64_t t = 0; t < M; ++t) {
        double sum = 0.0;
        for (int64_t j = 0; j < C; ++j) sum += (double)X[t * ld + j];
        double mean = sum / (double)C;
        double ss = 0.0;
        for (int64_t j = 0; j < C; ++j) {
            double d = (double)X[t * ld + j] - mean;
            ss += d * d;
        }
        mu[t] = mean;
        rstd[t] = 1.0 / sqrt(ss / (double)C + eps);
    }
}

/* Normative element-wise part of the folded LayerNorm, given fp32 row
 * statistics, as two fused multiply-adds in fp32:
 *   n = fma(x, rstd, -(mu * rstd)),  y = fma(n, gamma_hat_j, beta_hat_j);
 * y is NOT rounded to fp16/bf16 before it is quantised. */
void sqo_ln_apply(const float *X, int64_t M, int64_t C, int64_t ld, const float *mu,
                  const float *rstd, const float *gamma_hat, const float *beta_hat, float *Y) {
    for (int64_t t = 0; t < M; ++t) {
        float shift = -(mu[t] * rstd[t]);
        for (int64_t j = 0; j < C; ++j) {
            float n = fmaf(X[t * ld + j], rstd[t], shift);
            Y[t * C + j] = fmaf(n, gamma_hat[j], beta_hat ? beta_hat[j] : 0.0f);
        }
    }
}

/* fp64 LayerNorm output, for pins. */
void sqo_ln_f64(const float *X, int64_t M, int64_t C, int64_t ld, double eps, const double *gamma,
                const double *beta, double *Y) {
    for (int64_t t = 0; t < M; ++t) {
        double mu, rstd;
        sqo_ln_stats_f64(X + t * ld, 1, C, ld, eps, &mu, &rstd);
        for (int64_t j = 0; j < C; ++j)
            Y[t * C + j] = ((double)X[t * ld + j] - mu) * rstd * gamma[j] + (beta ? beta[j] : 0.0);
    }
}

/* ------------------------------------------------------------------------- */
/* INT8 GEMM of Eq. 2's inner factor: acc[t, o] = sum_j X_bar[t, j] *         */
/* W_bar[o, j], brute force, accumulated in int64 and checked to fit int32.   */
/* Returns the number of accumulators that would overflow int32 (must be 0).  */
/* Rows are independent, so they are spread over the host cores.              */
/* ------------------------------------------------------------------------- */
int64_t sqo_gemm_i32(const int8_t *Xq, const int8_t *Wq, int64_t M, int64_t N, int64_t K,
                     int64_t ldx, int64_t ldw, int32_t *acc) {
    int64_t overflow = 0;
#pragma omp parallel for schedule(static) reduction(+ : overflow) collapse(2)
    for (int64_t t = 0; t < M; ++t)
        for (int64_t o = 0; o < N; ++o) {
            const int8_t *x = Xq + t * ldx;
            const int8_t *w = Wq + o * ldw;
            int64_t sum = 0;
            for (int64_t j = 0; j < K; ++j) sum += (int64_t)((int32_t)x[j] * (int32_t)w[j]);
            if (sum > INT32_MAX || sum < INT32_MIN) ++overflow;
            acc[t * N + o] = (int32_t)sum;
        }
    return overflow;
}

/* The same product with the B operand stored [K, N] (N contiguous), as V is in
 * attention's P.V:  acc[t, o] = sum_j A[t, j] * B[j, o]. */
int64_t sqo_gemm_i32_bt(const int8_t *Aq, const int8_t *Bq, int64_t M, int64_t N, int64_t K,
                        int64_t lda, int64_t ldb, int32_t *acc) {
    int64_t overflow = 0;
#pragma omp parallel for schedule(static) reduction(+ : overflow)
    for (int64_t t = 0; t < M; ++t)
        for (int64_t o = 0; o < N; ++o) {
            int64_t sum = 0;
            for (int64_t j = 0; j < K; ++j)
                sum += (int64_t)((int32_t)Aq[t * lda + j] * (int32_t)Bq[j * ldb + o]);
            if (sum > INT32_MAX || sum < INT32_MIN) ++overflow;
            acc[t * N + o] = (int32_t)sum;
        }
    return overflow;
}

/* ------------------------------------------------------------------------- */
/* Eq. 2: Y = diag(Delta_X) (X_bar W_bar) diag(Delta_W), plus the layer's     */
/* bias and optional ReLU:                                                    */
/*   sc = Delta_X[t] * Delta_W[o]  (fp32);  y = fma((float)acc, sc, bias_o).  */
/* Output is the fp32 value before it is rounded to the output dtype.         */
/* ------------------------------------------------------------------------- */
void sqo_dequant(const int32_t *acc, int64_t M, int64_t N, const float *x_scale, int per_token,
                 const float *w_scale, int per_channel, const float *bias, int relu, float *Y) {
    for (int64_t t = 0; t < M; ++t)
        for (int64_t o = 0; o < N; ++o) {
            float sc = x_scale[per_token ? t : 0] * w_scale[per_channel ? o : 0];
            float y = fmaf((float)acc[t * N + o], sc, bias ? bias[o] : 0.0f);
            if (relu && y < 0.0f) y = 0.0f;
            Y[t * N + o] = y;
        }
}

/* Re-quantise an fp32 tensor with a given multiplier (1/Delta of the consumer,
 * static): q = clamp(round(y * r)), r per column when per_col != 0. */
void sqo_requant(const float *Y, int64_t M, int64_t N, const float *r, int per_col, int8_t *Q) {
    for (int64_t t = 0; t < M; ++t)
        for (int64_t o = 0; o < N; ++o) Q[t * N + o] = sqo_q(Y[t * N + o], r[per_col ? o : 0]);
}

/* Attention BMM dequantisation: y = (float)acc * alpha, alpha a scalar that
 * carries the two static step sizes (and 1/sqrt(d) for Q.K^T). */
void sqo_scale_acc(const int32_t *acc, int64_t n, float alpha, float *Y) {
    for (int64_t i = 0; i < n; ++i) Y[i] = (float)acc[i] * alpha;
}

/* ------------------------------------------------------------------------- */
/* Causal softmax over one [S, S] score matrix (Fig. 6 keeps Softmax in       */
/* floating point), fp32: p = exp(s - max) / sum over j <= i, zero elsewhere. */
/* ------------------------------------------------------------------------- */
void sqo_softmax_causal(const float *S, int64_t rows, int64_t cols, int64_t ld, float *P) {
    for (int64_t i = 0; i < rows; ++i) {
        int64_t n = i + 1 < cols ? i + 1 : cols;
        float mx = S[i * ld];
        for (int64_t j = 1; j < n; ++j)
            if (S[i * ld + j] > mx) mx = S[i * ld + j];
        float sum = 0.0f;
        for (int64_t j = 0; j < n; ++j) {
            float e = expf(S[i * ld + j] - mx);
            P[i * cols + j] = e;
            sum += e;
        }
        for (int64_t j = 0; j < n; ++j) P[i * cols + j] = P[i * cols + j] / sum;
        for (int64_t j = n; j < cols; ++j) P[i * cols + j] = 0.0f;
    }
}

void sqo_softmax_causal_f64(const float *S, int64_t rows, int64_t cols, int64_t ld, double *P) {
    for (int64_t i = 0; i < rows; ++i) {
        int64_t n = i + 1 < cols ? i + 1 : cols;
        double mx = (double)S[i * ld];
        for (int64_t j = 1; j < n; ++j)
            if ((double)S[i * ld + j] > mx) mx = (double)S[i * ld + j];
        double sum = 0.0;
        for (int64_t j = 0; j < n; ++j) {
            double e = exp((double)S[i * ld + j] - mx);
            P[i * cols + j] = e;
            sum += e;
        }
        for (int64_t j = 0; j < n; ++j) P[i * cols + j] /= sum;
        for (int64_t j = n; j < cols; ++j) P[i * cols + j] = 0.0;
    }
}

/* Softmax of rows that each see a prefix of the keys: row i sees the first
 * (first + i) of them.  first = 1 is the causal softmax of a prompt; one row
 * with first = L is the generation stage, where the newest token attends to
 * all L cached positions.  Same fp32 steps, in the same order, as above. */
void sqo_softmax_prefix(const float *S, int64_t rows, int64_t cols, int64_t ld, int64_t first,
                        float *P) {
    for (int64_t i = 0; i < rows; ++i) {
        int64_t n = first + i < cols ? first + i : cols;
        float mx = S[i * ld];
        for (int64_t j = 1; j < n; ++j)
            if (S[i * ld + j] > mx) mx = S[i * ld + j];
        float sum = 0.0f;
        for (int64_t j = 0; j < n; ++j) {
            float e = expf(S[i * ld + j] - mx);
            P[i * cols + j] = e;
            sum += e;
        }
        for (int64_t j = 0; j < n; ++j) P[i * cols + j] = P[i * cols + j] / sum;
        for (int64_t j = n; j < cols; ++j) P[i * cols + j] = 0.0f;
    }
}

/* ------------------------------------------------------------------------- */
/* fp64 truth: the unquantised linear layer Y = X W^T (+ b), stored W [N, K]. */
/* ------------------------------------------------------------------------- */
void sqo_linear_f64(const double *X, const double *W, const double *b, int64_t M, int64_t N,
                    int64_t K, double *Y) {
#pragma omp parallel for schedule(static)
    for (int64_t t = 0; t < M; ++t)
        for (int64_t o = 0; o < N; ++o) {
            double sum = 0.0;
            for (int64_t j = 0; j < K; ++j) sum += X[t * K + j] * W[o * K + j];
            Y[t * N + o] = sum + (b ? b[o] : 0.0);
        }
}
