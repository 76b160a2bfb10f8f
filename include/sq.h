/*
 * sq.h -- C ABI of libsq: the SmoothQuant W8A8 hot path on NVIDIA B200 (sm_100a).
 *
 * Notation follows the paper: an activation X has T tokens (rows, "M") and C_i input
 * channels (columns, "K"); a linear layer has C_o output channels ("N").  Weights are
 * STORED as W[C_o, C_i] row-major, i.e. the transpose of the paper's W in R^{C_i x C_o},
 * so both GEMM operands have the reduction dimension contiguous.  "A" below is the
 * activation dtype, SQ_F16 or SQ_BF16.
 *
 * Conventions shared by every call
 * --------------------------------
 *  - Every pointer is a DEVICE pointer owned by the caller (unless it says "host"),
 *    valid until the work queued on `stream` has finished.  The library never allocates
 *    or frees device memory in these calls and keeps no state between them.
 *  - Tensors are row-major with the innermost dimension contiguous.  Base pointers and
 *    row strides of INT8 operands of the GEMM/BMM must be multiples of 16 bytes
 *    (they are read by TMA); otherwise SQ_ERR_ALIGN.
 *  - `stream` is a cudaStream_t passed as void* (NULL = the legacy default stream).
 *    Calls only enqueue work: they never synchronise and never change the current device.
 *  - The return code reports argument validation and launch errors.  Device-side waits
 *    are bounded; if one expires the kernel records SQ_ERR_TIMEOUT | where << 8 at
 *    workspace[0] (the sticky device status word: written only while it is zero) and returns
 *    instead of hanging; the rows or tiles it had not finished stay unwritten.  This needs a
 *    workspace: the quantisers (sq_quant_act, sq_ln_quant, sq_quant_weight) accept NULL in
 *    their per-token / static / per-channel modes, and a call made without one cannot report
 *    an expired wait (it still returns).  sq_calib_absmax, which takes no workspace, marks the
 *    columns concerned with NaN instead.
 *  - Rounding is round-to-nearest-even everywhere; INT8 codes lie in [-127, 127].
 *  - Inputs must be finite; NaN/Inf give unspecified codes (never a fault).
 *  - A zero-sized problem (M == 0 or N == 0 ...) is a no-op that returns SQ_OK.
 */
#ifndef SQ_H_
#define SQ_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
    SQ_OK = 0,
    SQ_ERR_INVALID_ARG = 1, /* null pointer, bad enum, alpha outside [0,1] ...          */
    SQ_ERR_SHAPE = 2,       /* negative size, stride smaller than the row                */
    SQ_ERR_ALIGN = 3,       /* pointer or stride not aligned as the call requires        */
    SQ_ERR_UNSUPPORTED = 4, /* e.g. K > 133144 (INT32 accumulator could overflow)        */
    SQ_ERR_CUDA = 5,        /* a CUDA runtime/driver call failed (launch, tensor map)    */
    SQ_ERR_TIMEOUT = 6,     /* value stored at workspace[0] by a kernel whose wait ran out */
    SQ_ERR_WORKSPACE = 7    /* workspace missing or smaller than sq_workspace_bytes()    */
} sq_status;

typedef enum { SQ_F16 = 0, SQ_BF16 = 1, SQ_I8 = 2, SQ_I32 = 3 } sq_dtype;

/* Activation quantisation granularity (Table 2): O3, O2, O1. */
typedef enum {
    SQ_PER_TENSOR_STATIC = 0,
    SQ_PER_TENSOR_DYNAMIC = 1,
    SQ_PER_TOKEN_DYNAMIC = 2
} sq_act_gran;

/* Weight quantisation granularity (Fig. 3): one step size, or one per output channel. */
typedef enum { SQ_W_PER_TENSOR = 0, SQ_W_PER_CHANNEL = 1 } sq_w_gran;

typedef enum { SQ_EPI_NONE = 0, SQ_EPI_RELU = 1 } sq_epilogue_act;

/* Operation ids for sq_workspace_bytes(). */
typedef enum {
    SQ_OP_QUANT_ACT = 0,
    SQ_OP_LN_QUANT = 1,
    SQ_OP_QUANT_WEIGHT = 2,
    SQ_OP_GEMM = 3,
    SQ_OP_BMM = 4,
    SQ_OP_GEMM_FUSED_QUANT = 5
} sq_op;

/* Largest reduction length for which |sum| <= 127*127*K stays inside INT32. */
#define SQ_MAX_K 133144

/* Human-readable name of a status code (host pointer to a static string). */
const char* sq_status_str(sq_status s);

/* Bytes of caller-provided workspace `op` needs for the given sizes (host call, no CUDA
 * work).  The workspace must be 256-byte aligned and ZERO-FILLED ONCE by the caller before
 * its first use; every call leaves its first 33 024 bytes (header + arrival counters)
 * zero-filled again except for workspace[0..3], the sticky device status word (0 = no
 * device-side error); what lies beyond is scratch whose content is undefined between calls
 * (partial sums of decode-shaped GEMMs) and is never read before it is written.  M is the
 * token count, N/K as in the call; pass 0 for sizes the op does not have. */
size_t sq_workspace_bytes(sq_op op, int64_t M, int64_t N, int64_t K);

/*
 * Calibration statistic of Section 4 ("s_j = max(|X_j|)", estimated on calibration
 * samples): running per-channel absolute maximum
 *     absmax[j] = max(absmax[j], max_t |X[t, j]|).
 * X: [rows, cols] of dtype `dt` (F16/BF16) with row stride `ld` elements (ld >= cols).
 * absmax_inout: [cols] fp32, updated in place; the caller zero-initialises it before the
 * first batch and may call once per calibration batch.  Applied to the stored weight
 * W[C_o, C_i] it yields max(|W_j|) of Eq. 4 (one value per INPUT channel).
 * The fast path needs X 16-byte aligned with cols and ld multiples of 8; other shapes run
 * a slower element-wise kernel.  Batches of 2^27 elements or more stream through bulk copies
 * whose waits are bounded: should one never land, the columns concerned receive NaN.
 */
sq_status sq_calib_absmax(const void* X, sq_dtype dt, int64_t rows, int64_t cols, int64_t ld,
                          float* absmax_inout, void* stream);

/*
 * Calibration of a per-tensor STATIC step with the largest tokens set aside (Section 5.2: for
 * GLM-130B the top 2 % of tokens are clipped when the static step sizes are calibrated).
 * sq_token_absmax: token_absmax[t] = max_j |X[t, j]| for the M tokens of one calibration batch
 * (X: [M, C] of dtype dt, row stride ld elements; C and ld multiples of 8, X 16-byte aligned);
 * the caller lays the batches' results side by side in one [T] array.
 * sq_clipped_absmax: of those T values the n_clip largest are dropped (at least one value is
 * always kept) and the largest of the rest is written to absmax_out[0]; step_out (nullable)
 * receives the step size max(absmax, 1e-5) / 127 of Eq. 1.  n_clip = 0 gives the plain maximum.
 * The selection is exact (radix selection on the bit patterns; values must be >= 0, which
 * sq_token_absmax guarantees).  T < 2^32.
 */
sq_status sq_token_absmax(const void* X, sq_dtype dt, int64_t M, int64_t C, int64_t ld, float* token_absmax,
                          void* stream);
sq_status sq_clipped_absmax(const float* token_absmax, int64_t T, int64_t n_clip, float* absmax_out,
                            float* step_out, void* stream);

/*
 * Smoothing factor, Eq. 4:  s_j = max|X_j|^alpha / max|W_j|^(1-alpha),  j < C.
 * act_absmax, w_absmax: [C] fp32 (both floored at 1e-5 so that s_j is finite and
 * non-zero); alpha in [0, 1] else SQ_ERR_INVALID_ARG; s_out: [C] fp32.  The powers are
 * evaluated in double precision and rounded once to fp32.  s_inv_out: optional [C] fp32,
 * receives 1/s_j (fp32 division) -- the explicit activation-side multiplier of Eq. 3 for a
 * producer whose parameters cannot absorb it (see col_mul of sq_quant_act).
 */
sq_status sq_smooth_scales(const float* act_absmax, const float* w_absmax, int64_t C, float alpha,
                           float* s_out, float* s_inv_out, void* stream);

/*
 * Eq. 3, activation side, folded offline into the preceding LayerNorm (Section 4: the
 * smoothing factor is fused into the previous layer's parameters, so no scaling runs at
 * inference):  gamma_out = gamma / s,  beta_out = beta / s  (fp32 division, result rounded
 * to `dt`).  gamma, beta, gamma_out, beta_out: [C] of dtype dt; beta and beta_out may both
 * be NULL.  In-place (gamma_out == gamma) is allowed.
 */
sq_status sq_fold_ln_weight(const void* gamma, const void* beta, sq_dtype dt, const float* s,
                            int64_t C, void* gamma_out, void* beta_out, void* stream);

/*
 * Eq. 3 weight side and Eq. 1:  W_hat[o, j] = W[o, j] * s_j (fp32, s == NULL means s_j = 1),
 * Delta_w = max|W_hat| / 127 per output channel (row) or per tensor,
 * Wq = clamp(round(W_hat / Delta_w), -127, 127).
 * W: [N, K] dtype dt, contiguous.  Wq: [N, K] int8.  w_scale: [N] (per channel) or [1]
 * fp32, receives Delta_w.  workspace: sq_workspace_bytes(SQ_OP_QUANT_WEIGHT, ...) bytes
 * (required by the per-tensor mode; in the per-channel mode it may be NULL and only serves as
 * the device status word).  K must be a multiple of 8 and W 16-byte aligned.
 * This is the one call of the library that WRITES weights, and sq_w8a8_gemm with M <= 32 starts
 * fetching Wq before it waits for the launch in front of it; the call therefore ends with an
 * empty, fully serialised launch, so that it may be followed directly by a GEMM on the stream.
 */
sq_status sq_quant_weight(const void* W, sq_dtype dt, int64_t N, int64_t K, const float* s,
                          sq_w_gran g, int8_t* Wq, float* w_scale, void* workspace,
                          size_t ws_bytes, void* stream);

/*
 * Eq. 1 on an activation tensor, at the three granularities of Table 2.
 *   per-token dynamic : Delta_t = max_j |x[t, j]| / 127, written to x_scale[t]   ([M])
 *   per-tensor dynamic: one Delta from the whole [M, C] of this call -> x_scale[0]
 *   per-tensor static : Delta = x_scale[0] is an INPUT (from calibration); larger values
 *                       saturate at +-127
 * Xq = clamp(round(x * (1/Delta)), -127, 127); maxima are floored at 1e-5.
 * X: [M, C] dtype dt, contiguous, 16-byte aligned, C a multiple of 8.  col_mul: optional
 * [C] fp32 multiplier applied first in fp32 (an explicit 1/s when the producer is not a
 * LayerNorm); NULL for none.  Xq: [M, C] int8.  workspace: required by the per-tensor dynamic
 * mode (sq_workspace_bytes(SQ_OP_QUANT_ACT, ...)); otherwise optional, word 0 = device status.
 */
sq_status sq_quant_act(const void* X, sq_dtype dt, int64_t M, int64_t C, sq_act_gran g,
                       const float* col_mul, int8_t* Xq, float* x_scale, void* workspace,
                       size_t ws_bytes, void* stream);

/*
 * Two pieces for tensor-parallel serving of the W8A8 linears (Section 5.3 runs the larger models
 * with FasterTransformer's tensor parallelism over up to 8 GPUs: QKV / FC1 split by output
 * channels, out-proj / FC2 split by INPUT channels, partial results summed across GPUs).
 *
 * sq_quant_act_given_absmax: Eq. 1 per token when a token's channels are spread over several ranks.
 * The per-token maximum must then be the maximum over ALL ranks' slices, or the ranks' codes would
 * have different step sizes and their INT32 partial sums could not be added.  Each rank takes
 * sq_token_absmax of its slice, the ranks exchange a max-all-reduce of those [M] values, and this
 * call quantises the local slice with Delta_t = max(row_absmax[t], 1e-5) / 127 (written to
 * x_scale[t]; identical on every rank).  X: [M, C] slice, contiguous; row_absmax: [M] fp32 INPUT.
 * With row_absmax the slice's own maxima this is sq_quant_act(SQ_PER_TOKEN_DYNAMIC), bit for bit.
 *
 * sq_dequant_acc: Eq. 2 on INT32 accumulators that already sit in memory -- what the epilogue of
 * sq_w8a8_gemm / sq_w8a8_gemm_residual computes, operation for operation, as a pass of its own:
 *     y = fma((float)acc[t, o], x_scale[t] * w_scale[o], bias[o]), ReLU, then round to F16 / BF16
 *     (optionally + residual, as in sq_w8a8_gemm_residual) or clamp(round(y * requant_mul)) to I8.
 * A row-parallel layer runs sq_w8a8_gemm with out_dt = SQ_I32 on every rank (raw partial sums),
 * the ranks add them with an INT32 sum-all-reduce (exact: the result is bit for bit that of the
 * unsharded layer), and this call dequantises the sum once.  acc: [M, N] int32, row stride ld_acc
 * (a multiple of 4), 16-byte aligned; N a multiple of 8; Y: row stride ldy a multiple of 8.
 */
sq_status sq_quant_act_given_absmax(const void* X, sq_dtype dt, int64_t M, int64_t C, const float* row_absmax,
                                    int8_t* Xq, float* x_scale, void* workspace, size_t ws_bytes, void* stream);
sq_status sq_dequant_acc(const int32_t* acc, int64_t ld_acc, int64_t M, int64_t N, const float* x_scale,
                         int x_scale_is_per_token, const float* w_scale, int w_scale_is_per_channel, const void* bias,
                         sq_dtype bias_dt, sq_epilogue_act act, const float* requant_mul, int requant_is_per_channel,
                         const void* residual, int64_t ld_res, void* Y, sq_dtype out_dt, int64_t ldy, void* stream);

/*
 * Fused LayerNorm (with the smoothing factor already folded into gamma_hat, beta_hat by
 * sq_fold_ln_weight) + Eq. 1, one pass over X:
 *     mu_t, var_t = mean and biased variance of row t: fp32, one pass -- per-thread (mean, sum of
 *                   squared deviations) pairs merged with the parallel-variance update; rows whose
 *                   length does not divide evenly take the sum first and the deviations second,
 *     rstd_t = 1/sqrt(var_t + eps),
 *     n = fma(x, rstd_t, -(mu_t * rstd_t)),  y = fma(n, gamma_hat_j, beta_hat_j)     (fp32),
 * then y is quantised exactly as in sq_quant_act WITHOUT being rounded to A first.  The
 * statistics are a tolerance quantity (within 1e-6 relative of the fp64 two-pass values); the
 * element-wise part, given them, is bit-exact.
 * X: [M, C] dtype dt; gamma_hat, beta_hat: [C] dtype dt (beta_hat may be NULL).
 * dbg_mean_rstd: optional [2*M] fp32, receives mu_t at [2t] and rstd_t at [2t+1] so that a
 * checker can reproduce the element-wise part bit for bit.  Other arguments as sq_quant_act.
 */
sq_status sq_ln_quant(const void* X, sq_dtype dt, int64_t M, int64_t C, const void* gamma_hat,
                      const void* beta_hat, float eps, sq_act_gran g, int8_t* Xq, float* x_scale,
                      float* dbg_mean_rstd, void* workspace, size_t ws_bytes, void* stream);

/* Largest token count sq_ln_quant_tensor_noalloc accepts: it sizes the built-in scratch. */
#define SQ_NOALLOC_MAX_ROWS 16384

/*
 * The paper has no counterpart for this call; it exists for deployment.  Some callers cannot
 * give the library a workspace because they cannot allocate device memory at all: a plug-in
 * that is handed only its input and output buffers, code inside a serving engine whose memory
 * arena is sized up front, a latency-critical loop in which cudaMalloc (which may synchronise
 * the device) is forbidden.  For them this is sq_ln_quant in its per-tensor DYNAMIC mode
 * (one step size from the whole [M, C] of the call, written to x_scale[0]) with the scratch it
 * needs -- one running-maximum word and two floats of LayerNorm statistics per row -- held
 * in a fixed array inside the library image instead of a caller workspace.  It calls no
 * allocation routine of any kind.  Results are identical to sq_ln_quant(...,
 * SQ_PER_TENSOR_DYNAMIC, ...).
 *
 *  - M <= SQ_NOALLOC_MAX_ROWS, else SQ_ERR_UNSUPPORTED (nothing is launched).  The array costs
 *    about 128 KB of device memory on every GPU that loads the library, until process exit.
 *  - The first call on each device looks up the array's device address (a host-side query,
 *    made with that device current).  Make that first call outside any stream capture.
 *  - All calls on a device share the one array, and it keeps the previous call's contents; the
 *    call re-zeroes what must start at zero.  Calls that can overlap on the GPU (different
 *    streams without an ordering between them, or concurrent host threads) race on it and
 *    give wrong step sizes: order them, or use sq_ln_quant with separate workspaces.
 *  - Other arguments, alignment rules and arithmetic: exactly as sq_ln_quant.
 */
sq_status sq_ln_quant_tensor_noalloc(const void* X, sq_dtype dt, int64_t M, int64_t C,
                                     const void* gamma_hat, const void* beta_hat, float eps,
                                     int8_t* Xq, float* x_scale, void* stream);

/*
 * The W8A8 linear layer, Eq. 2:
 *     acc[t, o] = sum_j Xq[t, j] * Wq[o, j]                         (INT32, exact)
 *     y[t, o]   = fma((float)acc, x_scale[t] * w_scale[o], bias[o]) (fp32), optional ReLU
 * and then ONE of
 *     Y = round_to(out_dt)(y)                         out_dt = SQ_F16 / SQ_BF16
 *     Y = clamp(round(y * requant_mul[o or 0]))       out_dt = SQ_I8 (requant_mul != NULL)
 *     Y = acc                                         out_dt = SQ_I32 (raw accumulators;
 *                                                     scales, bias, ReLU ignored)
 * Xq: [M, K] int8, row stride K.  Wq: [N, K] int8, row stride K.  K a multiple of 16,
 * K <= SQ_MAX_K.  x_scale: [M] if x_scale_is_per_token else [1]; w_scale: [N] if
 * w_scale_is_per_channel else [1].  bias: [N] of dtype bias_dt (F16/BF16) or NULL.
 * requant_mul: [N] if requant_is_per_channel else [1]; required iff out_dt == SQ_I8.
 * row_absmax_out: optional [M] fp32, caller-zeroed; receives max_o |y[t, o]| (after ReLU,
 * before output rounding) via atomic max, so that the next layer's per-token step size
 * needs no extra pass.  Y: [M, N] with row stride ldy elements.
 * workspace: word 0 is the device status.  sq_workspace_bytes(SQ_OP_GEMM, M, N, K) bytes are
 * REQUIRED for M <= 32 (the weight-streaming kernel parks partial sums there) and RECOMMENDED
 * above: when the tiles do not fill the last wave of thread-block groups (or, with few tokens
 * against a narrow weight, fill at most half of the only wave), the tiles of that wave are cut
 * along K and their INT32 partial sums meet in the workspace (integer sums: the result does not
 * depend on it).  With a smaller workspace (>= 256 bytes) the cut is not made and the call is
 * merely slower.
 */
sq_status sq_w8a8_gemm(const int8_t* Xq, const int8_t* Wq, int64_t M, int64_t N, int64_t K,
                       const float* x_scale, int x_scale_is_per_token, const float* w_scale,
                       int w_scale_is_per_channel, const void* bias, sq_dtype bias_dt,
                       sq_epilogue_act act, const float* requant_mul, int requant_is_per_channel,
                       float* row_absmax_out, void* Y, sq_dtype out_dt, int64_t ldy,
                       void* workspace, size_t ws_bytes, void* stream);

/*
 * The same W8A8 linear with the block's residual connection folded into its epilogue (Fig. 6
 * keeps the residual stream in FP16; the two linears that feed it are out-proj and FC2):
 *     y[t, o]  = round_to(out_dt)(fma((float)acc[t, o], Delta_x * Delta_w, bias[o]))   as above
 *     Y[t, o]  = round_to(out_dt)((float)y[t, o] + (float)residual[t, o])
 * i.e. bit for bit what sq_w8a8_gemm followed by sq_residual_add gives, without writing y and
 * reading it back.  out_dt: SQ_F16 or SQ_BF16; residual: [M, N] of that type, row stride ld_res
 * elements (>= N, a multiple of 8), 16-byte aligned, N a multiple of 8; must not overlap Y.  No
 * activation function, no re-quantisation, no row_absmax_out.  Other arguments, workspace and
 * errors as for sq_w8a8_gemm.
 */
sq_status sq_w8a8_gemm_residual(const int8_t* Xq, const int8_t* Wq, int64_t M, int64_t N, int64_t K,
                                const float* x_scale, int x_scale_is_per_token, const float* w_scale,
                                int w_scale_is_per_channel, const void* bias, sq_dtype bias_dt,
                                const void* residual, int64_t ld_res, void* Y, sq_dtype out_dt, int64_t ldy,
                                void* workspace, size_t ws_bytes, void* stream);

/*
 * The generation-stage W8A8 linear (M <= 32 tokens) with the activation quantiser INSIDE the GEMM
 * kernel.  With a handful of tokens the layer is a single pass over the INT8 weights (the paper's
 * appendix on weight-only quantisation: this stage is memory-bound), and a quantiser launched in
 * front of it costs a tenth of that pass; here the kernel's first weight slices are already in
 * flight while thread block r turns token row r into INT8 codes:
 *     [ y = LayerNorm(x; gamma_hat, beta_hat, eps)      when gamma_hat != NULL, as sq_ln_quant ]
 *     Delta_t = max_j |y[t, j]| / 127 (SQ_PER_TOKEN_DYNAMIC)   or   Delta = x_scale[0] (SQ_PER_TENSOR_STATIC)
 *     Xq = clamp(round(y * (1 / Delta)), -127, 127)                                        (Eq. 1)
 * followed by exactly the arithmetic of sq_w8a8_gemm / sq_w8a8_gemm_residual (Eq. 2, bias, ReLU,
 * re-quantisation, residual add).  Codes and step sizes equal those of sq_quant_act (bit for bit)
 * and of sq_ln_quant (bit for bit given the same row statistics; the statistics are a two-pass fp32
 * reduction in another order, a tolerance quantity).
 * X: [M, K] of x_dt (F16/BF16), contiguous, 16-byte aligned; K a multiple of 16, K <= SQ_MAX_K.
 * gamma_hat, beta_hat: [K] of x_dt or NULL (beta_hat may be NULL alone).  g: SQ_PER_TOKEN_DYNAMIC or
 * SQ_PER_TENSOR_STATIC; SQ_PER_TENSOR_DYNAMIC and M > 32 return SQ_ERR_UNSUPPORTED (use sq_quant_act /
 * sq_ln_quant followed by sq_w8a8_gemm).  x_scale: static: [1] INPUT; dynamic: optional [M] OUTPUT
 * (NULL keeps the step sizes in the workspace).  Xq_out: optional [M, K] int8 OUTPUT, 16-byte aligned
 * (NULL keeps the codes in the workspace).  dbg_mean_rstd: optional [2 M] fp32, as in sq_ln_quant.
 * residual (nullable): as in sq_w8a8_gemm_residual (then out_dt is F16/BF16, no ReLU / re-quantisation).
 * out_dt: SQ_F16 / SQ_BF16 / SQ_I8.  Other arguments as sq_w8a8_gemm.
 * workspace: sq_workspace_bytes(SQ_OP_GEMM_FUSED_QUANT, M, N, K) bytes, REQUIRED.  The thread blocks
 * of the call meet once on a counter in it (bounded wait; on expiry SQ_ERR_TIMEOUT | 10 << 8 or
 * | 11 << 8 in the status word), so two calls that can overlap on the GPU must not share a workspace.
 */
sq_status sq_w8a8_gemm_fused_quant(const void* X, sq_dtype x_dt, int64_t M, int64_t N, int64_t K,
                                   const void* gamma_hat, const void* beta_hat, float eps, sq_act_gran g,
                                   float* x_scale, int8_t* Xq_out, float* dbg_mean_rstd, const int8_t* Wq,
                                   const float* w_scale, int w_scale_is_per_channel, const void* bias,
                                   sq_dtype bias_dt, sq_epilogue_act act, const float* requant_mul,
                                   int requant_is_per_channel, const void* residual, int64_t ld_res, void* Y,
                                   sq_dtype out_dt, int64_t ldy, void* workspace, size_t ws_bytes, void* stream);

/*
 * INT8 batched matmul for attention (Fig. 6: the BMMs run in INT8):
 * for every b < batch, h < heads
 *     acc = A[b,h] * B[b,h]^T   (B stored [N, K], K contiguous;  b_is_kn == 0)   e.g. Q.K^T
 *     acc = A[b,h] * B[b,h]     (B stored [K, N], N contiguous;  b_is_kn != 0)   e.g. P.V
 *     C[b,h] = round_to(out_dt)((float)acc * alpha)          out_dt = SQ_F16 / SQ_BF16
 *     C[b,h] = clamp(round(((float)acc * alpha) * *requant_mul))   out_dt = SQ_I8
 *     C[b,h] = acc                                           out_dt = SQ_I32
 * A[b,h]: [M, K] int8.  strideX[3] = {batch stride, head stride, row stride} in ELEMENTS
 * (HOST arrays); the innermost dimension is contiguous.  All strides of A and B must be
 * multiples of 16; K a multiple of 16; with b_is_kn, N must be a multiple of 16 and at
 * most 128 (the head dimension).  alpha carries the operands' static step sizes (and
 * 1/sqrt(d) for Q.K^T).  requant_mul: device pointer to one fp32, required iff out_dt == SQ_I8.
 * Strided views let Q, K, V be read in place from the fused QKV GEMM output [T, 3*H*d].
 * causal != 0 declares causal self-attention (M == number of keys).  For Q.K^T, score tiles that
 * lie entirely above the diagonal (first key > last query of the tile) are then neither computed
 * nor written -- sq_softmax_quant_p never reads them.  For P.V, where P is zero above the
 * diagonal, the K slices beyond a tile's last query are skipped; the result is unchanged.
 */
sq_status sq_w8a8_bmm(const int8_t* A, const int8_t* B, int64_t batch, int64_t heads, int64_t M,
                      int64_t N, int64_t K, const int64_t strideA[3], const int64_t strideB[3],
                      int b_is_kn, int causal, float alpha, const float* requant_mul, void* C, sq_dtype out_dt,
                      const int64_t strideC[3], void* workspace, size_t ws_bytes, void* stream);

/*
 * Fused causal INT8 self-attention (Fig. 6: both BMMs in INT8, softmax in floating point) over
 * the fused QKV code buffer:
 *     s[i, j]  = (float)(Q_i . K_j) * alpha_qk                      (INT32 accumulate; fp32 scores)
 *     p[i, j]  = exp(s[i, j] - max_i) / sum_{j' <= i} exp(s[i, j'] - max_i),   0 for j > i
 *     P[i, j]  = round(127 * p[i, j])                               (step 1/127)
 *     out[i,:] = clamp(round(((float)(P_i . V) * alpha_pv) * requant_mul))
 * i.e. the chain sq_w8a8_bmm -> sq_softmax_quant_p -> sq_w8a8_bmm with the scores kept in fp32
 * instead of being rounded to a 16-bit type, and without writing the [S, S] score and probability
 * matrices to memory.  exp and the row sums are not bit-reproducible against another
 * implementation, so individual P codes (and, through them, output codes) may differ by one
 * where a value sits on a rounding boundary.  alpha_qk must be positive.
 * qkv: [B*S, 3*H*d] int8, row-major (Q | K | V column blocks, head h at columns h*d .. of each),
 * 16-byte aligned; d must be 128 (else SQ_ERR_UNSUPPORTED); S a multiple of 16.
 * alpha_qk = Delta_q * Delta_k / sqrt(d); alpha_pv = Delta_v / 127; requant_mul: device pointer to
 * 1 / Delta_attn.  out: [B*S, H*d] int8.  workspace: sq_workspace_bytes(SQ_OP_BMM, ...) bytes.
 */
sq_status sq_w8a8_attention(const int8_t* qkv, int64_t B, int64_t H, int64_t S, int64_t d,
                            float alpha_qk, float alpha_pv, const float* requant_mul,
                            int8_t* out, void* workspace, size_t ws_bytes, void* stream);

/*
 * INT8 key/value cache for the generation stage (Section 7, Discussion: quantising activations
 * also reduces the memory held by the KV cache).  Layout, chosen for the reader below:
 *     k_cache [B, H, L_max, d]      int8: one key per d-byte row;
 *     v_cache [B, H, L_max/4, d, 4] int8: the values of four consecutive positions 4g .. 4g+3 of
 *                                   one channel share a 32-bit word (position 4g+r, channel c at
 *                                   byte ((g*d + c)*4 + r) of the head's block).
 * sq_kv_cache_write copies the K and V codes of T tokens per sequence out of the fused QKV code
 * buffer qkv [B*T, ld] (row b*T + t; Q | K | V column blocks of H*d, head h at columns h*d ..)
 * to cache positions pos0[b] .. pos0[b] + T - 1 of sequence b.  pos0: device pointer to B int32
 * (nullable = all zero).  T = prompt length fills the cache after the prompt pass; T = 1 appends
 * the newest token.  A sequence whose run would leave [0, L_max) is skipped and the device
 * status word is set (SQ_ERR_SHAPE).  d must be 128; L_max a multiple of 4; ld a multiple of 16;
 * pointers 16-byte aligned.  workspace: at least 256 bytes, 256-byte aligned; word 0 = device status.
 */
sq_status sq_kv_cache_write(const int8_t* qkv, int64_t ld, int64_t B, int64_t T, int64_t H, int64_t d,
                            const int32_t* pos0, int8_t* k_cache, int8_t* v_cache, int64_t L_max,
                            void* workspace, size_t ws_bytes, void* stream);

/*
 * Generation-stage attention of the newest token of each sequence over the INT8 cache, in the
 * precision mapping of Fig. 6 (both products in INT8, softmax in floating point):
 *     s[j]   = (float)(q . K_j) * alpha_qk                          j < seq_lens[b]
 *     p[j]   = exp(s[j] - max) / sum_j' exp(s[j'] - max)
 *     P[j]   = round(127 * p[j])                                    (step 1/127)
 *     out[:] = ((float)(sum_j P[j] * V_j)) * alpha_pv               -> 16-bit float, or
 *              clamp(round(that * requant_mul)) -> int8
 * i.e. what sq_w8a8_attention computes for the last row of a prompt of seq_lens[b] tokens.
 * exp and the sum are not bit-reproducible against another implementation, so P codes (and
 * through them output codes) may differ by one where a value sits on a rounding boundary; for a
 * given shape the result is deterministic.  alpha_qk must be positive.
 * q: [B, ldq] int8, head h at columns h*d .. (it may point into the QKV code buffer, ldq = 3*H*d);
 * k_cache / v_cache: as above; seq_lens: device pointer to B int32, the number of valid positions
 * INCLUDING the newest token.  k_new / v_new (both NULL, or both given): [B, ld_new] int8 rows
 * holding the newest token's k and v codes (head h at columns h*d ..; they may point into the
 * QKV code buffer).  When NULL the caller has already written them to the cache
 * (sq_kv_cache_write with T = 1).  When given, position seq_lens[b] - 1 of the cache is NOT read:
 * its key and value are taken from these rows, and the kernel stores them at that position
 * for the steps to come -- one launch less per generated token; the result is the same.
 * max_len: a host-side upper bound of seq_lens[] (<= L_max) that sizes shared memory and the
 * split of one sequence over a thread-block cluster -- a longer sequence is truncated to max_len
 * and the device status word is set (SQ_ERR_SHAPE): its output is the attention over the first
 * max_len cached positions and k_new / v_new are NOT appended (the cache is left as it was);
 * seq_lens[b] <= 0 gives a zero output row (and appends nothing).
 * out: [B, ldo] of out_dt (SQ_I8 needs requant_mul, a device pointer to one fp32; SQ_F16 / SQ_BF16
 * ignore it).  d must be 128 (else SQ_ERR_UNSUPPORTED), L_max a multiple of 4, ldq and ld_new
 * multiples of 16, q / k_new / v_new / caches 16-byte aligned; max_len beyond what eight CTAs can
 * hold in shared memory (about 300 000 positions) is SQ_ERR_UNSUPPORTED.  workspace: >= 256 bytes;
 * word 0 = device status.
 */
sq_status sq_w8a8_decode_attention(const int8_t* q, int64_t ldq, int8_t* k_cache, int8_t* v_cache,
                                   const int8_t* k_new, const int8_t* v_new, int64_t ld_new,
                                   const int32_t* seq_lens, int64_t B, int64_t H, int64_t d, int64_t L_max,
                                   int64_t max_len, float alpha_qk, float alpha_pv, const float* requant_mul,
                                   void* out, sq_dtype out_dt, int64_t ldo, void* workspace, size_t ws_bytes,
                                   void* stream);

/*
 * Attention plumbing between the two BMMs (Fig. 6 keeps Softmax in floating point):
 * causal softmax over each [S, S] score matrix followed by quantisation of the
 * probabilities with the fixed step 1/127 (softmax output lies in [0, 1]):
 *     p[i, j] = exp(s[i, j] - max_i) / sum_{j' <= i} exp(s[i, j'] - max_i),  0 for j > i
 *     Pq[i, j] = round(127 * p[i, j])
 * scores: [n_mat, S, S] dtype dt (F16/BF16), contiguous; Pq: [n_mat, S, S] int8.
 * S a multiple of 8.  Computed in fp32; exp and the row sum are not bit-reproducible
 * against another implementation, so codes may differ by one at rounding ties.
 */
sq_status sq_softmax_quant_p(const void* scores, sq_dtype dt, int64_t n_mat, int64_t S, int8_t* Pq,
                             void* stream);

/*
 * Residual add around a sub-layer (pre-LayerNorm block): out = a + b in fp32, rounded to dt.
 * a, b, out: [n] dtype dt, n a multiple of 8, 16-byte aligned; out may alias a.
 */
sq_status sq_residual_add(const void* a, const void* b, sq_dtype dt, int64_t n, void* out,
                          void* stream);

/*
 * Self-test of the bounded-wait machinery that every tensor-core kernel of the library uses
 * (no counterpart in the paper).  Launches one small CTA that waits, with a budget of
 * `budget_cycles` SM clock cycles, on an mbarrier that nothing will ever complete; when the
 * budget runs out the kernel stores SQ_ERR_TIMEOUT | (where << 8) into *status_word and returns
 * normally -- the same path a real kernel takes if a TMA copy or an MMA never signals.  The
 * context stays usable.  status_word: device pointer to a zero-initialised uint32.
 */
sq_status sq_selftest_bounded_wait(uint32_t* status_word, uint32_t budget_cycles, void* stream);

/*
 * The same self-test for the bounded wait of the row kernels (sq_quant_act, sq_ln_quant,
 * sq_quant_weight wait for each row's bulk copy on an mbarrier; no counterpart in the paper): one
 * thread waits `budget_cycles` on a barrier nothing completes, then stores
 * SQ_ERR_TIMEOUT | (5 << 8) into *status_word exactly as those kernels do, and returns.
 */
sq_status sq_selftest_row_wait(uint32_t* status_word, uint32_t budget_cycles, void* stream);

#ifdef __cplusplus
}
#endif
#endif /* SQ_H_ */
