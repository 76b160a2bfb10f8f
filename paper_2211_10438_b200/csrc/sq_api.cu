// extern "C" entry points of libsq: argument validation and kernel dispatch only.
#include "sq_common.cuh"
#include <algorithm>

#include "sq_kernels.h"

using namespace sq;

namespace {

inline bool is_act_dtype(sq_dtype dt) { return dt == SQ_F16 || dt == SQ_BF16; }
inline cudaStream_t as_stream(void* s) { return static_cast<cudaStream_t>(s); }
inline float* ws_absmax(void* ws) { return reinterpret_cast<float*>(static_cast<char*>(ws) + kWsAbsmaxOff); }
inline float* ws_stats(void* ws) { return reinterpret_cast<float*>(static_cast<char*>(ws) + kWsHeader); }
inline bool ws_ok(const void* ws, size_t have, size_t need) {
    return ws != nullptr && have >= need && (reinterpret_cast<uintptr_t>(ws) & 255) == 0;
}

// shared body of sq_quant_act / sq_ln_quant / sq_quant_weight
sq_status quant_rows_common(const void* X, sq_dtype dt, int64_t M, int64_t C, const float* col_mul,
                            const void* gamma, const void* beta, float eps, bool ln, int gran /*sq_act_gran*/,
                            int8_t* Xq, float* scale, float* dbg_stats, void* workspace, size_t ws_bytes,
                            size_t ws_need, cudaStream_t st) {
    // word 0 of a workspace, when the caller gave one, receives the device status of an expired wait
    uint32_t* status = ws_ok(workspace, ws_bytes, sizeof(uint32_t)) ? static_cast<uint32_t*>(workspace) : nullptr;
    if (gran == SQ_PER_TOKEN_DYNAMIC)
        return row_quant(X, dt, M, C, col_mul, gamma, beta, eps, ln, ROW_DYNAMIC, Xq, scale, nullptr,
                         dbg_stats, 0, status, st);
    if (gran == SQ_PER_TENSOR_STATIC)
        return row_quant(X, dt, M, C, col_mul, gamma, beta, eps, ln, ROW_GIVEN_SCALE, Xq, scale, nullptr,
                         dbg_stats, 0, status, st);
    // per-tensor dynamic: pass 1 folds every row's maximum into one word (and keeps the
    // LayerNorm statistics), pass 2 quantises with the step derived from it
    if (!ws_ok(workspace, ws_bytes, ws_need)) return SQ_ERR_WORKSPACE;
    float* word = ws_absmax(workspace);
    float* stats = ln ? (dbg_stats ? dbg_stats : ws_stats(workspace)) : nullptr;
    sq_status s = row_quant(X, dt, M, C, col_mul, gamma, beta, eps, ln, ROW_ABSMAX_ONLY, nullptr, nullptr,
                            word, stats, 0, status, st);
    if (s != SQ_OK) return s;
    s = row_quant(X, dt, M, C, col_mul, gamma, beta, eps, ln, ROW_FROM_ABSMAX_WORD, Xq, scale, word, stats,
                  ln ? 1 : 0, status, st);
    if (s != SQ_OK) return s;
    SQ_CUDA_OK(cudaMemsetAsync(word, 0, sizeof(float), st));  // leave the workspace zero-filled
    if (ln && !dbg_stats) SQ_CUDA_OK(cudaMemsetAsync(stats, 0, (size_t)M * 2 * sizeof(float), st));
    return SQ_OK;
}

}  // namespace

extern "C" {

const char* sq_status_str(sq_status s) {
    switch (s) {
        case SQ_OK: return "SQ_OK";
        case SQ_ERR_INVALID_ARG: return "SQ_ERR_INVALID_ARG";
        case SQ_ERR_SHAPE: return "SQ_ERR_SHAPE";
        case SQ_ERR_ALIGN: return "SQ_ERR_ALIGN";
        case SQ_ERR_UNSUPPORTED: return "SQ_ERR_UNSUPPORTED";
        case SQ_ERR_CUDA: return "SQ_ERR_CUDA";
        case SQ_ERR_TIMEOUT: return "SQ_ERR_TIMEOUT";
        case SQ_ERR_WORKSPACE: return "SQ_ERR_WORKSPACE";
    }
    return "SQ_ERR_UNKNOWN";
}

size_t sq_workspace_bytes(sq_op op, int64_t M, int64_t N, int64_t K) {
    (void)K;
    switch (op) {
        case SQ_OP_LN_QUANT: return kWsHeader + (size_t)(M > 0 ? M : 0) * 2 * sizeof(float);
        case SQ_OP_GEMM:  // decode-shaped calls keep split-K partial sums in the workspace
            if (!(M > 0 && N > 0 && K > 0)) return kWsHeader;
            if (M <= 32) return decode_workspace_bytes(M, N);
            return gemm_workspace_bytes(M, N, K);
        case SQ_OP_GEMM_FUSED_QUANT:  // the same + the codes and step sizes of the prologue quantiser
            if (!(M > 0 && M <= 32 && N > 0 && K > 0)) return kWsHeader;
            return decode_fused_workspace_bytes(M, N, K);
        case SQ_OP_QUANT_ACT:
        case SQ_OP_QUANT_WEIGHT:
        case SQ_OP_BMM: return kWsHeader;
    }
    return kWsHeader;
}

sq_status sq_calib_absmax(const void* X, sq_dtype dt, int64_t rows, int64_t cols, int64_t ld,
                          float* absmax_inout, void* stream) {
    if (!is_act_dtype(dt)) return SQ_ERR_INVALID_ARG;
    if (rows < 0 || cols < 0 || ld < cols) return SQ_ERR_SHAPE;
    if (rows == 0 || cols == 0) return SQ_OK;
    if (!X || !absmax_inout) return SQ_ERR_INVALID_ARG;
    return calib_absmax(X, dt, rows, cols, ld, absmax_inout, as_stream(stream));
}

sq_status sq_token_absmax(const void* X, sq_dtype dt, int64_t M, int64_t C, int64_t ld, float* out,
                          void* stream) {
    if (!is_act_dtype(dt)) return SQ_ERR_INVALID_ARG;
    if (M < 0 || C < 0 || ld < C) return SQ_ERR_SHAPE;
    if (M == 0) return SQ_OK;
    if (!X || !out) return SQ_ERR_INVALID_ARG;
    if (C % 8 != 0 || ld % 8 != 0 || !aligned16(X)) return SQ_ERR_ALIGN;
    if (M >= ((int64_t)1 << 34)) return SQ_ERR_UNSUPPORTED;
    return token_absmax(X, dt, M, C, ld, out, as_stream(stream));
}

sq_status sq_clipped_absmax(const float* vals, int64_t T, int64_t n_clip, float* absmax_out,
                            float* step_out, void* stream) {
    if (T < 0 || n_clip < 0) return SQ_ERR_SHAPE;
    if (T == 0) return SQ_ERR_SHAPE;  // no token to take a maximum of
    if (!vals || !absmax_out) return SQ_ERR_INVALID_ARG;
    if (T >= ((int64_t)1 << 32)) return SQ_ERR_UNSUPPORTED;
    return clipped_absmax(vals, T, n_clip, absmax_out, step_out, as_stream(stream));
}

sq_status sq_smooth_scales(const float* act_absmax, const float* w_absmax, int64_t C, float alpha,
                           float* s_out, float* s_inv_out, void* stream) {
    if (!(alpha >= 0.0f && alpha <= 1.0f)) return SQ_ERR_INVALID_ARG;
    if (C < 0) return SQ_ERR_SHAPE;
    if (C == 0) return SQ_OK;
    if (!act_absmax || !w_absmax || !s_out) return SQ_ERR_INVALID_ARG;
    return smooth_scales(act_absmax, w_absmax, C, alpha, s_out, s_inv_out, as_stream(stream));
}

sq_status sq_fold_ln_weight(const void* gamma, const void* beta, sq_dtype dt, const float* s, int64_t C,
                            void* gamma_out, void* beta_out, void* stream) {
    if (!is_act_dtype(dt)) return SQ_ERR_INVALID_ARG;
    if (C < 0) return SQ_ERR_SHAPE;
    if (C == 0) return SQ_OK;
    if (!gamma || !gamma_out || !s) return SQ_ERR_INVALID_ARG;
    if ((beta == nullptr) != (beta_out == nullptr)) return SQ_ERR_INVALID_ARG;
    return fold_ln_weight(gamma, beta, dt, s, C, gamma_out, beta_out, as_stream(stream));
}

sq_status sq_quant_weight(const void* W, sq_dtype dt, int64_t N, int64_t K, const float* s, sq_w_gran g,
                          int8_t* Wq, float* w_scale, void* workspace, size_t ws_bytes, void* stream) {
    if (!is_act_dtype(dt) || (g != SQ_W_PER_TENSOR && g != SQ_W_PER_CHANNEL)) return SQ_ERR_INVALID_ARG;
    if (N < 0 || K < 0) return SQ_ERR_SHAPE;
    if (N == 0 || K == 0) return SQ_OK;
    if (!W || !Wq || !w_scale) return SQ_ERR_INVALID_ARG;
    if (K % 8 != 0 || !aligned16(W) || (reinterpret_cast<uintptr_t>(Wq) & 7) != 0 || (s && !aligned16(s)))
        return SQ_ERR_ALIGN;
    // a weight row is quantised exactly like a token row whose column multiplier is s
    sq_status st = quant_rows_common(W, dt, N, K, s, nullptr, nullptr, 0.0f, false,
                                     g == SQ_W_PER_CHANNEL ? SQ_PER_TOKEN_DYNAMIC : SQ_PER_TENSOR_DYNAMIC, Wq, w_scale,
                                     nullptr, workspace, ws_bytes, sq_workspace_bytes(SQ_OP_QUANT_WEIGHT, N, N, K),
                                     as_stream(stream));
    if (st != SQ_OK) return st;
    // The decode-shaped GEMM fetches weights before it waits for the launch in front of it (weights
    // are normally static).  This offline call is the one library kernel that WRITES weights, so it
    // ends with a fully serialised empty launch: whatever follows on the stream finds Wq complete.
    return stream_full_dependency(as_stream(stream));
}

sq_status sq_quant_act(const void* X, sq_dtype dt, int64_t M, int64_t C, sq_act_gran g, const float* col_mul,
                       int8_t* Xq, float* x_scale, void* workspace, size_t ws_bytes, void* stream) {
    if (!is_act_dtype(dt) || g < SQ_PER_TENSOR_STATIC || g > SQ_PER_TOKEN_DYNAMIC) return SQ_ERR_INVALID_ARG;
    if (M < 0 || C < 0) return SQ_ERR_SHAPE;
    if (M == 0 || C == 0) return SQ_OK;
    if (!X || !Xq || !x_scale) return SQ_ERR_INVALID_ARG;
    if (C % 8 != 0 || !aligned16(X) || (reinterpret_cast<uintptr_t>(Xq) & 7) != 0 ||
        (col_mul && !aligned16(col_mul)))
        return SQ_ERR_ALIGN;
    return quant_rows_common(X, dt, M, C, col_mul, nullptr, nullptr, 0.0f, false, g, Xq, x_scale, nullptr,
                             workspace, ws_bytes, sq_workspace_bytes(SQ_OP_QUANT_ACT, M, 0, C),
                             as_stream(stream));
}

sq_status sq_quant_act_given_absmax(const void* X, sq_dtype dt, int64_t M, int64_t C, const float* row_absmax,
                                    int8_t* Xq, float* x_scale, void* workspace, size_t ws_bytes, void* stream) {
    if (!is_act_dtype(dt)) return SQ_ERR_INVALID_ARG;
    if (M < 0 || C < 0) return SQ_ERR_SHAPE;
    if (M == 0 || C == 0) return SQ_OK;
    if (!X || !Xq || !x_scale || !row_absmax) return SQ_ERR_INVALID_ARG;
    if (C % 8 != 0 || !aligned16(X) || (reinterpret_cast<uintptr_t>(Xq) & 7) != 0) return SQ_ERR_ALIGN;
    uint32_t* status = ws_ok(workspace, ws_bytes, sizeof(uint32_t)) ? static_cast<uint32_t*>(workspace) : nullptr;
    return row_quant(X, dt, M, C, nullptr, nullptr, nullptr, 0.0f, false, ROW_GIVEN_ROW_ABSMAX, Xq, x_scale,
                     const_cast<float*>(row_absmax), nullptr, 0, status, as_stream(stream));
}

sq_status sq_dequant_acc(const int32_t* acc, int64_t ld_acc, int64_t M, int64_t N, const float* x_scale,
                         int x_scale_is_per_token, const float* w_scale, int w_scale_is_per_channel, const void* bias,
                         sq_dtype bias_dt, sq_epilogue_act act, const float* requant_mul, int requant_is_per_channel,
                         const void* residual, int64_t ld_res, void* Y, sq_dtype out_dt, int64_t ldy, void* stream) {
    if (M < 0 || N < 0) return SQ_ERR_SHAPE;
    if (out_dt < SQ_F16 || out_dt > SQ_I8 || (act != SQ_EPI_NONE && act != SQ_EPI_RELU)) return SQ_ERR_INVALID_ARG;
    if (M == 0 || N == 0) return SQ_OK;
    if (!acc || !Y || !x_scale || !w_scale) return SQ_ERR_INVALID_ARG;
    if ((out_dt == SQ_I8) != (requant_mul != nullptr)) return SQ_ERR_INVALID_ARG;
    if (bias && !is_act_dtype(bias_dt)) return SQ_ERR_INVALID_ARG;
    if (residual && (out_dt == SQ_I8 || act != SQ_EPI_NONE)) return SQ_ERR_INVALID_ARG;
    if (ld_acc < N || ldy < N || (residual && ld_res < N)) return SQ_ERR_SHAPE;
    const int64_t out_vec = out_dt == SQ_I8 ? 8 : 8;  // 8 outputs per store: 8 or 16 bytes
    if (N % 8 != 0 || ld_acc % 4 != 0 || ldy % out_vec != 0 || !aligned16(acc) ||
        (reinterpret_cast<uintptr_t>(Y) & (out_dt == SQ_I8 ? 7 : 15)) != 0 ||
        (residual && (!aligned16(residual) || ld_res % 8 != 0)))
        return SQ_ERR_ALIGN;
    DequantArgs a{acc, ld_acc, M, N, x_scale, x_scale_is_per_token, w_scale, w_scale_is_per_channel, bias, bias_dt,
                  act == SQ_EPI_RELU, requant_mul, requant_is_per_channel, residual, ld_res, Y, out_dt, ldy};
    return dequant_acc(a, as_stream(stream));
}

sq_status sq_ln_quant(const void* X, sq_dtype dt, int64_t M, int64_t C, const void* gamma_hat,
                      const void* beta_hat, float eps, sq_act_gran g, int8_t* Xq, float* x_scale,
                      float* dbg_mean_rstd, void* workspace, size_t ws_bytes, void* stream) {
    if (!is_act_dtype(dt) || g < SQ_PER_TENSOR_STATIC || g > SQ_PER_TOKEN_DYNAMIC || !(eps >= 0.0f))
        return SQ_ERR_INVALID_ARG;
    if (M < 0 || C < 0) return SQ_ERR_SHAPE;
    if (M == 0 || C == 0) return SQ_OK;
    if (!X || !Xq || !x_scale || !gamma_hat) return SQ_ERR_INVALID_ARG;
    if (C % 8 != 0 || !aligned16(X) || (reinterpret_cast<uintptr_t>(Xq) & 7) != 0 || !aligned16(gamma_hat) ||
        (beta_hat && !aligned16(beta_hat)))
        return SQ_ERR_ALIGN;
    return quant_rows_common(X, dt, M, C, nullptr, gamma_hat, beta_hat, eps, true, g, Xq, x_scale,
                             dbg_mean_rstd, workspace, ws_bytes, sq_workspace_bytes(SQ_OP_LN_QUANT, M, 0, C),
                             as_stream(stream));
}

static sq_status w8a8_gemm_impl(const int8_t* Xq, const int8_t* Wq, int64_t M, int64_t N, int64_t K, const float* x_scale,
                                int x_scale_is_per_token, const float* w_scale, int w_scale_is_per_channel,
                                const void* bias, sq_dtype bias_dt, sq_epilogue_act act, const float* requant_mul,
                                int requant_is_per_channel, float* row_absmax_out, const void* residual,
                                int64_t ld_res, void* Y, sq_dtype out_dt, int64_t ldy, void* workspace,
                                size_t ws_bytes, void* stream) {

    if (M < 0 || N < 0 || K < 0) return SQ_ERR_SHAPE;
    if (out_dt < SQ_F16 || out_dt > SQ_I32 || (act != SQ_EPI_NONE && act != SQ_EPI_RELU)) return SQ_ERR_INVALID_ARG;
    if (M == 0 || N == 0) return SQ_OK;
    if (K == 0) return SQ_ERR_SHAPE;
    if (K > SQ_MAX_K) return SQ_ERR_UNSUPPORTED;
    if (ldy < N) return SQ_ERR_SHAPE;
    if (!Xq || !Wq || !Y) return SQ_ERR_INVALID_ARG;
    if (out_dt != SQ_I32 && (!x_scale || !w_scale)) return SQ_ERR_INVALID_ARG;
    if ((out_dt == SQ_I8) != (requant_mul != nullptr)) return SQ_ERR_INVALID_ARG;
    if (bias && !is_act_dtype(bias_dt)) return SQ_ERR_INVALID_ARG;
    if (K % 16 != 0 || !aligned16(Xq) || !aligned16(Wq)) return SQ_ERR_ALIGN;
    if (residual) {  // the residual stream has the output's 16-bit type and is read in 16-byte pieces
        if (!is_act_dtype(out_dt) || row_absmax_out) return SQ_ERR_INVALID_ARG;
        if (ld_res < N) return SQ_ERR_SHAPE;
        if (!aligned16(residual) || ld_res % 8 != 0 || N % 8 != 0) return SQ_ERR_ALIGN;
    }
    // decode-shaped calls need their scratch; a prefill GEMM only uses what it is given (see sq.h)
    if (!ws_ok(workspace, ws_bytes, M <= 32 ? sq_workspace_bytes(SQ_OP_GEMM, M, N, K) : kWsHeader)) return SQ_ERR_WORKSPACE;
    GemmArgs a{};
    a.ws_bytes = ws_bytes;
    a.A = Xq; a.B = Wq;
    a.batch = 1; a.heads = 1; a.M = M; a.N = N; a.K = K;
    a.strideA[0] = M * K; a.strideA[1] = M * K; a.strideA[2] = K;
    a.strideB[0] = N * K; a.strideB[1] = N * K; a.strideB[2] = K;
    a.b_is_kn = 0;
    a.x_scale = x_scale; a.x_per_row = x_scale_is_per_token;
    a.w_scale = w_scale; a.w_per_col = w_scale_is_per_channel;
    a.alpha = 1.0f;
    a.bias = bias; a.bias_dt = bias_dt;
    a.relu = act == SQ_EPI_RELU;
    a.requant_mul = requant_mul; a.requant_per_col = requant_is_per_channel;
    a.row_absmax_out = row_absmax_out;
    a.residual = residual; a.ld_res = ld_res;
    a.C = Y; a.out_dt = out_dt;
    a.strideC[0] = 0; a.strideC[1] = 0; a.strideC[2] = ldy;
    a.status = reinterpret_cast<uint32_t*>(workspace);
    return gemm_i8(a, as_stream(stream));
}

sq_status sq_w8a8_gemm(const int8_t* Xq, const int8_t* Wq, int64_t M, int64_t N, int64_t K,
                       const float* x_scale, int x_scale_is_per_token, const float* w_scale,
                       int w_scale_is_per_channel, const void* bias, sq_dtype bias_dt,
                       sq_epilogue_act act, const float* requant_mul, int requant_is_per_channel,
                       float* row_absmax_out, void* Y, sq_dtype out_dt, int64_t ldy,
                       void* workspace, size_t ws_bytes, void* stream) {
    return w8a8_gemm_impl(Xq, Wq, M, N, K, x_scale, x_scale_is_per_token, w_scale, w_scale_is_per_channel, bias, bias_dt,
                          act, requant_mul, requant_is_per_channel, row_absmax_out, nullptr, 0, Y, out_dt, ldy,
                          workspace, ws_bytes, stream);
}

sq_status sq_w8a8_gemm_residual(const int8_t* Xq, const int8_t* Wq, int64_t M, int64_t N, int64_t K,
                                const float* x_scale, int x_scale_is_per_token, const float* w_scale,
                                int w_scale_is_per_channel, const void* bias, sq_dtype bias_dt,
                                const void* residual, int64_t ld_res, void* Y, sq_dtype out_dt, int64_t ldy,
                                void* workspace, size_t ws_bytes, void* stream) {
    if (!residual) return SQ_ERR_INVALID_ARG;
    return w8a8_gemm_impl(Xq, Wq, M, N, K, x_scale, x_scale_is_per_token, w_scale, w_scale_is_per_channel, bias, bias_dt,
                          SQ_EPI_NONE, nullptr, 0, nullptr, residual, ld_res, Y, out_dt, ldy, workspace, ws_bytes, stream);
}

sq_status sq_w8a8_gemm_fused_quant(const void* X, sq_dtype x_dt, int64_t M, int64_t N, int64_t K,
                                   const void* gamma_hat, const void* beta_hat, float eps, sq_act_gran g,
                                   float* x_scale, int8_t* Xq_out, float* dbg_mean_rstd, const int8_t* Wq,
                                   const float* w_scale, int w_scale_is_per_channel, const void* bias,
                                   sq_dtype bias_dt, sq_epilogue_act act, const float* requant_mul,
                                   int requant_is_per_channel, const void* residual, int64_t ld_res, void* Y,
                                   sq_dtype out_dt, int64_t ldy, void* workspace, size_t ws_bytes, void* stream) {
    if (!is_act_dtype(x_dt) || (g != SQ_PER_TENSOR_STATIC && g != SQ_PER_TOKEN_DYNAMIC && g != SQ_PER_TENSOR_DYNAMIC))
        return SQ_ERR_INVALID_ARG;
    if (M < 0 || N < 0 || K < 0) return SQ_ERR_SHAPE;
    if (out_dt < SQ_F16 || out_dt > SQ_I8 || (act != SQ_EPI_NONE && act != SQ_EPI_RELU)) return SQ_ERR_INVALID_ARG;
    if (gamma_hat != nullptr && !(eps >= 0.0f)) return SQ_ERR_INVALID_ARG;
    if (gamma_hat == nullptr && (beta_hat != nullptr || dbg_mean_rstd != nullptr)) return SQ_ERR_INVALID_ARG;
    if (M == 0 || N == 0) return SQ_OK;
    if (K == 0) return SQ_ERR_SHAPE;
    // one step for the whole tensor would need a second meeting of the CTAs; beyond 32 tokens the
    // quantiser is a pass of its own: both go through sq_quant_act / sq_ln_quant + sq_w8a8_gemm
    if (M > 32 || g == SQ_PER_TENSOR_DYNAMIC || K > SQ_MAX_K) return SQ_ERR_UNSUPPORTED;
    if (ldy < N) return SQ_ERR_SHAPE;
    if (!X || !Wq || !Y || !w_scale) return SQ_ERR_INVALID_ARG;
    if (g == SQ_PER_TENSOR_STATIC && !x_scale) return SQ_ERR_INVALID_ARG;
    if ((out_dt == SQ_I8) != (requant_mul != nullptr)) return SQ_ERR_INVALID_ARG;
    if (bias && !is_act_dtype(bias_dt)) return SQ_ERR_INVALID_ARG;
    if (K % 16 != 0 || !aligned16(X) || !aligned16(Wq) || (Xq_out && !aligned16(Xq_out)) ||
        (gamma_hat && !aligned16(gamma_hat)) || (beta_hat && !aligned16(beta_hat)))
        return SQ_ERR_ALIGN;
    if (residual) {
        if (!is_act_dtype(out_dt)) return SQ_ERR_INVALID_ARG;
        if (ld_res < N) return SQ_ERR_SHAPE;
        if (!aligned16(residual) || ld_res % 8 != 0 || N % 8 != 0) return SQ_ERR_ALIGN;
    }
    if (!ws_ok(workspace, ws_bytes, sq_workspace_bytes(SQ_OP_GEMM_FUSED_QUANT, M, N, K))) return SQ_ERR_WORKSPACE;
    GemmArgs a{};
    a.ws_bytes = ws_bytes;
    a.A = nullptr; a.B = Wq;
    a.batch = 1; a.heads = 1; a.M = M; a.N = N; a.K = K;
    a.strideA[0] = M * K; a.strideA[1] = M * K; a.strideA[2] = K;
    a.strideB[0] = N * K; a.strideB[1] = N * K; a.strideB[2] = K;
    a.x_scale = x_scale; a.x_per_row = g == SQ_PER_TOKEN_DYNAMIC;
    a.w_scale = w_scale; a.w_per_col = w_scale_is_per_channel;
    a.alpha = 1.0f;
    a.bias = bias; a.bias_dt = bias_dt;
    a.relu = act == SQ_EPI_RELU;
    a.requant_mul = requant_mul; a.requant_per_col = requant_is_per_channel;
    a.residual = residual; a.ld_res = ld_res;
    a.C = Y; a.out_dt = out_dt;
    a.strideC[2] = ldy;
    a.status = reinterpret_cast<uint32_t*>(workspace);
    a.x_raw = X; a.x_raw_dt = x_dt;
    a.ln_gamma = gamma_hat; a.ln_beta = beta_hat; a.ln_eps = eps;
    a.x_static = g == SQ_PER_TENSOR_STATIC;
    a.xq_out = Xq_out;
    a.xs_out = g == SQ_PER_TOKEN_DYNAMIC ? x_scale : nullptr;
    a.ln_stats_out = dbg_mean_rstd;
    return decode_gemm(a, workspace, ws_bytes, as_stream(stream));
}

sq_status sq_w8a8_bmm(const int8_t* A, const int8_t* B, int64_t batch, int64_t heads, int64_t M, int64_t N,
                      int64_t K, const int64_t strideA[3], const int64_t strideB[3], int b_is_kn, int causal,
                      float alpha,
                      const float* requant_mul, void* C, sq_dtype out_dt, const int64_t strideC[3],
                      void* workspace, size_t ws_bytes, void* stream) {
    if (batch < 0 || heads < 0 || M < 0 || N < 0 || K < 0) return SQ_ERR_SHAPE;
    if (out_dt < SQ_F16 || out_dt > SQ_I32) return SQ_ERR_INVALID_ARG;
    if (batch == 0 || heads == 0 || M == 0 || N == 0) return SQ_OK;
    if (K == 0) return SQ_ERR_SHAPE;
    if (K > SQ_MAX_K) return SQ_ERR_UNSUPPORTED;
    if (!A || !B || !C || !strideA || !strideB || !strideC) return SQ_ERR_INVALID_ARG;
    if ((out_dt == SQ_I8) != (requant_mul != nullptr)) return SQ_ERR_INVALID_ARG;
    if (b_is_kn && N > 128) return SQ_ERR_UNSUPPORTED;
    if (K % 16 != 0 || (b_is_kn && N % 16 != 0) || !aligned16(A) || !aligned16(B)) return SQ_ERR_ALIGN;
    for (int i = 0; i < 3; ++i) {
        if (strideA[i] < 0 || strideB[i] < 0 || strideC[i] < 0) return SQ_ERR_SHAPE;
        if (strideA[i] % 16 != 0 || strideB[i] % 16 != 0) return SQ_ERR_ALIGN;
    }
    if (strideA[2] < K || strideB[2] < (b_is_kn ? N : K) || strideC[2] < N) return SQ_ERR_SHAPE;
    if (!ws_ok(workspace, ws_bytes, sq_workspace_bytes(SQ_OP_BMM, M, N, K))) return SQ_ERR_WORKSPACE;
    GemmArgs a{};
    a.ws_bytes = ws_bytes;
    a.A = A; a.B = B;
    a.batch = batch; a.heads = heads; a.M = M; a.N = N; a.K = K;
    for (int i = 0; i < 3; ++i) { a.strideA[i] = strideA[i]; a.strideB[i] = strideB[i]; a.strideC[i] = strideC[i]; }
    a.b_is_kn = b_is_kn ? 1 : 0;
    a.causal = causal ? 1 : 0;
    a.x_scale = nullptr; a.x_per_row = 0;
    a.w_scale = nullptr; a.w_per_col = 0;
    a.alpha = alpha;
    a.bias = nullptr; a.bias_dt = SQ_F16;
    a.relu = 0;
    a.requant_mul = requant_mul; a.requant_per_col = 0;
    a.row_absmax_out = nullptr;
    a.C = C; a.out_dt = out_dt;
    a.status = reinterpret_cast<uint32_t*>(workspace);
    return gemm_i8(a, as_stream(stream));
}

sq_status sq_w8a8_attention(const int8_t* qkv, int64_t B, int64_t H, int64_t S, int64_t d, float alpha_qk,
                            float alpha_pv, const float* requant_mul, int8_t* out, void* workspace,
                            size_t ws_bytes, void* stream) {
    if (B < 0 || H < 0 || S < 0 || d < 0) return SQ_ERR_SHAPE;
    if (!(alpha_qk > 0.0f)) return SQ_ERR_INVALID_ARG;  // the row maximum is taken on the integer accumulators
    if (B == 0 || H == 0 || S == 0) return SQ_OK;
    if (d != 128) return SQ_ERR_UNSUPPORTED;
    if (!qkv || !out || !requant_mul) return SQ_ERR_INVALID_ARG;
    if (S % 16 != 0 || !aligned16(qkv) || !aligned16(out)) return SQ_ERR_ALIGN;
    if (B * S >= ((int64_t)1 << 31) || B > 65535 || H > 65535) return SQ_ERR_UNSUPPORTED;
    if (!ws_ok(workspace, ws_bytes, sq_workspace_bytes(SQ_OP_BMM, S, S, d))) return SQ_ERR_WORKSPACE;
    return attention_i8(qkv, B, H, S, d, alpha_qk, alpha_pv, requant_mul, out,
                        reinterpret_cast<uint32_t*>(workspace), as_stream(stream));
}

sq_status sq_kv_cache_write(const int8_t* qkv, int64_t ld, int64_t B, int64_t T, int64_t H, int64_t d,
                            const int32_t* pos0, int8_t* k_cache, int8_t* v_cache, int64_t L_max, void* workspace,
                            size_t ws_bytes, void* stream) {
    if (B < 0 || T < 0 || H < 0 || d < 0 || L_max < 0) return SQ_ERR_SHAPE;
    if (B == 0 || T == 0 || H == 0) return SQ_OK;
    if (d != 128) return SQ_ERR_UNSUPPORTED;
    if (!qkv || !k_cache || !v_cache) return SQ_ERR_INVALID_ARG;
    if (T > L_max || ld < 3 * H * d) return SQ_ERR_SHAPE;
    if (L_max % 4 != 0 || ld % 16 != 0 || !aligned16(qkv) || !aligned16(k_cache) || !aligned16(v_cache)) return SQ_ERR_ALIGN;
    if (B > 65535 || H > 65535 || B * T >= ((int64_t)1 << 31) || L_max >= ((int64_t)1 << 31)) return SQ_ERR_UNSUPPORTED;
    if (!ws_ok(workspace, ws_bytes, kWsHeader)) return SQ_ERR_WORKSPACE;
    return kv_cache_write(qkv, ld, B, T, H, pos0, k_cache, v_cache, L_max, reinterpret_cast<uint32_t*>(workspace),
                          as_stream(stream));
}

sq_status sq_w8a8_decode_attention(const int8_t* q, int64_t ldq, int8_t* k_cache, int8_t* v_cache,
                                   const int8_t* k_new, const int8_t* v_new, int64_t ld_new,
                                   const int32_t* seq_lens, int64_t B, int64_t H, int64_t d, int64_t L_max,
                                   int64_t max_len, float alpha_qk, float alpha_pv, const float* requant_mul, void* out,
                                   sq_dtype out_dt, int64_t ldo, void* workspace, size_t ws_bytes, void* stream) {
    if (B < 0 || H < 0 || d < 0 || L_max < 0 || max_len < 0) return SQ_ERR_SHAPE;
    if (!(alpha_qk > 0.0f)) return SQ_ERR_INVALID_ARG;  // the maximum is taken on the integer accumulators
    if (out_dt != SQ_I8 && !is_act_dtype(out_dt)) return SQ_ERR_INVALID_ARG;
    if (B == 0 || H == 0) return SQ_OK;
    if (d != 128) return SQ_ERR_UNSUPPORTED;
    if (!q || !k_cache || !v_cache || !seq_lens || !out || (out_dt == SQ_I8 && !requant_mul)) return SQ_ERR_INVALID_ARG;
    if ((k_new == nullptr) != (v_new == nullptr)) return SQ_ERR_INVALID_ARG;
    if (max_len > L_max || max_len == 0 || ldq < H * d || ldo < H * d || (k_new && ld_new < H * d)) return SQ_ERR_SHAPE;
    if (L_max % 4 != 0 || ldq % 16 != 0 || !aligned16(q) || !aligned16(k_cache) || !aligned16(v_cache)) return SQ_ERR_ALIGN;
    if (k_new && (ld_new % 16 != 0 || !aligned16(k_new) || !aligned16(v_new))) return SQ_ERR_ALIGN;
    if (B > 65535 || H > 65535 || L_max >= ((int64_t)1 << 31)) return SQ_ERR_UNSUPPORTED;
    if (!ws_ok(workspace, ws_bytes, kWsHeader)) return SQ_ERR_WORKSPACE;
    return kv_decode_attention(q, ldq, k_cache, v_cache, k_new, v_new, ld_new, seq_lens, B, H, L_max, max_len, alpha_qk, alpha_pv, requant_mul,
                               out, out_dt, ldo, reinterpret_cast<uint32_t*>(workspace), as_stream(stream));
}

sq_status sq_softmax_quant_p(const void* scores, sq_dtype dt, int64_t n_mat, int64_t S, int8_t* Pq,
                             void* stream) {
    if (!is_act_dtype(dt)) return SQ_ERR_INVALID_ARG;
    if (n_mat < 0 || S < 0) return SQ_ERR_SHAPE;
    if (n_mat == 0 || S == 0) return SQ_OK;
    if (!scores || !Pq) return SQ_ERR_INVALID_ARG;
    if (S % 8 != 0 || !aligned16(scores) || (reinterpret_cast<uintptr_t>(Pq) & 7) != 0) return SQ_ERR_ALIGN;
    return softmax_quant_p(scores, dt, n_mat, S, Pq, as_stream(stream));
}

sq_status sq_selftest_bounded_wait(uint32_t* status_word, uint32_t budget_cycles, void* stream) {
    if (!status_word) return SQ_ERR_INVALID_ARG;
    if (budget_cycles > 100000000u) return SQ_ERR_INVALID_ARG;  // a self-test never waits longer than ~50 ms
    return bounded_wait_selftest(status_word, budget_cycles, as_stream(stream));
}

sq_status sq_selftest_row_wait(uint32_t* status_word, uint32_t budget_cycles, void* stream) {
    if (!status_word) return SQ_ERR_INVALID_ARG;
    if (budget_cycles > 100000000u) return SQ_ERR_INVALID_ARG;
    return row_wait_selftest(status_word, budget_cycles, as_stream(stream));
}

sq_status sq_residual_add(const void* a, const void* b, sq_dtype dt, int64_t n, void* out, void* stream) {
    if (!is_act_dtype(dt)) return SQ_ERR_INVALID_ARG;
    if (n < 0) return SQ_ERR_SHAPE;
    if (n == 0) return SQ_OK;
    if (!a || !b || !out) return SQ_ERR_INVALID_ARG;
    if (n % 8 != 0 || !aligned16(a) || !aligned16(b) || !aligned16(out)) return SQ_ERR_ALIGN;
    return residual_add(a, b, dt, n, out, as_stream(stream));
}

}  // extern "C"
