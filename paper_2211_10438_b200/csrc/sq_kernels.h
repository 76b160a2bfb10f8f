// Internal launch interface between the C-ABI layer (sq_api.cu) and the kernel files.
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

#include <algorithm>

#include "../../include/sq.h"

namespace sq {

// How a row kernel obtains its step size.
enum RowMode {
    ROW_DYNAMIC = 0,          // Delta_row = absmax(row)/127, written to scale[row]
    ROW_GIVEN_SCALE = 1,      // Delta = scale[0], an input (static)
    ROW_FROM_ABSMAX_WORD = 2, // Delta = step_size(*absmax_word); scale[0] receives it
    ROW_ABSMAX_ONLY = 3,      // no codes: atomically fold the row's absmax into *absmax_word
    ROW_GIVEN_ROW_ABSMAX = 4  // Delta_row = step_size(absmax_word[row]), an INPUT array [M] (a maximum agreed on
                              // across tensor-parallel ranks); written to scale[row]; larger values saturate
};

// Workspace layout (bytes).  Word 0 is the sticky device status.
constexpr size_t kWsStatusOff = 0;
constexpr size_t kWsAbsmaxOff = 16;   // per-tensor dynamic absmax word
constexpr size_t kWsHeader = 256;     // per-row LayerNorm statistics / decode-GEMM arrival counters start here
constexpr size_t kDecCounterBytes = 32768;  // decode-shaped GEMM: one arrival counter per 128-channel tile, then partial sums

sq_status calib_absmax(const void* X, sq_dtype dt, int64_t rows, int64_t cols, int64_t ld, float* a,
                       cudaStream_t st);
sq_status token_absmax(const void* X, sq_dtype dt, int64_t M, int64_t C, int64_t ld, float* out, cudaStream_t st);
sq_status clipped_absmax(const float* token_absmax, int64_t T, int64_t n_clip, float* absmax_out, float* step_out,
                         cudaStream_t st);
sq_status smooth_scales(const float* ax, const float* aw, int64_t C, float alpha, float* s, float* s_inv,
                        cudaStream_t st);
sq_status fold_ln_weight(const void* g, const void* b, sq_dtype dt, const float* s, int64_t C,
                         void* go, void* bo, cudaStream_t st);
sq_status row_quant(const void* X, sq_dtype dt, int64_t M, int64_t C, const float* col_mul,
                    const void* gamma, const void* beta, float eps, bool ln, int mode, int8_t* Xq,
                    float* scale, float* absmax_word, float* stats, int stats_are_input,
                    uint32_t* status /*nullable: device status word for an expired bulk-copy wait*/,
                    cudaStream_t st);
sq_status stream_full_dependency(cudaStream_t st);  // empty, fully serialised launch (see its definition)
sq_status row_wait_selftest(uint32_t* status, uint32_t budget, cudaStream_t st);
bool row_pipeline_supports(int64_t M, int64_t C, bool ln, bool has_col_mul);
sq_status row_pipeline(const void* X, sq_dtype dt, int64_t M, int64_t C, const float* col_mul, const void* gamma,
                       const void* beta, float eps, bool ln, int mode, int8_t* Xq, float* scale, float* absmax_word,
                       float* stats, int stats_are_input, uint32_t* status, cudaStream_t st);
sq_status softmax_quant_p(const void* scores, sq_dtype dt, int64_t n_mat, int64_t S, int8_t* Pq,
                          cudaStream_t st);
sq_status residual_add(const void* a, const void* b, sq_dtype dt, int64_t n, void* out,
                       cudaStream_t st);
// Eq. 2 (+ bias, ReLU, re-quantisation, residual add) on INT32 accumulators that already sit in memory
struct DequantArgs {
    const int32_t* acc; int64_t ld_acc; int64_t M, N;
    const float* x_scale; int x_per_row; const float* w_scale; int w_per_col;
    const void* bias; sq_dtype bias_dt; int relu;
    const float* requant_mul; int requant_per_col;
    const void* residual; int64_t ld_res;
    void* Y; sq_dtype out_dt; int64_t ldy;
};
sq_status dequant_acc(const DequantArgs& a, cudaStream_t st);

// Batched INT8 GEMM on the tensor cores (tcgen05, kind::i8) with the fused epilogue.
struct GemmArgs {
    const int8_t* A;      // [batch, heads, M, K]  K contiguous
    const int8_t* B;      // [batch, heads, N, K] (K contiguous) or [batch, heads, K, N] (b_is_kn)
    int64_t batch, heads, M, N, K;
    int64_t strideA[3];   // batch, head, row (elements)
    int64_t strideB[3];
    int b_is_kn;
    int causal;           // attention BMMs only: skip work above the diagonal
    const float* x_scale; int x_per_row;     // Delta_x[t] or Delta_x
    const float* w_scale; int w_per_col;     // Delta_w[o] or Delta_w; nullptr = 1
    float alpha;                             // used when x_scale == nullptr
    const void* bias; sq_dtype bias_dt;      // nullable
    int relu;
    const float* requant_mul; int requant_per_col;
    float* row_absmax_out;
    const void* residual; int64_t ld_res;    // nullable: [M, N] of the output dtype, added after the output rounding
    void* C; sq_dtype out_dt;
    int64_t strideC[3];   // batch, head, row (elements)
    uint32_t* status;     // device status word (= workspace base)
    size_t ws_bytes;      // size of the caller's workspace
    // Decode-shaped calls only (M <= 32): the activation quantiser runs in the GEMM's prologue.
    // A is then ignored; the codes go to xq_out (nullable: scratch in the workspace).
    const void* x_raw; sq_dtype x_raw_dt;     // [M, K] fp16 / bf16, contiguous
    const void* ln_gamma; const void* ln_beta; float ln_eps;  // nullable: folded LayerNorm in front of Eq. 1
    int x_static;                             // x_scale[0] is a given static step (else per-token dynamic)
    int8_t* xq_out; float* xs_out;            // nullable outputs: codes [M, K], step sizes [M] (dynamic mode)
    float* ln_stats_out;                      // nullable [2 M]
};
sq_status gemm_i8(const GemmArgs& a, cudaStream_t st);
size_t gemm_workspace_bytes(int64_t M, int64_t N, int64_t K);  // scratch for the K split of the last wave
sq_status attention_i8(const int8_t* qkv, int64_t B, int64_t H, int64_t S, int64_t d, float alpha_qk, float alpha_pv,
                       const float* requant_mul, int8_t* out, uint32_t* status, cudaStream_t st);
sq_status kv_cache_write(const int8_t* qkv, int64_t ld, int64_t B, int64_t T, int64_t H, const int32_t* pos0, int8_t* kc,
                         int8_t* vc, int64_t lmax, uint32_t* status, cudaStream_t st);
sq_status kv_decode_attention(const int8_t* q, int64_t ldq, int8_t* kc, int8_t* vc, const int8_t* k_new,
                              const int8_t* v_new, int64_t ld_new, const int32_t* lens,
                              int64_t B, int64_t H, int64_t lmax, int64_t max_len, float alpha_qk, float alpha_pv,
                              const float* requant_mul, void* out, sq_dtype out_dt, int64_t ldo, uint32_t* status,
                              cudaStream_t st);
sq_status bounded_wait_selftest(uint32_t* status, uint32_t budget, cudaStream_t st);

// Decode-shaped path (M <= 16): swapped operands, split-K with INT32 scratch in the workspace.
size_t decode_workspace_bytes(int64_t M, int64_t N);
size_t decode_fused_workspace_bytes(int64_t M, int64_t N, int64_t K);  // + codes and step sizes of the prologue quantiser
constexpr size_t kWsSyncOff = 32;     // decode-shaped GEMM with the quantiser in its prologue: two meeting counters
bool decode_supports(const GemmArgs& a);
sq_status decode_gemm(const GemmArgs& a, void* workspace, size_t ws_bytes, cudaStream_t st);

}  // namespace sq
