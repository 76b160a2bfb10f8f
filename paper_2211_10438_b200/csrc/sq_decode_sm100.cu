// Decode-shaped W8A8 linear (M <= 16 tokens): the weight matrix is streamed once from HBM and
// everything else is noise, so the kernel is laid out around that stream.
//
//   * operands are swapped: 128 OUTPUT CHANNELS of W (128 x 128 bytes per K slice) ride on the
//     MMA's M dimension and the <= 16 tokens on its N dimension (tcgen05.mma.kind::i8,
//     128 x 16 x 32), so no tile is padded from 16 to 128 rows and a stage is 18 KB;
//   * work units are (128-channel tile, K split): the split count is chosen so that the units
//     fill all SMs in whole waves whatever N is (INT32 partial sums add exactly in any order);
//   * a 10-stage TMA ring keeps ~180 KB of weights in flight per SM;
//   * with K splits, partial accumulators are added into an INT32 scratch in the workspace
//     with red.global.add; the unit that arrives last for a tile applies Eq. 2 (dequant, bias,
//     ReLU), writes Y and leaves scratch and counter zeroed for the next call.
// Every wait is bounded (status word, as in the prefill kernel).
#include "sq_kernels.h"
#include "sq_tcgen05.cuh"

namespace sq {

namespace {

using namespace tc;

constexpr int DEC_THREADS = 192;      // warp 0: TMA, warp 1: MMA + TMEM, warps 2-5: epilogue
constexpr int DEC_N = 16;             // tokens per MMA (N dimension)
constexpr int W_BYTES = BLOCK_M * BLOCK_K;  // 16 KB of weights per stage
constexpr int X_BYTES = DEC_N * BLOCK_K;    // 2 KB of activations per stage
constexpr int DEC_STAGE = W_BYTES + X_BYTES;
constexpr int DEC_STAGES = 10;
constexpr int DEC_TMEM_COLS = 32;     // two accumulator slots of 16 columns
constexpr int DEC_SMEM = 1024 + DEC_STAGES * DEC_STAGE + (2 * DEC_STAGES + 4) * 8 + 64;

struct DecParams {
    int M;
    int64_t N, K;
    int num_n, splits, kb_per_split, num_kb;
    int64_t total_units;
    const float* x_scale; int x_per_row;
    const float* w_scale; int w_per_col;
    const void* bias; int bias_is_bf16;
    int relu;
    const float* requant_mul; int requant_per_col;  // INT8 output: code = round(y * r)
    void* Y; int out_dt; int64_t ldy;
    int32_t* acc;        // [16][N] scratch (splits > 1), zero on entry and on exit
    uint32_t* counters;  // [num_n]   arrivals per tile, zero on entry and on exit
    uint32_t* status;
};

__device__ __forceinline__ void tmem_ld16(uint32_t taddr, uint32_t (&r)[16]) {
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x16.b32 "
        "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15}, [%16];"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
          "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15])
        : "r"(taddr)
        : "memory");
}
__device__ __forceinline__ void dec_epi_sync() { asm volatile("bar.sync 2, 128;" ::: "memory"); }

// Eq. 2 for one output channel (this thread) and all tokens, then the stores.
__device__ __forceinline__ void dec_finish(const DecParams& p, const int32_t (&acc)[16], int64_t col) {
    if (col >= p.N) return;
    if (p.out_dt == SQ_I32) {
        int32_t* y = static_cast<int32_t*>(p.Y);
#pragma unroll
        for (int t = 0; t < DEC_N; ++t)
            if (t < p.M) y[(int64_t)t * p.ldy + col] = acc[t];
        return;
    }
    const float ws = p.w_scale ? __ldg(p.w_scale + (p.w_per_col ? col : 0)) : 1.0f;
    float bs = 0.0f;
    if (p.bias)
        bs = p.bias_is_bf16 ? __bfloat162float(static_cast<const __nv_bfloat16*>(p.bias)[col])
                            : __half2float(static_cast<const __half*>(p.bias)[col]);
    const float rq = p.requant_mul ? __ldg(p.requant_mul + (p.requant_per_col ? col : 0)) : 1.0f;
#pragma unroll
    for (int t = 0; t < DEC_N; ++t) {
        if (t < p.M) {
            const float xs = __ldg(p.x_scale + (p.x_per_row ? t : 0));
            float v = __fmaf_rn(__int2float_rn(acc[t]), __fmul_rn(xs, ws), bs);
            if (p.relu) v = fmaxf(v, 0.0f);
            if (p.out_dt == SQ_I8)
                static_cast<int8_t*>(p.Y)[(int64_t)t * p.ldy + col] = (int8_t)(quant_code(v, rq) & 0xffu);
            else if (p.out_dt == SQ_BF16)
                static_cast<__nv_bfloat16*>(p.Y)[(int64_t)t * p.ldy + col] = __float2bfloat16_rn(v);
            else
                static_cast<__half*>(p.Y)[(int64_t)t * p.ldy + col] = __float2half_rn(v);
        }
    }
}

__global__ void __launch_bounds__(DEC_THREADS, 1)
decode_gemm_kernel(const __grid_constant__ CUtensorMap tmap_w, const __grid_constant__ CUtensorMap tmap_x,
                   const DecParams p) {
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
    uint64_t* full_bar = reinterpret_cast<uint64_t*>(smem + DEC_STAGES * DEC_STAGE);
    uint64_t* empty_bar = full_bar + DEC_STAGES;
    uint64_t* tmem_full = empty_bar + DEC_STAGES;
    uint64_t* tmem_empty = tmem_full + 2;
    uint32_t* tmem_holder = reinterpret_cast<uint32_t*>(tmem_empty + 2);
    volatile uint32_t* abort_flag = tmem_holder + 1;
    volatile uint32_t* epi_go = tmem_holder + 2;
    volatile uint32_t* epi_last = tmem_holder + 3;

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

    if (threadIdx.x == 0) {
        asm volatile("prefetch.tensormap [%0];" ::"l"(&tmap_w) : "memory");
        asm volatile("prefetch.tensormap [%0];" ::"l"(&tmap_x) : "memory");
        for (int s = 0; s < DEC_STAGES; ++s) {
            mbar_init(full_bar + s, 1);
            mbar_init(empty_bar + s, 1);
        }
        for (int s = 0; s < 2; ++s) {
            mbar_init(tmem_full + s, 1);
            mbar_init(tmem_empty + s, 128);
        }
        *abort_flag = 0u;
        *epi_go = 0u;
        *epi_last = 0u;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    if (warp == 1) tmem_alloc<1>(tmem_holder, DEC_TMEM_COLS);
    tcgen05_fence_before();
    __syncthreads();
    tcgen05_fence_after();
    const uint32_t tmem_base = *tmem_holder;
    pdl_launch_dependents();

    if (warp == 0) {
        // ============================ TMA producer ============================
        if (lane == 0) {
            int stage = 0;
            uint32_t phase = 0;
            bool ok = true;
            // The weights are static, the activations come from the kernel in front (the per-token
            // quantiser): fill the ring with weight slices first, wait for the predecessor, then
            // add the activation slices of those stages.
            int prefetched = 0;
            bool waited = false;
            for (int64_t u = blockIdx.x; ok && u < p.total_units; u += gridDim.x) {
                const int ni = (int)(u / p.splits), ks = (int)(u % p.splits);
                const int kb0 = ks * p.kb_per_split, kb1 = min(p.num_kb, kb0 + p.kb_per_split);
                int kb = kb0;
                if (!waited) {
                    const int n_pre = min(DEC_STAGES, kb1 - kb0);
                    for (int i = 0; i < n_pre; ++i) {
                        mbar_expect_tx(full_bar + i, DEC_STAGE);
                        tma_load_4d<1>(smem + i * DEC_STAGE, &tmap_w, full_bar + i, (kb0 + i) * BLOCK_K, ni * BLOCK_M, 0, 0);
                    }
                    pdl_wait();
                    for (int i = 0; i < n_pre; ++i)
                        tma_load_4d<1>(smem + i * DEC_STAGE + W_BYTES, &tmap_x, full_bar + i, (kb0 + i) * BLOCK_K, 0, 0, 0);
                    prefetched = n_pre;
                    waited = true;
                    kb = kb0 + n_pre;
                    stage = n_pre % DEC_STAGES;
                    phase = (n_pre == DEC_STAGES) ? 1u : 0u;
                }
                for (; kb < kb1; ++kb) {
                    if (!(ok = mbar_wait(empty_bar + stage, phase ^ 1u, abort_flag, p.status, 6))) break;
                    uint8_t* sw = smem + stage * DEC_STAGE;
                    mbar_expect_tx(full_bar + stage, DEC_STAGE);
                    tma_load_4d<1>(sw, &tmap_w, full_bar + stage, kb * BLOCK_K, ni * BLOCK_M, 0, 0);
                    tma_load_4d<1>(sw + W_BYTES, &tmap_x, full_bar + stage, kb * BLOCK_K, 0, 0, 0);
                    if (++stage == DEC_STAGES) { stage = 0; phase ^= 1u; }
                }
            }
            (void)prefetched;
        }
    } else if (warp == 1) {
        // ============================ MMA issuer ==============================
        if (lane == 0) {
            const uint32_t idesc = make_idesc(BLOCK_M, DEC_N, 0);
            int stage = 0;
            uint32_t phase = 0;
            int slot = 0;
            uint32_t slot_phase = 0;
            bool ok = true;
            for (int64_t u = blockIdx.x; ok && u < p.total_units; u += gridDim.x) {
                const int ks = (int)(u % p.splits);
                const int kb0 = ks * p.kb_per_split, kb1 = min(p.num_kb, kb0 + p.kb_per_split);
                if (!(ok = mbar_wait(tmem_empty + slot, slot_phase ^ 1u, abort_flag, p.status, 7))) break;
                tcgen05_fence_after();
                const uint32_t d_tmem = tmem_base + (uint32_t)(slot * DEC_N);
                for (int kb = kb0; kb < kb1; ++kb) {
                    if (!(ok = mbar_wait(full_bar + stage, phase, abort_flag, p.status, 8))) break;
                    tcgen05_fence_after();
                    const uint32_t sw = smem_u32(smem + stage * DEC_STAGE);
                    const uint32_t sx = sw + W_BYTES;
#pragma unroll
                    for (int k = 0; k < BLOCK_K / UMMA_K; ++k)
                        umma_i8<1>(d_tmem, make_smem_desc(sw + k * UMMA_K, 16), make_smem_desc(sx + k * UMMA_K, 16),
                                   idesc, (kb > kb0 || k > 0) ? 1u : 0u);
                    umma_commit<1>(empty_bar + stage);
                    if (++stage == DEC_STAGES) { stage = 0; phase ^= 1u; }
                }
                if (!ok) break;
                umma_commit<1>(tmem_full + slot);
                slot ^= 1;
                if (slot == 0) slot_phase ^= 1u;
            }
        }
    } else {
        // ============================ epilogue (warps 2-5) ====================
        pdl_wait();  // x_scale and the split-K scratch belong to earlier kernels until here
        const int quarter = warp & 3;           // TMEM lanes this warp may read
        const int ch = quarter * 32 + lane;     // output channel within the tile
        const int et = threadIdx.x - 64;        // 0..127
        int slot = 0;
        uint32_t slot_phase = 0;
        for (int64_t u = blockIdx.x; u < p.total_units; u += gridDim.x) {
            const int ni = (int)(u / p.splits);
            if (et == 0) *epi_go = mbar_wait(tmem_full + slot, slot_phase, abort_flag, p.status, 9) ? 1u : 0u;
            dec_epi_sync();
            if (*epi_go == 0u) break;
            tcgen05_fence_after();
            uint32_t r[16];
            tmem_ld16(tmem_base + ((uint32_t)(quarter * 32) << 16) + (uint32_t)(slot * DEC_N), r);
            tmem_ld_wait();
            tcgen05_fence_before();
            mbar_arrive(tmem_empty + slot);  // slot drained into registers
            slot ^= 1;
            if (slot == 0) slot_phase ^= 1u;

            const int64_t col = (int64_t)ni * BLOCK_M + ch;
            int32_t acc[16];
#pragma unroll
            for (int t = 0; t < 16; ++t) acc[t] = (int32_t)r[t];
            if (p.splits == 1) {
                dec_finish(p, acc, col);
            } else {
                // add this unit's partial sums; the last unit of the tile finishes it
                if (col < p.N) {
#pragma unroll
                    for (int t = 0; t < DEC_N; ++t)
                        if (t < p.M) atomicAdd(p.acc + (int64_t)t * p.N + col, acc[t]);
                }
                __threadfence();
                dec_epi_sync();
                if (et == 0) *epi_last = (atomicAdd(p.counters + ni, 1u) == (uint32_t)(p.splits - 1)) ? 1u : 0u;
                dec_epi_sync();
                if (*epi_last != 0u) {
                    __threadfence();
                    if (col < p.N) {
#pragma unroll
                        for (int t = 0; t < DEC_N; ++t) {
                            if (t < p.M) {
                                acc[t] = __ldcg(p.acc + (int64_t)t * p.N + col);
                                __stcg(p.acc + (int64_t)t * p.N + col, 0);  // hand the scratch back zeroed
                            }
                        }
                    }
                    dec_finish(p, acc, col);
                    if (et == 0) p.counters[ni] = 0u;
                }
            }
            dec_epi_sync();  // epi_go / epi_last are rewritten by thread 0 in the next round
        }
    }

    __syncwarp();
    if (*abort_flag) __nanosleep(1000000);
    tcgen05_fence_before();
    __syncthreads();
    if (warp == 1) {
        tcgen05_fence_after();
        tmem_dealloc<1>(tmem_base, DEC_TMEM_COLS);
    }
}

// K splits.  The kernel is HBM-bound, so a partly filled last wave only costs time when it has
// too few SMs to saturate HBM; splitting K adds INT32 atomics that grow with M.  Pick the split
// that minimises a small time model (microseconds): every wave streams its bytes at
// min(HBM rate, SMs in the wave x per-SM streaming rate), plus the atomics.
int choose_splits(int M, int64_t N, int num_n, int num_kb, int sms) {
    const double hbm = 6100.0e3, per_sm = 57.0e3;  // bytes per microsecond (measured on B200)
    const double atomic_us = 14.0e-6;              // per partial sum added through the scratch
    int best = 1;
    double best_t = 1e30;
    for (int s = 1; s <= 16 && num_kb / s >= 8; ++s) {
        const int per = (num_kb + s - 1) / s;
        if ((num_kb + per - 1) / per != s) continue;  // some split would get no work
        const double unit_bytes = (double)per * W_BYTES;
        int64_t units = (int64_t)num_n * s;
        double t = 0.0;
        while (units > 0) {
            const int64_t in_wave = std::min<int64_t>(units, sms);
            t += in_wave * unit_bytes / std::min(hbm, per_sm * (double)in_wave);
            units -= in_wave;
        }
        if (s > 1) t += atomic_us * (double)M * (double)N * s;
        if (t < best_t) { best_t = t; best = s; }
    }
    return best;
}

}  // namespace

size_t decode_workspace_bytes(int64_t N) {
    const int64_t num_n = (N + tc::BLOCK_M - 1) / tc::BLOCK_M;
    return kWsHeader + (size_t)DEC_N * N * sizeof(int32_t) + (size_t)num_n * sizeof(uint32_t);
}

bool decode_supports(const GemmArgs& a) {
    return a.M <= DEC_N && a.batch == 1 && a.heads == 1 && !a.b_is_kn &&
           a.row_absmax_out == nullptr && a.strideA[2] == a.K && a.strideB[2] == a.K;
}

sq_status decode_gemm(const GemmArgs& a, void* workspace, size_t ws_bytes, cudaStream_t st) {
    DecParams p;
    p.M = (int)a.M; p.N = a.N; p.K = a.K;
    p.num_n = (int)((a.N + BLOCK_M - 1) / BLOCK_M);
    p.num_kb = (int)((a.K + BLOCK_K - 1) / BLOCK_K);
    p.splits = choose_splits(p.M, p.N, p.num_n, p.num_kb, sm_count());
    if (ws_bytes < decode_workspace_bytes(a.N)) p.splits = 1;  // no scratch: every tile in one unit
    p.kb_per_split = (p.num_kb + p.splits - 1) / p.splits;
    p.total_units = (int64_t)p.num_n * p.splits;
    p.x_scale = a.x_scale; p.x_per_row = a.x_per_row;
    p.w_scale = a.w_scale; p.w_per_col = a.w_per_col;
    p.bias = a.bias; p.bias_is_bf16 = a.bias_dt == SQ_BF16;
    p.relu = a.relu;
    p.requant_mul = a.requant_mul; p.requant_per_col = a.requant_per_col;
    p.Y = a.C; p.out_dt = (int)a.out_dt; p.ldy = a.strideC[2];
    p.acc = reinterpret_cast<int32_t*>(static_cast<char*>(workspace) + kWsHeader);
    p.counters = reinterpret_cast<uint32_t*>(p.acc + (size_t)DEC_N * a.N);
    p.status = a.status;
    CUtensorMap mw, mx;
    int s0, s1, s2;
    if (!make_map(&mw, a.B, 1, a.K, a.N, 1, 1, a.K, 0, 0, BLOCK_K, BLOCK_M, &s0, &s1, &s2)) return SQ_ERR_CUDA;
    if (!make_map(&mx, a.A, 1, a.K, a.M, 1, 1, a.K, 0, 0, BLOCK_K, DEC_N, &s0, &s1, &s2)) return SQ_ERR_CUDA;
    static bool attr_set[64] = {false};
    int dev = 0;
    SQ_CUDA_OK(cudaGetDevice(&dev));
    if (dev < 0 || dev >= 64 || !attr_set[dev]) {
        SQ_CUDA_OK(cudaFuncSetAttribute(decode_gemm_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, DEC_SMEM));
        if (dev >= 0 && dev < 64) attr_set[dev] = true;
    }
    const int grid = (int)std::min<int64_t>(p.total_units, sm_count());
    return launch_pdl(decode_gemm_kernel, dim3((unsigned)grid), dim3(DEC_THREADS), (size_t)DEC_SMEM, st, 1, mw, mx, p);
}

}  // namespace sq
