// Fused causal INT8 self-attention for one decoder block (Fig. 6: both attention BMMs in INT8,
// softmax in floating point), reading Q, K, V in place from the fused QKV code buffer:
//     S   = (Q K^T) * alpha_qk                               INT8 MMA, INT32 accumulate; fp32 scores
//     p   = softmax over keys j <= i of S                    fp32
//     P   = round(127 p)                                     INT8, fixed step 1/127
//     out = clamp(round( ((P V) * alpha_pv) * requant ))     INT8 MMA, INT32 accumulate
// The [S, S] score and probability matrices never leave the SM.  Because the INT32 accumulator
// of P.V cannot be rescaled exactly, the probabilities are quantised with the FINAL row
// maximum and sum: pass 1 walks the key tiles and keeps an online (max, sum) per query row,
// pass 2 walks them again, recomputes the scores, quantises P and multiplies by V.
//
// One CTA per (128-query tile, head, batch), two CTAs per SM.  Warps 0-3: softmax (thread = one
// query row = one TMEM lane, so row reductions are thread-local); warp 4: one lane issues the
// TMA loads and the tcgen05 MMAs.  TMEM: 128 columns of scores + 128 columns of output.
// The softmax is the instruction-bound part, so it is kept lean: the row maximum is taken on the
// INT32 accumulators (alpha_qk > 0 keeps the order), exp(s - max) is one FMA + one ex2.approx with
// alpha_qk * log2(e) folded into the multiplier, and 127 / rowsum is folded into the rounding FMA.
// Every wait is bounded and reports through the status word.
#include "sq_kernels.h"
#include "sq_tcgen05.cuh"

namespace sq {

namespace {

using namespace tc;

constexpr int ATT_THREADS = 160;
constexpr int TILE = 128;                    // queries per CTA, keys per step, head dimension
constexpr int TILE_BYTES = TILE * 128;       // one INT8 operand tile: 128 rows x 128 bytes
constexpr int ATT_SMEM = 1024 + 6 * TILE_BYTES + 16 * 8 + 64;  // Q, K x2, V x2, P + barriers
constexpr int ATT_TMEM_COLS = 256;
constexpr float kLog2e = 1.4426950408889634f;

struct AttParams {
    int S, H, hid;       // sequence length, heads, H * d
    float alpha_qk, alpha_pv;
    const float* requant_mul;
    int8_t* out;         // [B*S, hid]
    uint32_t* status;
};

__device__ __forceinline__ void softmax_bar() { asm volatile("bar.sync 1, 128;" ::: "memory"); }

// One softmax thread waits (bounded), the other 127 learn the outcome through shared memory.
__device__ __forceinline__ bool group_wait(uint64_t* bar, uint32_t parity, volatile uint32_t* abort_flag,
                                           volatile uint32_t* flag, uint32_t* status, uint32_t where) {
    if (threadIdx.x == 0) *flag = mbar_wait(bar, parity, abort_flag, status, where) ? 1u : 0u;
    softmax_bar();
    const bool ok = *flag != 0u;
    softmax_bar();  // everyone has read the flag before it can be rewritten
    return ok;
}

__device__ __forceinline__ float ex2_approx(float x) {
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}

__global__ void __launch_bounds__(ATT_THREADS, 2)
attention_kernel(const __grid_constant__ CUtensorMap tmap_qkv, const AttParams p) {
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
    uint8_t* s_q = smem;
    uint8_t* s_k = smem + TILE_BYTES;      // two stages
    uint8_t* s_v = smem + 3 * TILE_BYTES;  // two stages
    uint8_t* s_p = smem + 5 * TILE_BYTES;
    uint64_t* bars = reinterpret_cast<uint64_t*>(smem + 6 * TILE_BYTES);
    uint64_t* bar_q = bars;            // TMA: Q landed
    uint64_t* bar_k = bars + 1;        // [2] TMA: K stage landed
    uint64_t* bar_v = bars + 3;        // [2] TMA: V stage landed
    uint64_t* bar_s_full = bars + 5;   // MMA: scores complete in TMEM
    uint64_t* bar_s_free = bars + 6;   // softmax: scores read out of TMEM (128 arrivals)
    uint64_t* bar_p_full = bars + 7;   // softmax: P tile written to shared memory (128 arrivals)
    uint64_t* bar_pv_done = bars + 8;  // MMA: P.V of this step complete (P tile and V stage reusable)
    uint32_t* tmem_holder = reinterpret_cast<uint32_t*>(bars + 9);
    volatile uint32_t* abort_flag = tmem_holder + 1;
    volatile uint32_t* flag = tmem_holder + 2;

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int n_qt = (p.S + TILE - 1) / TILE;
    const int qt = n_qt - 1 - (int)blockIdx.x;  // heaviest query tiles are scheduled first
    const int h = blockIdx.y, b = blockIdx.z;
    const int n_kv = qt + 1;                    // causal: key tiles 0 .. qt
    const int row_base = b * p.S;               // first row of this batch in the QKV matrix
    const int xq = h * TILE, xk = p.hid + h * TILE, xv = 2 * p.hid + h * TILE;  // column offsets of Q, K, V

    if (threadIdx.x == 128) {
        asm volatile("prefetch.tensormap [%0];" ::"l"(&tmap_qkv) : "memory");
        mbar_init(bar_q, 1);
        for (int i = 0; i < 2; ++i) { mbar_init(bar_k + i, 1); mbar_init(bar_v + i, 1); }
        mbar_init(bar_s_full, 1);
        mbar_init(bar_s_free, 128);
        mbar_init(bar_p_full, 128);
        mbar_init(bar_pv_done, 1);
        *abort_flag = 0u;
        *flag = 0u;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    if (warp == 4) tmem_alloc<1>(tmem_holder, ATT_TMEM_COLS);
    tcgen05_fence_before();
    __syncthreads();
    tcgen05_fence_after();
    const uint32_t tmem_base = *tmem_holder;
    const uint32_t tmem_s = tmem_base, tmem_o = tmem_base + TILE;
    pdl_wait();
    pdl_launch_dependents();

    if (warp == 4) {
        // ===================== control lane: TMA loads and MMA issue =====================
        if (lane == 0) {
            const uint32_t idesc_s = make_idesc(TILE, TILE, 0);   // Q (K-major) x K^T (K-major)
            const uint32_t idesc_pv = make_idesc(TILE, TILE, 1);  // P (K-major) x V ([keys, d]: N contiguous)
            bool ok = true;
            mbar_expect_tx(bar_q, TILE_BYTES);
            tma_load_4d<1>(s_q, &tmap_qkv, bar_q, xq, row_base + qt * TILE, 0, 0);
            uint32_t kph[2] = {0, 0}, vph[2] = {0, 0};
            uint32_t s_free_ph = 0, p_full_ph = 0, pv_done_ph = 0;
            int it = 0;  // key-tile steps issued so far (over both passes)
            // first key tile of pass 1
            mbar_expect_tx(bar_k, TILE_BYTES);
            tma_load_4d<1>(s_k, &tmap_qkv, bar_k, xk, row_base, 0, 0);
            ok = mbar_wait(bar_q, 0, abort_flag, p.status, 20);
            for (int pass = 0; ok && pass < 2; ++pass) {
                for (int j = 0; ok && j < n_kv; ++j, ++it) {
                    const int st = it & 1;
                    // scores of this step: wait for K, and for the softmax warps to have drained the previous scores
                    if (!(ok = mbar_wait(bar_k + st, kph[st], abort_flag, p.status, 21))) break;
                    kph[st] ^= 1u;
                    if (it > 0) {
                        if (!(ok = mbar_wait(bar_s_free, s_free_ph, abort_flag, p.status, 22))) break;
                        s_free_ph ^= 1u;
                    }
                    tcgen05_fence_after();
                    {
                        const uint32_t qa = smem_u32(s_q), ka = smem_u32(s_k + st * TILE_BYTES);
#pragma unroll
                        for (int k = 0; k < TILE / UMMA_K; ++k)
                            umma_i8<1>(tmem_s, make_smem_desc(qa + k * UMMA_K, 16), make_smem_desc(ka + k * UMMA_K, 16),
                                       idesc_s, k > 0 ? 1u : 0u);
                        umma_commit<1>(bar_s_full);
                    }
                    // prefetch the next step's K (and V in pass 2) into the other stage; that stage's
                    // previous K was consumed by the previous step's score MMA (complete: its scores
                    // were drained), its previous V by the previous P.V (waited for below)
                    const int nj = j + 1 < n_kv ? j + 1 : (pass == 0 ? 0 : -1);
                    const int npass = j + 1 < n_kv ? pass : pass + 1;
                    if (pass == 1 && j > 0) {  // P.V of step j-1 must be complete before its V stage is reused
                        if (!(ok = mbar_wait(bar_pv_done, pv_done_ph, abort_flag, p.status, 23))) break;
                        pv_done_ph ^= 1u;
                    }
                    if (nj >= 0) {
                        const int nst = st ^ 1;
                        mbar_expect_tx(bar_k + nst, TILE_BYTES);
                        tma_load_4d<1>(s_k + nst * TILE_BYTES, &tmap_qkv, bar_k + nst, xk, row_base + nj * TILE, 0, 0);
                        if (npass == 1) {
                            mbar_expect_tx(bar_v + nst, TILE_BYTES);
                            tma_load_4d<1>(s_v + nst * TILE_BYTES, &tmap_qkv, bar_v + nst, xv, row_base + nj * TILE, 0, 0);
                        }
                    }
                    if (pass == 1) {
                        // out += P V once the softmax warps have written this step's P tile
                        if (!(ok = mbar_wait(bar_p_full, p_full_ph, abort_flag, p.status, 24))) break;
                        p_full_ph ^= 1u;
                        if (!(ok = mbar_wait(bar_v + st, vph[st], abort_flag, p.status, 25))) break;
                        vph[st] ^= 1u;
                        tcgen05_fence_after();
                        const uint32_t pa = smem_u32(s_p), va = smem_u32(s_v + st * TILE_BYTES);
#pragma unroll
                        for (int k = 0; k < TILE / UMMA_K; ++k)
                            umma_i8<1>(tmem_o, make_smem_desc(pa + k * UMMA_K, 16),
                                       make_smem_desc(va + k * (UMMA_K * 128), 16384u), idesc_pv, (j > 0 || k > 0) ? 1u : 0u);
                        umma_commit<1>(bar_pv_done);
                    }
                }
            }
        }
    } else {
        // ===================== softmax warps: thread = query row =====================
        const int r = warp * 32 + lane;             // row inside the tile == TMEM lane
        const int qi = qt * TILE + r;               // query position
        const uint32_t lane_addr = (uint32_t)(warp * 32) << 16;
        uint32_t s_full_ph = 0, pv_done_ph = 0;
        const float c1 = p.alpha_qk * kLog2e;  // exp(alpha * acc - max) = exp2(c1 * acc - m2)
        float m2 = -INFINITY, l = 0.0f;        // running maximum (in the exp2 domain) and sum
        bool ok = true;
        // ---- pass 1: online row maximum and sum over the visible keys ----
        for (int j = 0; ok && j < n_kv; ++j) {
            if (!(ok = group_wait(bar_s_full, s_full_ph, abort_flag, flag, p.status, 26))) break;
            s_full_ph ^= 1u;
            tcgen05_fence_after();
            const bool diag = j == qt;  // only the diagonal tile holds keys this query must not see
#pragma unroll 1
            for (int cc = 0; cc < TILE / 32; ++cc) {
                uint32_t acc[32];
                tmem_ld32(tmem_s + lane_addr + cc * 32, acc);  // warp-collective
                tmem_ld_wait();
                const int nvis = diag ? min(32, r - cc * 32 + 1) : 32;  // visible keys of this chunk
                if (nvis <= 0) continue;
                int cmax = INT_MIN;
#pragma unroll
                for (int c = 0; c < 32; ++c)
                    if (c < nvis) cmax = max(cmax, (int)acc[c]);
                const float cm2 = c1 * __int2float_rn(cmax);
                if (cm2 > m2) {  // rescale the running sum to the new maximum
                    l *= ex2_approx(m2 - cm2);
                    m2 = cm2;
                }
                float sum = 0.0f;
#pragma unroll
                for (int c = 0; c < 32; ++c)
                    if (c < nvis) sum += ex2_approx(fmaf(__int2float_rn((int)acc[c]), c1, -m2));
                l += sum;
            }
            tcgen05_fence_before();
            mbar_arrive(bar_s_free);
        }
        const float k127 = __fdiv_rn(127.0f, l);  // P = round(127 * e / l)
        // ---- pass 2: quantise P with the final (max, sum), one key tile at a time ----
        for (int j = 0; ok && j < n_kv; ++j) {
            if (!(ok = group_wait(bar_s_full, s_full_ph, abort_flag, flag, p.status, 27))) break;
            s_full_ph ^= 1u;
            if (j > 0) {  // the previous step's P.V has finished reading the P tile
                if (!(ok = group_wait(bar_pv_done, pv_done_ph, abort_flag, flag, p.status, 28))) break;
                pv_done_ph ^= 1u;
            }
            tcgen05_fence_after();
            const bool diag = j == qt;
            uint8_t* prow = s_p + r * 128;
#pragma unroll 1
            for (int cc = 0; cc < TILE / 32; ++cc) {
                uint32_t acc[32];
                tmem_ld32(tmem_s + lane_addr + cc * 32, acc);
                tmem_ld_wait();
                const int nvis = diag ? min(32, r - cc * 32 + 1) : 32;
                uint32_t w[8];
#pragma unroll
                for (int v = 0; v < 8; ++v) {
                    uint32_t q[4];
#pragma unroll
                    for (int e = 0; e < 4; ++e) {
                        const int c = 4 * v + e;
                        const float ex = ex2_approx(fmaf(__int2float_rn((int)acc[c]), c1, -m2));
                        q[e] = c < nvis ? quant_code<false>(ex, k127) : 0u;  // e <= l: the code cannot exceed 127
                    }
                    w[v] = pack4(q[0], q[1], q[2], q[3]);
                }
                // 32 keys = two 16-byte pieces of this row of the K-major, 128B-swizzled P tile
                const int piece = cc * 2;
                *reinterpret_cast<uint4*>(prow + (((piece) ^ (r & 7)) << 4)) = make_uint4(w[0], w[1], w[2], w[3]);
                *reinterpret_cast<uint4*>(prow + (((piece + 1) ^ (r & 7)) << 4)) = make_uint4(w[4], w[5], w[6], w[7]);
            }
            tcgen05_fence_before();
            mbar_arrive(bar_s_free);
            asm volatile("fence.proxy.async.shared::cta;" ::: "memory");  // P tile: generic writes -> MMA reads
            mbar_arrive(bar_p_full);
        }
        // ---- epilogue: out = round(((P V) * alpha_pv) * requant) ----
        if (ok && (ok = group_wait(bar_pv_done, pv_done_ph, abort_flag, flag, p.status, 29))) {
            tcgen05_fence_after();
            const float rq = __ldg(p.requant_mul);
            int8_t* orow = p.out + ((int64_t)(row_base + qi)) * p.hid + h * TILE;
#pragma unroll 1
            for (int cc = 0; cc < TILE / 32; ++cc) {
                uint32_t acc[32];
                tmem_ld32(tmem_o + lane_addr + cc * 32, acc);
                tmem_ld_wait();
                if (qi < p.S) {
                    uint32_t w[8];
#pragma unroll
                    for (int v = 0; v < 8; ++v) {
                        uint32_t q[4];
#pragma unroll
                        for (int e = 0; e < 4; ++e)
                            q[e] = quant_code(__fmul_rn(__int2float_rn((int32_t)acc[4 * v + e]), p.alpha_pv), rq);
                        w[v] = pack4(q[0], q[1], q[2], q[3]);
                    }
                    reinterpret_cast<uint4*>(orow + cc * 32)[0] = make_uint4(w[0], w[1], w[2], w[3]);
                    reinterpret_cast<uint4*>(orow + cc * 32)[1] = make_uint4(w[4], w[5], w[6], w[7]);
                }
            }
        }
    }

    __syncwarp();
    if (*abort_flag) __nanosleep(1000000);
    tcgen05_fence_before();
    __syncthreads();
    if (warp == 4) {
        tcgen05_fence_after();
        tmem_dealloc<1>(tmem_base, ATT_TMEM_COLS);
    }
}

}  // namespace

sq_status attention_i8(const int8_t* qkv, int64_t B, int64_t H, int64_t S, int64_t d, float alpha_qk, float alpha_pv,
                       const float* requant_mul, int8_t* out, uint32_t* status, cudaStream_t st) {
    if (d != TILE) return SQ_ERR_UNSUPPORTED;
    const int64_t hid = H * d;
    AttParams p;
    p.S = (int)S; p.H = (int)H; p.hid = (int)hid;
    p.alpha_qk = alpha_qk; p.alpha_pv = alpha_pv;
    p.requant_mul = requant_mul;
    p.out = out;
    p.status = status;
    // Q, K and V are column blocks of one [B*S, 3*H*d] matrix: a single 2-D map with 128 x 128 boxes serves all three
    CUtensorMap map;
    int s0, s1, s2;
    if (!make_map(&map, qkv, 1, 3 * hid, B * S, 1, 1, 3 * hid, 0, 0, TILE, TILE, &s0, &s1, &s2)) return SQ_ERR_CUDA;
    static bool attr_set[64] = {false};
    int dev = 0;
    SQ_CUDA_OK(cudaGetDevice(&dev));
    if (dev < 0 || dev >= 64 || !attr_set[dev]) {
        SQ_CUDA_OK(cudaFuncSetAttribute(attention_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, ATT_SMEM));
        if (dev >= 0 && dev < 64) attr_set[dev] = true;
    }
    const dim3 grid((unsigned)((S + TILE - 1) / TILE), (unsigned)H, (unsigned)B);
    return launch_pdl(attention_kernel, grid, dim3(ATT_THREADS), (size_t)ATT_SMEM, st, 1, map, p);
}

}  // namespace sq
