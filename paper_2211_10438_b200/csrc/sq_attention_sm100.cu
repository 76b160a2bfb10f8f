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
// One CTA per (128-query tile, head, batch), two CTAs per SM.  Warps 0-7: softmax, two threads per
// query row (warps 0-3 own key half 0 of every tile, warps 4-7 half 1; the row is the thread's TMEM
// lane, so row reductions are thread-local per half and merged once after pass 1); warp 8 walks the
// steps converged and one elected lane of it issues the TMA loads and the tcgen05 MMAs.  TMEM: 2 x 64 columns of scores + 128 of output.
// The score MMA is issued per key half with separate full / free barriers, so the tensor core
// refills one half while the other is being read, and the next step's first half is issued as
// soon as the current one is drained.  The softmax is kept lean: the row maximum is taken on the
// INT32 accumulators (alpha_qk > 0 keeps the order), INT32 -> fp32 goes through an exact
// magic-number add instead of the conversion unit, exp(s - max) is one FMA + one ex2.approx with
// alpha_qk * log2(e) folded into the multiplier, 127 / rowsum is folded into the rounding FMA, and
// keys above the diagonal are masked by selecting -inf as the exponent argument (no branches).
// Measured: time = 5.2 us per CTA + 2.05 us per (key tile, pass) over 296 resident CTAs (the CTAs
// with the most key tiles are dispatched first over the whole grid, so the tail is made of short
// ones: batch 4 x 512 went from 55.5 to 50.1 us); backing
// the waiting lanes off with nanosleep, or prefetching TMEM chunks into a second register buffer,
// was slower, and a persistent variant (two CTAs per SM walking a list of tiles, one TMEM
// allocation and barrier set-up per CTA) took the same time: the per-tile cost is the serial
// load -> first MMA -> ... -> epilogue latency of a tile, not the launch of its CTA.
// Every wait is bounded and reports through the status word.
#include "sq_kernels.h"
#include "sq_tcgen05.cuh"

namespace sq {

namespace {

using namespace tc;

constexpr int ATT_THREADS = 288;             // 8 softmax warps + the control warp
constexpr int CTRL_WARP = 8;
constexpr int TILE = 128;                    // queries per CTA, keys per step, head dimension
constexpr int HALF = 64;                     // keys per score MMA (half a key tile)
constexpr int TILE_BYTES = TILE * 128;       // one INT8 operand tile: 128 rows x 128 bytes
constexpr int ATT_SMEM = 1024 + 6 * TILE_BYTES + 16 * 8 + 64 + 2 * TILE * 8;  // Q, K x2, V x2, P, barriers, row statistics
constexpr int ATT_TMEM_COLS = 256;
constexpr float kLog2e = 1.4426950408889634f;

struct AttParams {
    int S, H, hid;       // sequence length, heads, H * d
    float alpha_qk, alpha_pv;
    const float* requant_mul;
    int8_t* out;         // [B*S, hid]
    uint32_t* status;
};

// Lane 0 of a softmax warp waits (bounded); the other lanes learn the outcome by shuffle.
__device__ __forceinline__ bool warp_wait(uint64_t* bar, uint32_t parity, volatile uint32_t* abort_flag,
                                          uint32_t* status, uint32_t where) {
    uint32_t ok = 1u;
    if ((threadIdx.x & 31) == 0) ok = mbar_wait(bar, parity, abort_flag, status, where) ? 1u : 0u;
    return __shfl_sync(0xffffffffu, ok, 0) != 0u;
}

__device__ __forceinline__ float ex2_approx(float x) {
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}

// INT32 -> fp32 for |a| < 2^22 without the conversion unit (which shares its pipe with ex2): adding
// the integer to the bit pattern of 1.5 * 2^23 gives the float 1.5 * 2^23 + a exactly (one unit in
// the last place is 1 there), and the subtraction is exact.  Scores obey |q . k| <= 127^2 * 128 < 2^21.
// (Done on pairs in score_pair_x below.)

// Pass 1 on one chunk of 32 scores: running maximum (exp2 domain) and sum.  NVIS = 32 for chunks
// that lie entirely below the diagonal (no per-element visibility test), otherwise the count of
// visible keys is passed in.  Four partial sums keep the adds independent of one another.
// Invisible keys of a diagonal chunk are handled without branches: their exponent argument is
// replaced by -inf (ex2 gives 0, the P code rounds to 0) and their score by INT_MIN in the maximum.
// The softmax warps are bound by instruction issue, so the per-score work is done on PAIRS with the
// two-wide fp32 instructions (each half rounds exactly like the scalar instruction; one issue slot for
// two values) and the integer maximum with the three-input form: bit for bit the scalar sequence --
// magic-number conversion, x = fma(s, c1, -m2), ex2, four partial sums over the scores c = 0..3 mod 4.
__device__ __forceinline__ float2 score_pair_x(uint32_t a0, uint32_t a1, float2 c1v, float2 neg_m2) {
    const float2 s = __fadd2_rn(make_float2(__int_as_float((int)a0 + 0x4B400000), __int_as_float((int)a1 + 0x4B400000)),
                                make_float2(-12582912.0f, -12582912.0f));
    return __ffma2_rn(s, c1v, neg_m2);
}

template <bool FULL>
__device__ __forceinline__ void pass1_chunk(const uint32_t (&acc)[32], int nvis, float c1, float& m2, float& l) {
    int cmax = INT_MIN;
    if (FULL) {
        cmax = max((int)acc[0], (int)acc[1]);
#pragma unroll
        for (int c = 2; c < 32; c += 2) cmax = __vimax3_s32(cmax, (int)acc[c], (int)acc[c + 1]);
    } else {
#pragma unroll
        for (int c = 0; c < 32; ++c) cmax = max(cmax, c < nvis ? (int)acc[c] : INT_MIN);
    }
    const float cm2 = c1 * __int2float_rn(cmax);
    if (cm2 > m2) {  // rescale the running sum to the new maximum
        l *= ex2_approx(m2 - cm2);
        m2 = cm2;
    }
    const float2 c1v = make_float2(c1, c1), neg_m2 = make_float2(-m2, -m2);
    float2 s[2] = {make_float2(0.0f, 0.0f), make_float2(0.0f, 0.0f)};  // four partial sums keep the adds independent
#pragma unroll
    for (int c = 0; c < 32; c += 2) {
        const float2 x = score_pair_x(acc[c], acc[c + 1], c1v, neg_m2);
        const float2 e = make_float2(ex2_approx((FULL || c < nvis) ? x.x : -INFINITY),
                                     ex2_approx((FULL || c + 1 < nvis) ? x.y : -INFINITY));
        s[(c >> 1) & 1] = __fadd2_rn(s[(c >> 1) & 1], e);
    }
    l += (s[0].x + s[0].y) + (s[1].x + s[1].y);
}

// Pass 2 on one chunk: P = round(127 * e / l) as INT8 codes, 32 keys = eight packed words (two 16-byte
// pieces of this row of the K-major, 128B-swizzled P tile, stored by the caller once the tile is free).
template <bool FULL>
__device__ __forceinline__ void pass2_chunk(const uint32_t (&acc)[32], int nvis, float c1, float m2, float k127,
                                            uint32_t (&w)[8]) {
    const float2 c1v = make_float2(c1, c1), neg_m2 = make_float2(-m2, -m2);
    const float2 k2 = make_float2(k127, k127), magic2 = make_float2(kRoundMagic, kRoundMagic);
#pragma unroll
    for (int v = 0; v < 8; ++v) {
        uint32_t q[4];
#pragma unroll
        for (int h2 = 0; h2 < 2; ++h2) {
            const int c = 4 * v + 2 * h2;
            const float2 x = score_pair_x(acc[c], acc[c + 1], c1v, neg_m2);
            const float2 e = make_float2(ex2_approx((FULL || c < nvis) ? x.x : -INFINITY),
                                         ex2_approx((FULL || c + 1 < nvis) ? x.y : -INFINITY));
            const float2 rr = __ffma2_rn(e, k2, magic2);  // e <= l: the code cannot exceed 127, no clamp
            q[2 * h2] = __float_as_uint(rr.x);
            q[2 * h2 + 1] = __float_as_uint(rr.y);
        }
        w[v] = pack4(q[0], q[1], q[2], q[3]);
    }
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
    uint64_t* bar_s_full = bars + 5;   // [2] MMA: scores of key half 0 / 1 complete in TMEM
    uint64_t* bar_s_free = bars + 7;   // [2] softmax: that half read out of TMEM (128 arrivals)
    uint64_t* bar_p_full = bars + 9;   // softmax: P tile written to shared memory (128 arrivals)
    uint64_t* bar_pv_done = bars + 10; // MMA: P.V of this step complete (P tile and V stage reusable)
    uint32_t* tmem_holder = reinterpret_cast<uint32_t*>(bars + 11);
    volatile uint32_t* abort_flag = tmem_holder + 1;
    float2* s_stat = reinterpret_cast<float2*>(smem + 6 * TILE_BYTES + 16 * 8 + 64);  // [2][128] (max, sum) per row and half

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int n_qt = (p.S + TILE - 1) / TILE;
    // CTAs are dispatched in the order of their linear index: the heaviest query tiles (most key
    // tiles below the diagonal) of ALL heads and sequences go first, the lightest last, so the
    // tail of the grid is made of short CTAs
    const uint32_t lin = blockIdx.x + gridDim.x * (blockIdx.y + gridDim.y * blockIdx.z);
    const uint32_t per_qt = gridDim.y * gridDim.z;
    const int qt = n_qt - 1 - (int)(lin / per_qt);
    const int h = (int)((lin % per_qt) % gridDim.y), b = (int)((lin % per_qt) / gridDim.y);
    const int n_kv = qt + 1;                    // causal: key tiles 0 .. qt
    const int row_base = b * p.S;               // first row of this batch in the QKV matrix
    const int xq = h * TILE, xk = p.hid + h * TILE, xv = 2 * p.hid + h * TILE;  // column offsets of Q, K, V

    if (threadIdx.x == CTRL_WARP * 32) {
        asm volatile("prefetch.tensormap [%0];" ::"l"(&tmap_qkv) : "memory");
        mbar_init(bar_q, 1);
        for (int i = 0; i < 2; ++i) { mbar_init(bar_k + i, 1); mbar_init(bar_v + i, 1); }
        for (int i = 0; i < 2; ++i) { mbar_init(bar_s_full + i, 1); mbar_init(bar_s_free + i, 128); }
        mbar_init(bar_p_full, 256);
        mbar_init(bar_pv_done, 1);
        *abort_flag = 0u;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    if (warp == CTRL_WARP) tmem_alloc<1>(tmem_holder, ATT_TMEM_COLS);
    tcgen05_fence_before();
    __syncthreads();
    tcgen05_fence_after();
    const uint32_t tmem_base = *tmem_holder;
    const uint32_t tmem_s = tmem_base, tmem_o = tmem_base + TILE;
    pdl_wait();
    pdl_launch_dependents();

    if (warp == CTRL_WARP) {
        // ===================== control warp: TMA loads and MMA issue =====================
        // The whole warp walks the steps and waits on the barriers, converged; one elected lane issues the
        // loads, the MMAs and the commits (their operands are then warp-uniform values to the compiler).
        {
            // The score MMA is issued per HALF of the key tile (64 keys, 64 TMEM columns), each half
            // with its own full / free barriers: while the softmax warps work on one half, the
            // tensor core already fills the other, and the next step's first half is issued as
            // soon as the current first half has been read out.  Steps t = 0 .. 2*n_kv - 1 run
            // through pass 1 (t < n_kv) and pass 2; key tile of step t is t % n_kv.
            const uint32_t idesc_s = make_idesc(TILE, HALF, 0);   // Q (K-major) x K^T (K-major), 64 keys
            const uint32_t idesc_pv = make_idesc(TILE, TILE, 1);  // P (K-major) x V ([keys, d]: N contiguous)
            const uint32_t q_lo = smem_desc_lo(smem_u32(s_q), 16), k_lo0 = smem_desc_lo(smem_u32(s_k), 16);
            const uint32_t p_lo = smem_desc_lo(smem_u32(s_p), 16), v_lo0 = smem_desc_lo(smem_u32(s_v), 16384u);
            const uint32_t bars0 = smem_u32(bars);
            auto bar_addr = [&](uint64_t* b) { return bars0 + (uint32_t)(b - bars) * 8u; };
            const int T = 2 * n_kv;
            bool ok = true;
            uint32_t kph[2] = {0, 0}, vph[2] = {0, 0}, s_free_ph[2] = {0, 0};
            uint32_t p_full_ph = 0, pv_done_ph = 0;
            auto wait = [&](uint64_t* b, uint32_t parity, uint32_t where) {
                return mbar_wait_warp(b, bar_addr(b), parity, abort_flag, p.status, where);
            };
            auto load_kv = [&](int t) {  // operands of step t into stage t & 1
                if (!elect_one()) return;
                const int st = t & 1, j = t % n_kv;
                mbar_expect_tx(bar_k + st, TILE_BYTES);
                tma_load_4d<1>(s_k + st * TILE_BYTES, &tmap_qkv, bar_k + st, xk, row_base + j * TILE, 0, 0);
                if (t >= n_kv) {
                    mbar_expect_tx(bar_v + st, TILE_BYTES);
                    tma_load_4d<1>(s_v + st * TILE_BYTES, &tmap_qkv, bar_v + st, xv, row_base + j * TILE, 0, 0);
                }
            };
            auto issue_qk = [&](int t, int hh) {  // scores of key half hh of step t
                if (!elect_one()) return;
                const uint32_t k_lo = k_lo0 + (uint32_t)(((t & 1) * TILE_BYTES + hh * (HALF * 128)) >> 4);
                umma_i8_lo<1>(tmem_s + hh * HALF, q_lo, k_lo, idesc_s, 0u);
#pragma unroll
                for (int k = 1; k < TILE / UMMA_K; ++k)
                    umma_i8_lo<1>(tmem_s + hh * HALF, q_lo + k * (UMMA_K >> 4), k_lo + k * (UMMA_K >> 4), idesc_s, 1u);
                umma_commit_u32<1>(bar_addr(bar_s_full + hh));
            };
            if (elect_one()) {
                mbar_expect_tx(bar_q, TILE_BYTES);
                tma_load_4d<1>(s_q, &tmap_qkv, bar_q, xq, row_base + qt * TILE, 0, 0);
            }
            load_kv(0);
            load_kv(1);  // T >= 2 always
            ok = wait(bar_q, 0, 20);
            if (ok) ok = wait(bar_k, kph[0], 21);
            kph[0] ^= 1u;
            if (ok) {
                tcgen05_fence_after();
                issue_qk(0, 0);
                issue_qk(0, 1);
            }
            for (int t = 0; ok && t < T; ++t) {
                const int st = t & 1;
                const bool more = t + 1 < T;
                if (more) {  // (a) first half of the next step, once this step's first half is drained
                    if (!(ok = wait(bar_k + (st ^ 1), kph[st ^ 1], 21))) break;
                    kph[st ^ 1] ^= 1u;
                    if (!(ok = wait(bar_s_free, s_free_ph[0], 22))) break;
                    s_free_ph[0] ^= 1u;
                    tcgen05_fence_after();
                    issue_qk(t + 1, 0);
                }
                if (t >= n_kv) {  // (b) out += P V once the softmax warps have written this step's P tile
                    if (!(ok = wait(bar_p_full, p_full_ph, 24))) break;
                    p_full_ph ^= 1u;
                    if (!(ok = wait(bar_v + st, vph[st], 25))) break;
                    vph[st] ^= 1u;
                    tcgen05_fence_after();
                    if (elect_one()) {
                        const uint32_t v_lo = v_lo0 + (uint32_t)((st * TILE_BYTES) >> 4);
#pragma unroll
                        for (int k = 0; k < TILE / UMMA_K; ++k)
                            umma_i8_lo<1>(tmem_o, p_lo + k * (UMMA_K >> 4), v_lo + k * ((UMMA_K * 128) >> 4), idesc_pv,
                                          (t > n_kv || k > 0) ? 1u : 0u);
                        umma_commit_u32<1>(bar_addr(bar_pv_done));
                    }
                }
                if (more) {  // (c) second half of the next step
                    if (!(ok = wait(bar_s_free + 1, s_free_ph[1], 23))) break;
                    s_free_ph[1] ^= 1u;
                    tcgen05_fence_after();
                    issue_qk(t + 1, 1);
                }
                if (t + 2 < T) {  // (d) this step's stages are free once its MMAs are complete: refill them
                    if (t >= n_kv) {  // K(t): both halves drained above; V(t): wait for P.V
                        if (!(ok = wait(bar_pv_done, pv_done_ph, 27))) break;
                        pv_done_ph ^= 1u;
                    }
                    load_kv(t + 2);
                }
            }
        }
    } else {
        // ===================== softmax warps =====================
        // Two threads per query row: warps 0-3 own key half 0 of every tile (TMEM columns 0..63),
        // warps 4-7 half 1; both have the row as their TMEM lane, so the two halves of a step are
        // processed at the same time.  Row statistics are thread-local per half and merged once.
        const int g = warp >> 2;                     // key half of this thread
        const int r = (warp & 3) * 32 + lane;        // row inside the tile == TMEM lane
        const int qi = qt * TILE + r;                // query position
        const uint32_t lane_addr = (uint32_t)((warp & 3) * 32) << 16;
        uint32_t s_full_ph = 0, pv_done_ph = 0;
        const float rq = __ldg(p.requant_mul);  // requested now: read in the epilogue it would be a dependent trip to L2
        const float c1 = p.alpha_qk * kLog2e;  // exp(alpha * acc - max) = exp2(c1 * acc - m2)
        float m2 = -INFINITY, l = 0.0f;        // running maximum (in the exp2 domain) and sum of this half
        bool ok = true;
        // ---- pass 1: online row maximum and sum over the visible keys of this half ----
        for (int j = 0; ok && j < n_kv; ++j) {
            const bool diag = j == qt;  // only the diagonal tile holds keys this query must not see
            if (!(ok = warp_wait(bar_s_full + g, s_full_ph, abort_flag, p.status, 26))) break;
            s_full_ph ^= 1u;
            tcgen05_fence_after();
#pragma unroll 1
            for (int cc = 2 * g; cc < 2 * g + 2; ++cc) {
                uint32_t acc[32];
                tmem_ld32(tmem_s + lane_addr + cc * 32, acc);  // warp-collective
                tmem_ld_wait();
                if (!diag) {
                    pass1_chunk<true>(acc, 32, c1, m2, l);
                } else {
                    const int nvis = min(32, r - cc * 32 + 1);  // visible keys of this chunk
                    if (nvis > 0) pass1_chunk<false>(acc, nvis, c1, m2, l);  // a row with none keeps its (max, sum)
                }
            }
            tcgen05_fence_before();
            mbar_arrive(bar_s_free + g);
        }
        // merge the two halves' (max, sum): both threads of a row evaluate the same expression
        s_stat[g * TILE + r] = make_float2(m2, l);
        asm volatile("bar.sync 1, 256;" ::: "memory");
        {
            const float2 a0 = s_stat[r], a1 = s_stat[TILE + r];
            m2 = fmaxf(a0.x, a1.x);  // half 0 always sees at least key 0, so the maximum is finite
            l = a0.y * ex2_approx(a0.x - m2) + a1.y * ex2_approx(a1.x - m2);
        }
        const float k127 = __fdiv_rn(127.0f, l);  // P = round(127 * e / l)
        // ---- pass 2: quantise P with the final (max, sum) ----
        for (int j = 0; ok && j < n_kv; ++j) {
            const bool diag = j == qt;
            uint8_t* prow = s_p + r * 128;
            if (!(ok = warp_wait(bar_s_full + g, s_full_ph, abort_flag, p.status, 27))) break;
            s_full_ph ^= 1u;
            tcgen05_fence_after();
            // The codes of this step are computed into registers while the previous step's P.V may still be
            // reading the P tile; only the stores wait for it.  The score half is handed back as soon as it
            // has been read, so the next step's score MMA overlaps the rest of this one.
            uint32_t w[2][8];
#pragma unroll
            for (int ci = 0; ci < 2; ++ci) {
                const int cc = 2 * g + ci;
                uint32_t acc[32];
                tmem_ld32(tmem_s + lane_addr + cc * 32, acc);
                tmem_ld_wait();
                if (!diag) pass2_chunk<true>(acc, 32, c1, m2, k127, w[ci]);
                else pass2_chunk<false>(acc, min(32, r - cc * 32 + 1), c1, m2, k127, w[ci]);
            }
            tcgen05_fence_before();
            mbar_arrive(bar_s_free + g);
            if (j > 0) {  // the previous step's P.V has finished reading the P tile
                if (!(ok = warp_wait(bar_pv_done, pv_done_ph, abort_flag, p.status, 28))) break;
                pv_done_ph ^= 1u;
            }
#pragma unroll
            for (int ci = 0; ci < 2; ++ci) {
                const int piece = (2 * g + ci) * 2;
                *reinterpret_cast<uint4*>(prow + (((piece) ^ (r & 7)) << 4)) = make_uint4(w[ci][0], w[ci][1], w[ci][2], w[ci][3]);
                *reinterpret_cast<uint4*>(prow + (((piece + 1) ^ (r & 7)) << 4)) = make_uint4(w[ci][4], w[ci][5], w[ci][6], w[ci][7]);
            }
            asm volatile("fence.proxy.async.shared::cta;" ::: "memory");  // P tile: generic writes -> MMA reads
            mbar_arrive(bar_p_full);
        }
        // ---- epilogue: out = round(((P V) * alpha_pv) * requant); each half takes 64 output channels ----
        if (ok && (ok = warp_wait(bar_pv_done, pv_done_ph, abort_flag, p.status, 29))) {
            tcgen05_fence_after();
            int8_t* orow = p.out + ((int64_t)(row_base + qi)) * p.hid + h * TILE;
#pragma unroll 1
            for (int cc = 2 * g; cc < 2 * g + 2; ++cc) {
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
    if (warp == CTRL_WARP) {
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
