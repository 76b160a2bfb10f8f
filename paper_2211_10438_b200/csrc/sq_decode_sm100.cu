// Decode-shaped W8A8 linear (M <= 32 tokens): the weight matrix is streamed once from HBM and
// everything else is noise, so the kernel is laid out around that stream.
//
//   * operands are swapped: 128 OUTPUT CHANNELS of W (128 x 128 bytes per K slice) ride on the
//     MMA's M dimension and the tokens on its N dimension (tcgen05.mma.kind::i8, 128 x 16 x 32
//     or 128 x 32 x 32), so no tile is padded from 16 to 128 rows and a stage is 18 or 20 KB;
//   * every CTA gets the same number of K blocks whatever N and K are: as many whole 128-channel
//     tiles as divide evenly among the CTAs, plus an equal contiguous range of the remaining
//     tiles' (tile, K block) pairs, tile-major ("stream-K"), whose K ranges are then shared by
//     two or more CTAs.  The shared part is done first, the whole tiles last;
//   * a 10-stage TMA ring keeps ~180 KB of weights in flight per SM;
//   * a CTA parks the partial accumulators of a shared tile in its own slot of the workspace
//     with plain stores (INT32 partial sums add exactly in any order); the CTA that arrives
//     last for a tile (one atomic counter per tile) adds the other slots, applies Eq. 2
//     (dequant, bias, ReLU, requant), writes Y and leaves the counter zeroed for the next call.
//   * optionally the activation quantiser runs INSIDE this kernel (Eq. 1 per token, or with a given
//     static step; optionally behind the folded LayerNorm): while every CTA's first weight slices
//     are already in flight, CTA r pulls token row r into the top of its own ring with one bulk
//     copy and quantises it (16-bit values -> INT8 codes + step size), the CTAs meet on one
//     counter, and only then are the activation slices fetched.  The codes are parked in the
//     workspace K block by K block, each block already in the 128-byte-swizzled image the MMA
//     reads, so an activation slice is ONE contiguous bulk copy per stage instead of a strided
//     box of 16 or 32 rows.  The quantiser's cost hides behind the first fill of the ring instead
//     of being a launch of its own in front of the GEMM.
// Every wait is bounded (status word, as in the prefill kernel).
#include "sq_bulk.cuh"
#include "sq_kernels.h"
#include "sq_tcgen05.cuh"

namespace sq {

namespace {

using namespace tc;

constexpr int DEC_THREADS = 192;      // warp 0: TMA, warp 1: MMA + TMEM, warps 2-5: epilogue
constexpr int DEC_QUANT_THREADS = 256;  // prologue quantiser: the epilogue warps + 4 helper warps (more warps hide
                                        // the latency of its dependent instruction chains; 12 would cap the kernel
                                        // at 128 registers per thread and spill the 32-token epilogue)
constexpr int DEC_THREADS_FUSED = 64 + DEC_QUANT_THREADS;
constexpr int DEC_MAX_N = 32;         // most tokens this kernel takes
constexpr int W_BYTES = BLOCK_M * BLOCK_K;  // 16 KB of weights per stage
// DN = tokens per MMA (its N dimension): 16 or 32.  A stage holds 16 KB of weights and
// DN * 128 bytes of activations; the ring is as deep as shared memory allows (10 stages).
template <int DN>
struct DecCfg {
    static constexpr int X_BYTES = DN * BLOCK_K;
    static constexpr int STAGE = W_BYTES + X_BYTES;
#ifndef SQ_DEC_STAGES  // tuning builds may override it (-DSQ_DEC_STAGES=5)
#define SQ_DEC_STAGES 10
#endif
    static constexpr int STAGES = SQ_DEC_STAGES;
    static constexpr int TMEM_COLS = 2 * DN < 32 ? 32 : 2 * DN;  // two accumulator slots
    static constexpr int SMEM = 1024 + STAGES * STAGE + (2 * STAGES + 7) * 8 + 64 + DN * 4 + 64;
};

// Tuning aid, compiled out unless SQ_DEC_TRACE is defined (python -m paper_2211_10438_b200.build --trace
// builds libsq_trace.so): one thread per role stores its SM's cycle counter at fixed points of a
// CTA's life (reading the global nanosecond timer costs a fraction of a microsecond per read and
// would inflate every interval; cycle counters of different SMs are not aligned, so only differences
// within a CTA mean anything); sq_debug_decode_trace() copies the table of the last launch to the
// host and clears it.
#ifdef SQ_DEC_TRACE
constexpr int kTraceSlots = 16, kTraceLaunches = 8;
__device__ unsigned long long g_dec_trace[kTraceLaunches][256][kTraceSlots];  // the last 8 launches, round robin
__device__ __forceinline__ void dec_trace(int launch, int slot) {
    g_dec_trace[launch][blockIdx.x][slot] = (unsigned long long)clock64();
}
#define DEC_TRACE(slot) dec_trace(p.trace_id, slot)
#else
#define DEC_TRACE(slot) ((void)0)
#endif

struct DecParams {
    int M;
    int64_t N, K;
    int num_n, num_kb;
    int64_t total_kb;    // sk_tiles * num_kb: the (tile, K block) pairs of the shared tiles, tile-major
    int range;           // of those, K blocks per CTA: CTA g owns positions [g * range, (g + 1) * range)
    int maxcount;        // most CTAs that share one tile
    int trace_id;        // SQ_DEC_TRACE builds: which of the trace tables this launch writes
    int l2_ahead;        // K blocks beyond the ring that a CTA pulls into L2 while it waits at its start
    int sk_tiles;        // tiles [0, sk_tiles) are shared; tile sk_tiles + i * grid + g is whole tile i of CTA g
    int whole_per_cta;
    const float* x_scale; int x_per_row;
    const float* w_scale; int w_per_col;
    float alpha;         // the tokens' common factor when x_scale == nullptr (batched-matmul calls)
    const void* bias; int bias_is_bf16;
    int relu;
    const float* requant_mul; int requant_per_col;  // INT8 output: code = round(y * r)
    void* Y; int out_dt; int64_t ldy;
    int32_t* part;       // [num_n][maxcount][M][128] partial sums of tiles shared by several CTAs
    uint32_t* counters;  // [num_n] arrivals per shared tile, zero on entry and on exit
    const void* residual;  // nullable: [M, N] of the output type, row stride ld_res
    int64_t ld_res;
    uint32_t* status;
    // Activation quantiser in the prologue (x_raw != nullptr).  x_scale then points at the step sizes
    // the prologue itself writes (per-token dynamic) or at the caller's static step.
    const void* x_raw;      // [M, K] fp16 / bf16, contiguous
    int x_is_bf16;
    const void* ln_gamma;   // nullable: folded LayerNorm parameters [K] of x_raw's type -> LayerNorm first
    const void* ln_beta;    // nullable
    float ln_eps;
    int x_static;           // 1: Delta = x_scale[0] is given; 0: Delta_t = absmax(row t) / 127 -> xs_out[t]
    int8_t* xq;             // [num_kb][DN][128] codes, K block by K block, each block in the swizzled
                            // shared-memory image of a stage's activation slot
    int8_t* xq_rows;        // nullable: [M, K] the same codes row-major (a caller who wants to see them)
    int row_stages;         // ring stages a token row of x_raw (and the LayerNorm parameters behind it) occupy
                            // while it is quantised; 0: they do not fit and are read from global memory
    float* xs_out;          // [M] step sizes (dynamic mode)
    float* stats_out;       // nullable [2 M]: mean and 1/sqrt(var + eps) of every row
    uint32_t* sync;         // [2]: rows quantised so far, CTAs past the meeting point; zero between calls
};

// A CTA's work in the order it is done: first its contiguous range of the SHARED tiles' (tile, K
// block) pairs, then its whole tiles.  The shared tiles come first so that their fix-up (partial
// sums parked, the last arriver adds them) runs in the epilogue warps while the CTA already streams
// its next tile; what a CTA ends on is a whole tile with a plain epilogue.  (With every tile shared
// and finished at the very end, each CTA spent 4.4 us between its last MMA and its exit.)
struct DecWalk {
    int64_t pos, end;
    int whole_i;
    __device__ __forceinline__ explicit DecWalk(const DecParams& p)
        : pos((int64_t)blockIdx.x * p.range), end(min((int64_t)blockIdx.x * p.range + (int64_t)p.range, p.total_kb)), whole_i(0) {}
    __device__ __forceinline__ bool next(const DecParams& p, int& ni, int& kb0, int& kb1) {
        if (pos < end) {
            ni = (int)(pos / p.num_kb);
            kb0 = (int)(pos % p.num_kb);
            kb1 = (int)min((int64_t)p.num_kb, kb0 + (end - pos));
            pos += kb1 - kb0;
            return true;
        }
        if (whole_i < p.whole_per_cta) {
            ni = p.sk_tiles + whole_i * (int)gridDim.x + (int)blockIdx.x;
            ++whole_i;
            kb0 = 0;
            kb1 = p.num_kb;
            return ni < p.num_n;
        }
        return false;
    }
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
__device__ __forceinline__ void dec_quant_sync() { asm volatile("bar.sync 3, %0;" ::"n"(DEC_QUANT_THREADS) : "memory"); }

// ------------------------------------------------------------------------------------
// The activation quantiser of the prologue: one token row per call, by DEC_QUANT_THREADS threads.
// Arithmetic is the library's normative fp32 sequence (Eq. 1: Delta = max(m, 1e-5) / 127,
// code = round(v * (1 / Delta)); LayerNorm: n = fma(x, rstd, -(mu * rstd)), y = fma(n, g, b),
// statistics two-pass in fp32), so codes and step sizes equal those of sq_quant_act /
// sq_ln_quant given the same statistics.
// ------------------------------------------------------------------------------------
template <bool IS_MAX>
__device__ __forceinline__ float dec_quant_reduce(float v, float* red, int wq, int lane) {
    constexpr int NW = DEC_QUANT_THREADS / 32;
    v = IS_MAX ? warp_max(v) : warp_sum(v);
    if (lane == 0) red[wq] = v;
    dec_quant_sync();
    float r = red[0];  // every thread folds the partials in the same order
#pragma unroll
    for (int i = 1; i < NW; ++i) r = IS_MAX ? fmaxf(r, red[i]) : r + red[i];
    dec_quant_sync();  // `red` is rewritten by the next reduction
    return r;
}

template <typename T>
__device__ __forceinline__ void dec_ln_vec(const uint4& xv, const uint4* g4, const uint4* b4, int v, float rstd,
                                           float shift, float (&y)[8]) {
    float x[8], g[8], b[8];
    unpack8<T>(xv, x);
    unpack8<T>(g4[v], g);
    if (b4 != nullptr) unpack8<T>(b4[v], b);
#pragma unroll
    for (int k = 0; k < 8; ++k)
        y[k] = __fmaf_rn(__fmaf_rn(x[k], rstd, shift), g[k], b4 != nullptr ? b[k] : 0.0f);
}

// `src`: the row's 16-byte vectors, in shared memory (the usual case) or in global memory.
// This code runs once per launch, so what it costs is fetching its instructions: with the passes
// unrolled (or the row cached in registers by straight-line code) a 12 288-element row took 1.4 us
// whatever the arithmetic was; as compact loops whose body is fetched once it takes a third of that.
template <typename T, int DN>
__device__ void dec_quant_row(const DecParams& p, int row, int et, const uint4* __restrict__ src,
                              const uint4* __restrict__ g4, const uint4* __restrict__ b4, float static_delta, float* red) {
    constexpr int NT = DEC_QUANT_THREADS;
    const int wq = et >> 5, lane = et & 31;
    const int nvec = (int)(p.K >> 3);
    const bool ln = g4 != nullptr;
    float rstd = 1.0f, shift = 0.0f;
    if (ln) {
        const float inv_C = __fdiv_rn(1.0f, (float)p.K);
        float sum = 0.0f;
#pragma unroll 2
        for (int v = et; v < nvec; v += NT) {
            float f[8];
            unpack8<T>(src[v], f);
            sum += ((f[0] + f[1]) + (f[2] + f[3])) + ((f[4] + f[5]) + (f[6] + f[7]));
        }
        const float mu = dec_quant_reduce<false>(sum, red, wq, lane) * inv_C;
        float ss = 0.0f;
#pragma unroll 2
        for (int v = et; v < nvec; v += NT) {
            float f[8];
            unpack8<T>(src[v], f);
#pragma unroll
            for (int k = 0; k < 8; ++k) { const float d = f[k] - mu; ss = fmaf(d, d, ss); }
        }
        ss = dec_quant_reduce<false>(ss, red, wq, lane);
        rstd = rsqrt_refined(ss * inv_C + p.ln_eps);
        shift = -__fmul_rn(mu, rstd);
        if (p.stats_out != nullptr && et == 0) {
            p.stats_out[2 * row] = mu;
            p.stats_out[2 * row + 1] = rstd;
        }
    }
    float delta;
    if (p.x_static) {
        delta = static_delta;
    } else {
        float m = 0.0f;
        if (ln) {
#pragma unroll 2
            for (int v = et; v < nvec; v += NT) {
                float y[8];
                dec_ln_vec<T>(src[v], g4, b4, v, rstd, shift, y);
#pragma unroll
                for (int k = 0; k < 8; ++k) m = fmaxf(m, fabsf(y[k]));
            }
        } else {
            uint32_t pm0 = 0u, pm1 = 0u;  // |x| and max are exact on the packed 16-bit values
#pragma unroll 2
            for (int v = et; v < nvec; v += NT) {
                const uint4 x = src[v];
                pm0 = Act<T>::absmax2(pm0, x.x); pm1 = Act<T>::absmax2(pm1, x.y);
                pm0 = Act<T>::absmax2(pm0, x.z); pm1 = Act<T>::absmax2(pm1, x.w);
            }
            m = fmaxf(Act<T>::hmax_of2(pm0), Act<T>::hmax_of2(pm1));
        }
        m = dec_quant_reduce<true>(m, red, wq, lane);
        if (et == 0) DEC_TRACE(13);
        delta = step_size(m);
        if (et == 0) p.xs_out[row] = delta;
    }
    const float inv = recip_step(delta);
    uint2* rows_out = p.xq_rows != nullptr ? reinterpret_cast<uint2*>(p.xq_rows + (int64_t)row * p.K) : nullptr;
    int8_t* const blk_row = p.xq + (size_t)row * BLOCK_K;
    const int sw = row & 7;
    const float lo = p.x_static ? kRoundMagic - 127.0f : -INFINITY, hi = p.x_static ? kRoundMagic + 127.0f : INFINITY;
#pragma unroll 2
    for (int v = et; v < nvec; v += NT) {
        float y[8];
        if (ln) dec_ln_vec<T>(src[v], g4, b4, v, rstd, shift, y);
        else unpack8<T>(src[v], y);
        uint32_t cdw[8];
#pragma unroll
        for (int k = 0; k < 8; ++k)  // round(y * inv) in one FMA; a given static step may be exceeded: saturate
            cdw[k] = __float_as_uint(fminf(fmaxf(__fmaf_rn(y[k], inv, kRoundMagic), lo), hi));
        const uint2 q = make_uint2(pack4(cdw[0], cdw[1], cdw[2], cdw[3]), pack4(cdw[4], cdw[5], cdw[6], cdw[7]));
        // vector v = bytes 8v .. 8v+7 of the row: K block kb, 16-byte chunk j of its 128-byte slice;
        // the slice of token `row` sits where a 128-byte-swizzled tensor copy would have put it
        const int kb = v >> 4, j = (v >> 1) & 7, half = v & 1;
        *reinterpret_cast<uint2*>(blk_row + (size_t)kb * (DN * BLOCK_K) + ((j ^ sw) << 4) + half * 8) = q;
        if (rows_out != nullptr) rows_out[v] = q;
    }
}

__device__ __forceinline__ uint32_t ld_acquire_gpu(const uint32_t* ptr) {
    uint32_t v;
    asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(ptr) : "memory");
    return v;
}

// Per-channel constants of Eq. 2, fetched while the tile's weights are still streaming.
struct DecChan { float ws, bs, rq; };
__device__ __forceinline__ DecChan dec_chan(const DecParams& p, int64_t col) {
    DecChan c = {1.0f, 0.0f, 1.0f};
    if (col >= p.N || p.out_dt == SQ_I32) return c;
    if (p.w_scale) c.ws = __ldg(p.w_scale + (p.w_per_col ? col : 0));
    if (p.bias)
        c.bs = p.bias_is_bf16 ? __bfloat162float(static_cast<const __nv_bfloat16*>(p.bias)[col])
                              : __half2float(static_cast<const __half*>(p.bias)[col]);
    if (p.requant_mul) c.rq = __ldg(p.requant_mul + (p.requant_per_col ? col : 0));
    return c;
}

// Eq. 2 for one output channel (this thread) and all tokens, then the stores.  xs: the tokens'
// step sizes, staged in shared memory.
// The residual elements of one output channel, all tokens (16-bit bit patterns).  Fetched with the
// per-channel constants, before the accumulators are waited for: in the last arriver's tail a
// demand load would wait microseconds behind the other CTAs' weight streams.
template <int DN>
__device__ __forceinline__ void dec_residual(const DecParams& p, int64_t col, uint16_t (&res)[DN]) {
#pragma unroll
    for (int t = 0; t < DN; ++t)
        res[t] = (p.residual && t < p.M && col < p.N)
                     ? __ldg(static_cast<const uint16_t*>(p.residual) + (int64_t)t * p.ld_res + col) : (uint16_t)0;
}

template <int DN>
__device__ __forceinline__ void dec_finish(const DecParams& p, const int32_t (&acc)[DN], int64_t col, const DecChan& c,
                                           const float* xs_smem, const uint16_t (&res)[DN]) {
    if (col >= p.N) return;
    if (p.out_dt == SQ_I32) {
        int32_t* y = static_cast<int32_t*>(p.Y);
#pragma unroll
        for (int t = 0; t < DN; ++t)
            if (t < p.M) y[(int64_t)t * p.ldy + col] = acc[t];
        return;
    }
#pragma unroll
    for (int t = 0; t < DN; ++t) {
        if (t < p.M) {
            float v = __fmaf_rn(__int2float_rn(acc[t]), __fmul_rn(xs_smem[t], c.ws), c.bs);
            if (p.relu) v = fmaxf(v, 0.0f);
            if (p.residual) {  // round to the output type, then the residual add (rounded by the store below)
                v = p.out_dt == SQ_BF16
                        ? __bfloat162float(__float2bfloat16_rn(v)) + __uint_as_float((uint32_t)res[t] << 16)
                        : __half2float(__float2half_rn(v)) + __half2float(__ushort_as_half(res[t]));
            }
            if (p.out_dt == SQ_I8)
                static_cast<int8_t*>(p.Y)[(int64_t)t * p.ldy + col] = (int8_t)(quant_code(v, c.rq) & 0xffu);
            else if (p.out_dt == SQ_BF16)
                static_cast<__nv_bfloat16*>(p.Y)[(int64_t)t * p.ldy + col] = __float2bfloat16_rn(v);
            else
                static_cast<__half*>(p.Y)[(int64_t)t * p.ldy + col] = __float2half_rn(v);
        }
    }
}

// FUSED: the activation quantiser runs in the prologue (8 helper warps more; see the file header).
template <int DN, bool FUSED>
__global__ void __launch_bounds__(FUSED ? DEC_THREADS_FUSED : DEC_THREADS, 1)
decode_gemm_kernel(const __grid_constant__ CUtensorMap tmap_w, const __grid_constant__ CUtensorMap tmap_x,
                   const DecParams p) {
    constexpr int DEC_N = DN, DEC_STAGE = DecCfg<DN>::STAGE, DEC_STAGES = DecCfg<DN>::STAGES;
    constexpr int DEC_TMEM_COLS = DecCfg<DN>::TMEM_COLS;
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
    uint64_t* full_bar = reinterpret_cast<uint64_t*>(smem + DEC_STAGES * DEC_STAGE);
    uint64_t* empty_bar = full_bar + DEC_STAGES;
    uint64_t* tmem_full = empty_bar + DEC_STAGES;
    uint64_t* tmem_empty = tmem_full + 2;
    uint64_t* x_ready = tmem_empty + 2;  // prologue quantiser: every token row has been written
    uint64_t* x_row_bar = x_ready + 1;   // prologue quantiser: this CTA's token row has landed in the ring
    uint64_t* x_ln_bar = x_row_bar + 1;  // prologue quantiser: the LayerNorm parameters have landed in the ring
    uint32_t* tmem_holder = reinterpret_cast<uint32_t*>(x_ln_bar + 1);
    volatile uint32_t* abort_flag = tmem_holder + 1;
    volatile uint32_t* epi_go = tmem_holder + 2;
    volatile uint32_t* epi_last = tmem_holder + 3;
    float* s_xs = reinterpret_cast<float*>(tmem_holder + 4);  // [DN] the tokens' step sizes
    float* s_red = s_xs + DEC_N;                              // [8] reduction scratch of the prologue quantiser

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
        mbar_init(x_ready, 1);
        mbar_init(x_row_bar, 1);
        mbar_init(x_ln_bar, 1);
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
            DEC_TRACE(0);
            int stage = 0;
            uint32_t phase = 0;
            bool ok = true;
            // The weights are static, the activations come from the kernel in front (or from this
            // kernel's own quantiser): fill the ring with weight slices first, wait for the
            // predecessor (and for the quantiser), then add the activation slices of those stages.
            // A CTA that quantises a token row keeps the top of its ring free for that row.
            constexpr bool fused = FUSED;
            const uint64_t stream_once = l2_policy_evict_first();
            auto load_x = [&](uint8_t* sx, uint64_t* bar, int kb) {
                if (fused)  // one contiguous, pre-swizzled block per K block
                    bulk::bulk_load(sx, p.xq + (size_t)kb * DecCfg<DN>::X_BYTES, DecCfg<DN>::X_BYTES, bar);
                else
                    tma_load_4d<1>(sx, &tmap_x, bar, kb * BLOCK_K, 0, 0, 0);
            };
            bool waited = false;
            DecWalk walk(p);
            int ni, kb0, kb1;
            while (ok && walk.next(p, ni, kb0, kb1)) {
                int kb = kb0;
                if (!waited) {
                    int n_pre = min(DEC_STAGES, kb1 - kb0);
                    if (fused && (int)blockIdx.x < p.M) n_pre = max(0, min(n_pre, DEC_STAGES - p.row_stages));
                    for (int i = 0; i < n_pre; ++i) {
                        mbar_expect_tx(full_bar + i, DEC_STAGE);
                        tma_load_4d_policy(smem + i * DEC_STAGE, &tmap_w, full_bar + i, (kb0 + i) * BLOCK_K, ni * BLOCK_M, 0, 0,
                                           stream_once);
                    }
                    // The weights are static and this lane is about to wait (for the launch in front, then
                    // for the quantiser): meanwhile the next slices of this CTA's stream go to L2, so that
                    // HBM keeps working through the gap between two launches.
                    {
                        DecWalk ahead(p);
                        int ni2, a2, b2, idx = 0;
                        const int stop = n_pre + p.l2_ahead;
                        while (idx < stop && ahead.next(p, ni2, a2, b2))
                            for (int k2 = a2; k2 < b2 && idx < stop; ++k2, ++idx)
                                if (idx >= n_pre) tma_prefetch_l2_4d(&tmap_w, k2 * BLOCK_K, ni2 * BLOCK_M, 0, 0);
                    }
                    DEC_TRACE(1);
                    pdl_wait();
                    DEC_TRACE(2);
#ifdef SQ_DEC_TRACE
                    {  // one global-timer read per CTA relates the launches of a chain to each other
                        unsigned long long t;
                        asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
                        g_dec_trace[p.trace_id][blockIdx.x][4] = t;
                    }
#endif
                    // with the quantiser in the prologue the codes of X exist once every CTA's rows are done
                    if (fused && !(ok = mbar_wait(x_ready, 0u, abort_flag, p.status, 11))) break;
                    DEC_TRACE(3);
                    for (int i = 0; i < n_pre; ++i) load_x(smem + i * DEC_STAGE + W_BYTES, full_bar + i, kb0 + i);
                    waited = true;
                    kb = kb0 + n_pre;
                    stage = n_pre % DEC_STAGES;
                    phase = (n_pre == DEC_STAGES) ? 1u : 0u;
                }
                for (; kb < kb1; ++kb) {
                    if (!(ok = mbar_wait(empty_bar + stage, phase ^ 1u, abort_flag, p.status, 6))) break;
                    uint8_t* sw = smem + stage * DEC_STAGE;
                    mbar_expect_tx(full_bar + stage, DEC_STAGE);
                    tma_load_4d_policy(sw, &tmap_w, full_bar + stage, kb * BLOCK_K, ni * BLOCK_M, 0, 0, stream_once);
                    load_x(sw + W_BYTES, full_bar + stage, kb);
                    if (++stage == DEC_STAGES) { stage = 0; phase ^= 1u; }
                }
            }
        }
    } else if (warp == 1) {
        // ============================ MMA issuer ==============================
        // The whole warp walks the tiles and waits on the barriers, converged; one elected lane issues the
        // MMAs and the commits (their operands are then warp-uniform values to the compiler).
        {
            const uint32_t idesc = make_idesc(BLOCK_M, DEC_N, 0);
            constexpr uint32_t kStage16 = (uint32_t)DEC_STAGE >> 4;
            const uint32_t w_lo0 = smem_desc_lo(smem_u32(smem), 16);
            const uint32_t x_lo0 = smem_desc_lo(smem_u32(smem) + (uint32_t)W_BYTES, 16);
            const uint32_t full0 = smem_u32(full_bar), empty0 = smem_u32(empty_bar);
            const uint32_t tmem_full0 = smem_u32(tmem_full), tmem_empty0 = smem_u32(tmem_empty);
            int stage = 0;
            uint32_t phase = 0;
            int slot = 0;
            uint32_t slot_phase = 0;
            bool ok = true;
            DecWalk walk(p);
            int ni, kb0, kb1;
            while (ok && walk.next(p, ni, kb0, kb1)) {
                if (!(ok = mbar_wait_warp(tmem_empty + slot, tmem_empty0 + (uint32_t)slot * 8u, slot_phase ^ 1u, abort_flag,
                                          p.status, 7)))
                    break;
                tcgen05_fence_after();
                const uint32_t d_tmem = tmem_base + (uint32_t)(slot * DEC_N);
                uint32_t accumulate = 0u;  // the tile's first MMA overwrites the slot
                for (int kb = kb0; kb < kb1; ++kb) {
                    if (!(ok = mbar_wait_warp(full_bar + stage, full0 + (uint32_t)stage * 8u, phase, abort_flag, p.status, 8)))
                        break;
#ifdef SQ_DEC_TRACE
                    if (lane == 0 && g_dec_trace[p.trace_id][blockIdx.x][5] == 0ull) DEC_TRACE(5);
#endif
                    tcgen05_fence_after();
                    const uint32_t w_lo = w_lo0 + (uint32_t)stage * kStage16;
                    const uint32_t x_lo = x_lo0 + (uint32_t)stage * kStage16;
                    if (elect_one()) {
                        umma_i8_lo<1>(d_tmem, w_lo, x_lo, idesc, accumulate);
#pragma unroll
                        for (int k = 1; k < BLOCK_K / UMMA_K; ++k)
                            umma_i8_lo<1>(d_tmem, w_lo + k * (UMMA_K >> 4), x_lo + k * (UMMA_K >> 4), idesc, 1u);
                        umma_commit_u32<1>(empty0 + (uint32_t)stage * 8u);
                    }
                    accumulate = 1u;
                    if (++stage == DEC_STAGES) { stage = 0; phase ^= 1u; }
                }
                if (!ok) break;
                if (elect_one()) umma_commit_u32<1>(tmem_full0 + (uint32_t)slot * 8u);
#ifdef SQ_DEC_TRACE
                if (lane == 0) DEC_TRACE(6);
#endif
                slot ^= 1;
                if (slot == 0) slot_phase ^= 1u;
            }
        }
    } else {
        // ============================ epilogue (warps 2-5) ====================
        float static_delta = 0.0f;
        if constexpr (FUSED) {
            // The folded LayerNorm parameters are static: a CTA that will quantise a token row pulls them
            // into the top of its ring (behind the row's own place) before it waits for the launch in front
            if (threadIdx.x == 64 && p.ln_gamma != nullptr && p.row_stages > 0 && (int)blockIdx.x < p.M) {
                uint8_t* top = smem + (DEC_STAGES - p.row_stages) * DEC_STAGE;
                const uint32_t rb = (uint32_t)(p.K * 2);
                mbar_expect_tx(x_ln_bar, p.ln_beta != nullptr ? 2 * rb : rb);
                bulk::bulk_load(top + rb, p.ln_gamma, rb, x_ln_bar);
                if (p.ln_beta != nullptr) bulk::bulk_load(top + 2 * rb, p.ln_beta, rb, x_ln_bar);
            }
            // ... and a static step is a calibrated constant: fetched now, it is there when the row lands
            // (read after the wait, one L2 miss queued behind every CTA's weight prefetch cost 3-5 us)
            if (p.x_static) static_delta = __ldg(p.x_scale);
        }
        pdl_wait();  // a dynamic x_scale and the split-K scratch belong to earlier kernels until here
        if (threadIdx.x == 64) DEC_TRACE(7);
        const int quarter = warp & 3;           // TMEM lanes this warp may read
        const int ch = quarter * 32 + lane;     // output channel within the tile
        const int et = threadIdx.x - 64;        // 0..127
        bool x_ok = true;
        if constexpr (FUSED) {
            // ---- activation quantiser (warps 2-9): CTA r takes token rows r, r + grid, ... ----
            uint32_t done = 0;
            bool row_ok = true;
            for (int row = (int)blockIdx.x; row < p.M; row += (int)gridDim.x, ++done) {
                const uint8_t* grow = static_cast<const uint8_t*>(p.x_raw) + (size_t)row * (size_t)p.K * 2;
                const uint4* src = reinterpret_cast<const uint4*>(grow);
                const uint4* g4 = reinterpret_cast<const uint4*>(p.ln_gamma);
                const uint4* b4 = reinterpret_cast<const uint4*>(p.ln_beta);
                if (p.row_stages > 0) {
                    // the row lands in the top stages of the ring (the producer lane leaves them
                    // alone until the meeting below) with one bulk copy
                    uint8_t* rowbuf = smem + (DEC_STAGES - p.row_stages) * DEC_STAGE;
                    const uint32_t rb = (uint32_t)(p.K * 2);
                    if (et == 0) {
                        mbar_expect_tx(x_row_bar, rb);
                        bulk::bulk_load(rowbuf, grow, rb, x_row_bar);
                        bool ok = mbar_wait(x_row_bar, done & 1u, abort_flag, p.status, 12);
                        if (ok && g4 != nullptr && done == 0) ok = mbar_wait(x_ln_bar, 0u, abort_flag, p.status, 13);
                        *epi_go = ok ? 1u : 0u;
                    }
                    if (g4 != nullptr) {
                        g4 = reinterpret_cast<const uint4*>(rowbuf + rb);
                        if (b4 != nullptr) b4 = reinterpret_cast<const uint4*>(rowbuf + 2 * rb);
                    }
                    dec_quant_sync();
                    if (et == 0) DEC_TRACE(8);
                    row_ok = *epi_go != 0u;
                    src = reinterpret_cast<const uint4*>(rowbuf);
                    if (!row_ok) break;  // the copy never landed (same outcome in every thread)
                }
                if (p.x_is_bf16) dec_quant_row<__nv_bfloat16, DEC_N>(p, row, et, src, g4, b4, static_delta, s_red);
                else dec_quant_row<__half, DEC_N>(p, row, et, src, g4, b4, static_delta, s_red);
                dec_quant_sync();  // everyone is done with the row buffer (and with epi_go)
            }
            if (et == 0) {
                DEC_TRACE(14);
                if (done) {
                    // the barrier above ordered every thread's stores before this fence: the count moves
                    // only once this CTA's codes are visible device-wide (also to bulk copies)
                    __threadfence();
                    asm volatile("fence.proxy.async.global;" ::: "memory");
                    atomicAdd(p.sync, done);
                }
                DEC_TRACE(15);
                // meet: all M rows written (bounded, like every other wait of the kernel)
                const long long t0 = clock64();
                bool ok = row_ok;
                while (ok && ld_acquire_gpu(p.sync) < (uint32_t)p.M) {
                    if (*abort_flag || (unsigned long long)(clock64() - t0) > (unsigned long long)kWaitCycles) ok = false;
                }
                if (ok) {
                    DEC_TRACE(10);
                    asm volatile("fence.proxy.async.global;" ::: "memory");
                    mbar_arrive(x_ready);  // the producer lane may fetch activation slices now
                } else {
                    *abort_flag = 1u;
                    atomicCAS(p.status, 0u, ((uint32_t)SQ_ERR_TIMEOUT) | (10u << 8));
                }
                *epi_go = ok ? 1u : 0u;
                // whoever passes last hands the two counters back zeroed (every CTA has added its rows
                // before it came here, and nobody looks at them again)
                if (atomicAdd(p.sync + 1, 1u) == gridDim.x - 1) {
                    p.sync[0] = 0u;
                    p.sync[1] = 0u;
                }
            }
            dec_quant_sync();
            x_ok = *epi_go != 0u;
        }
        if (warp < 6) {  // the helper warps of the quantiser are done; the four epilogue warps go on
        dec_epi_sync();  // (epi_go is rewritten in the loop below)
        // step sizes: the caller's, or the ones the prologue just wrote (read through L2)
        if (et < DEC_N) s_xs[et] = (et < p.M && p.x_scale) ? __ldcg(p.x_scale + (p.x_per_row ? et : 0)) : p.alpha;
        dec_epi_sync();
        int slot = 0;
        uint32_t slot_phase = 0;
        DecWalk walk(p);
        int ni, kb0, kb1;
        while (x_ok && walk.next(p, ni, kb0, kb1)) {
            const int64_t col = (int64_t)ni * BLOCK_M + ch;
            const DecChan chan = dec_chan(p, col);  // in flight while the K blocks stream
            uint16_t res[DEC_N];
            dec_residual<DEC_N>(p, col, res);
            if (et == 0) *epi_go = mbar_wait(tmem_full + slot, slot_phase, abort_flag, p.status, 9) ? 1u : 0u;
            dec_epi_sync();
            if (*epi_go == 0u) break;
#ifdef SQ_DEC_TRACE
            if (et == 0 && g_dec_trace[p.trace_id][blockIdx.x][11] == 0ull) DEC_TRACE(11);
#endif
            tcgen05_fence_after();
            int32_t acc[DEC_N];
#pragma unroll
            for (int c0 = 0; c0 < DEC_N; c0 += 16) {
                uint32_t r[16];
                tmem_ld16(tmem_base + ((uint32_t)(quarter * 32) << 16) + (uint32_t)(slot * DEC_N + c0), r);
                tmem_ld_wait();
#pragma unroll
                for (int t = 0; t < 16; ++t) acc[c0 + t] = (int32_t)r[t];
            }
            tcgen05_fence_before();
            mbar_arrive(tmem_empty + slot);  // slot drained into registers
            slot ^= 1;
            if (slot == 0) slot_phase ^= 1u;

            if (kb0 == 0 && kb1 == p.num_kb) {
                dec_finish<DEC_N>(p, acc, col, chan, s_xs, res);  // the whole K range of this tile was ours
            } else {
                // The tile is shared: CTAs g0 .. g0 + count - 1 each hold one K piece.  Park this
                // piece in its own slot (plain stores: integer partial sums add exactly in any
                // order); whoever arrives last adds the others and applies Eq. 2.
                const int g0 = (int)(((int64_t)ni * p.num_kb) / p.range);
                const int count = (int)(((int64_t)(ni + 1) * p.num_kb - 1) / p.range) - g0 + 1;
                const int mine = (int)blockIdx.x - g0;
                int32_t* slot0 = p.part + ((int64_t)ni * p.maxcount) * p.M * BLOCK_M;
#pragma unroll
                for (int t = 0; t < DEC_N; ++t)
                    if (t < p.M) __stcg(slot0 + ((int64_t)mine * p.M + t) * BLOCK_M + ch, acc[t]);
                __threadfence();
                dec_epi_sync();
                if (et == 0) *epi_last = (atomicAdd(p.counters + ni, 1u) == (uint32_t)(count - 1)) ? 1u : 0u;
                dec_epi_sync();
                if (*epi_last != 0u) {
                    __threadfence();
                    // the other pieces, several at a time so that their loads are in flight together
                    constexpr int J = DEC_N <= 16 ? 4 : 2;
                    for (int o0 = 0; o0 < count; o0 += J) {
                        int32_t other[J][DEC_N];
#pragma unroll
                        for (int j = 0; j < J; ++j) {
                            const int o = o0 + j;
                            const bool use = o < count && o != mine;
#pragma unroll
                            for (int t = 0; t < DEC_N; ++t)
                                other[j][t] = (use && t < p.M) ? __ldcg(slot0 + ((int64_t)o * p.M + t) * BLOCK_M + ch) : 0;
                        }
#pragma unroll
                        for (int j = 0; j < J; ++j)
#pragma unroll
                            for (int t = 0; t < DEC_N; ++t) acc[t] += other[j][t];
                    }
                    dec_finish<DEC_N>(p, acc, col, chan, s_xs, res);
                    if (et == 0) p.counters[ni] = 0u;  // hand the counters back zeroed
                }
            }
            dec_epi_sync();  // epi_go / epi_last are rewritten by thread 0 in the next round
        }
        if (et == 0) DEC_TRACE(12);
        }  // warp < 6
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

// Work split ("stream-K"): the (tile, K block) pairs, tile-major, are cut into equal contiguous
// ranges, one per CTA, so every SM streams the same number of weight bytes whatever the shape;
// a tile whose K range is cut is finished by the last of the CTAs that share it.
constexpr int kMinKbPerCta = 4;       // below this a CTA's fixed costs outweigh its stream
constexpr int kMaxCtas = 256;         // bound used by the workspace formula
constexpr int64_t kMaxSharedTiles = (int64_t)kDecCounterBytes / 4;

// K blocks beyond its ring that a CTA pulls into L2 while it waits at its start (8 x 16 KB x 148 CTAs =
// 19 MB).  Measured on the GPT-3 shapes, back-to-back calls: 0 -> 8 blocks gains 1.5 to 2 us per call
// (12288 x 49152, 16 tokens: 95.6 -> 93.5 us), 16 the same, 32 and 64 lose it again (the lines are
// evicted before they are used, and the activations with them).
constexpr int kL2AheadBlocks = 8;

struct DecPlan { int ctas, range, maxcount, sk_tiles, whole_per_cta; };
DecPlan plan_decode(int num_n, int num_kb, int sms, bool may_share) {
    DecPlan pl{};
    const int ctas_max = std::min(sms, kMaxCtas);
    if (!may_share) {  // whole tiles only
        pl.ctas = std::min(num_n, ctas_max);
        pl.whole_per_cta = (num_n + pl.ctas - 1) / pl.ctas;
        pl.sk_tiles = 0;
        pl.range = 0;
        pl.maxcount = 1;
        return pl;
    }
    // as many whole tiles per CTA as divide evenly; the remaining tiles (fewer than CTAs) are shared:
    // their (tile, K block) pairs are cut into equal contiguous ranges
    pl.whole_per_cta = num_n / ctas_max;
    pl.sk_tiles = num_n - pl.whole_per_cta * ctas_max;
    const int64_t sk_total = (int64_t)pl.sk_tiles * num_kb;
    if (sk_total == 0) {
        pl.ctas = ctas_max;
        pl.range = 0;
        pl.maxcount = 1;
        return pl;
    }
    const int64_t sk_ctas = std::min<int64_t>(ctas_max, std::max<int64_t>(1, sk_total / kMinKbPerCta));
    pl.range = (int)((sk_total + sk_ctas - 1) / sk_ctas);
    pl.ctas = pl.whole_per_cta > 0 ? ctas_max : (int)((sk_total + pl.range - 1) / pl.range);
    pl.maxcount = (num_kb + pl.range - 2) / pl.range + 1;
    return pl;
}

template <int DN, bool FUSED>
sq_status launch_decode(const GemmArgs& a, const DecParams& p, int ctas, cudaStream_t st) {
    CUtensorMap mw, mx;
    int s0, s1, s2;
    if (!make_map(&mw, a.B, 1, a.K, a.N, 1, 1, a.K, 0, 0, BLOCK_K, BLOCK_M, &s0, &s1, &s2)) return SQ_ERR_CUDA;
    // (with the quantiser in the prologue the activation slices come by plain bulk copies: the
    // map of X is then a placeholder over the weights)
    const void* x_codes = p.x_raw != nullptr ? static_cast<const void*>(a.B) : static_cast<const void*>(a.A);
    if (!make_map(&mx, x_codes, 1, a.K, a.M, 1, 1, a.K, 0, 0, BLOCK_K, DN, &s0, &s1, &s2)) return SQ_ERR_CUDA;
    static bool attr_set[64] = {false};  // per instantiation and device
    int dev = 0;
    SQ_CUDA_OK(cudaGetDevice(&dev));
    if (dev < 0 || dev >= 64 || !attr_set[dev]) {
        SQ_CUDA_OK(cudaFuncSetAttribute(decode_gemm_kernel<DN, FUSED>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                        DecCfg<DN>::SMEM));
        if (dev >= 0 && dev < 64) attr_set[dev] = true;
    }
    return launch_pdl(decode_gemm_kernel<DN, FUSED>, dim3((unsigned)ctas), dim3(FUSED ? DEC_THREADS_FUSED : DEC_THREADS),
                      (size_t)DecCfg<DN>::SMEM, st, 1, mw, mx, p);
}

}  // namespace

// Counters (fixed area, zero between calls) + one slot per (shared tile, sharing CTA).  The
// number of slots is at most ctas + 2 * tiles for any balanced cut, with ctas <= kMaxCtas.
size_t decode_workspace_bytes(int64_t M, int64_t N) {
    const int64_t num_n = (N + tc::BLOCK_M - 1) / tc::BLOCK_M;
    return kWsHeader + kDecCounterBytes + (size_t)(kMaxCtas + 2 * num_n) * (size_t)M * tc::BLOCK_M * sizeof(int32_t);
}

// The same plus what the prologue quantiser writes: 256 bytes of step sizes, then the [M, K] codes.
static size_t round256(size_t v) { return (v + 255) & ~(size_t)255; }
size_t decode_fused_workspace_bytes(int64_t M, int64_t N, int64_t K) {
    const size_t num_kb = (size_t)((K + BLOCK_K - 1) / BLOCK_K), dn = M <= 16 ? 16 : 32;
    return round256(decode_workspace_bytes(M, N)) + 256 + num_kb * dn * BLOCK_K;
}

// Up to 32 tokens the activation slices are a small addition to the weight stream and this kernel
// wins.  Beyond, every K block of every tile would re-read 64 x 128 bytes of activations next to
// its 128 x 128 bytes of weights -- half as many requests again for one SM's copy engine -- and a
// 64-token instantiation measured slower than the prefill kernel on every shape once that kernel
// cut a sparsely filled wave along K and took 128-channel tiles (7168 x 28672, 64 tokens: 62 us
// here, 47 us there; 21504 x 7168: 50 against 38), so it is not built.
bool decode_supports(const GemmArgs& a) {
    return a.M <= DEC_MAX_N && a.batch == 1 && a.heads == 1 && !a.b_is_kn && a.row_absmax_out == nullptr &&
           a.strideA[2] == a.K && a.strideB[2] == a.K;
}

sq_status decode_gemm(const GemmArgs& a, void* workspace, size_t ws_bytes, cudaStream_t st) {
    DecParams p;
    p.M = (int)a.M; p.N = a.N; p.K = a.K;
    p.num_n = (int)((a.N + BLOCK_M - 1) / BLOCK_M);
    p.num_kb = (int)((a.K + BLOCK_K - 1) / BLOCK_K);
    const bool may_share = ws_bytes >= decode_workspace_bytes(a.M, a.N) && p.num_n <= kMaxSharedTiles;
    const DecPlan plan = plan_decode(p.num_n, p.num_kb, sm_count(), may_share);
    p.total_kb = (int64_t)plan.sk_tiles * p.num_kb;
    p.range = plan.range;
    p.maxcount = plan.maxcount;
    p.l2_ahead = kL2AheadBlocks;
    p.trace_id = 0;
#ifdef SQ_DEC_TRACE
    static int trace_launch = 0;
    p.trace_id = (trace_launch++) & 7;
#endif
    p.sk_tiles = plan.sk_tiles;
    p.whole_per_cta = plan.whole_per_cta;
    p.x_scale = a.x_scale; p.x_per_row = a.x_per_row;
    p.w_scale = a.w_scale; p.w_per_col = a.w_per_col;
    p.alpha = a.alpha;
    p.bias = a.bias; p.bias_is_bf16 = a.bias_dt == SQ_BF16;
    p.relu = a.relu;
    p.requant_mul = a.requant_mul; p.requant_per_col = a.requant_per_col;
    p.Y = a.C; p.out_dt = (int)a.out_dt; p.ldy = a.strideC[2];
    p.residual = a.residual; p.ld_res = a.ld_res;
    p.counters = reinterpret_cast<uint32_t*>(static_cast<char*>(workspace) + kWsHeader);
    p.part = reinterpret_cast<int32_t*>(static_cast<char*>(workspace) + kWsHeader + kDecCounterBytes);
    p.status = a.status;
    p.x_raw = a.x_raw; p.x_is_bf16 = a.x_raw_dt == SQ_BF16;
    p.ln_gamma = a.ln_gamma; p.ln_beta = a.ln_beta; p.ln_eps = a.ln_eps;
    p.x_static = a.x_static;
    p.xq = nullptr; p.xq_rows = nullptr; p.row_stages = 0; p.xs_out = nullptr; p.stats_out = a.ln_stats_out; p.sync = nullptr;
    if (a.x_raw != nullptr) {  // the caller (sq_api.cu) has checked that the workspace holds the scratch
        char* scratch = static_cast<char*>(workspace) + round256(decode_workspace_bytes(a.M, a.N));
        p.xs_out = a.xs_out != nullptr ? a.xs_out : reinterpret_cast<float*>(scratch);
        p.xq = reinterpret_cast<int8_t*>(scratch + 256);
        p.xq_rows = a.xq_out;
        // a token row (2 K bytes) is quantised out of the top stages of its CTA's ring when it fits
        const int64_t stage_bytes = a.M <= 16 ? DecCfg<16>::STAGE : DecCfg<32>::STAGE;
        const int64_t parts = a.ln_gamma == nullptr ? 1 : (a.ln_beta == nullptr ? 2 : 3);  // row [+ gamma [+ beta]]
        const int64_t need = (parts * 2 * a.K + stage_bytes - 1) / stage_bytes;
        p.row_stages = need <= DecCfg<16>::STAGES ? (int)need : 0;
        p.sync = reinterpret_cast<uint32_t*>(static_cast<char*>(workspace) + kWsSyncOff);
        if (!a.x_static) { p.x_scale = p.xs_out; p.x_per_row = 1; }
    }
    if (a.x_raw != nullptr)
        return a.M <= 16 ? launch_decode<16, true>(a, p, plan.ctas, st) : launch_decode<32, true>(a, p, plan.ctas, st);
    return a.M <= 16 ? launch_decode<16, false>(a, p, plan.ctas, st) : launch_decode<32, false>(a, p, plan.ctas, st);
}

}  // namespace sq

#ifdef SQ_DEC_TRACE
// Copies the timestamps of the last eight decode-shaped launches to host_out[8 * 256 * 16] and clears them.
extern "C" int sq_debug_decode_trace(unsigned long long* host_out) {
    if (cudaMemcpyFromSymbol(host_out, sq::g_dec_trace, sizeof(sq::g_dec_trace)) != cudaSuccess) return 1;
    void* addr = nullptr;
    if (cudaGetSymbolAddress(&addr, sq::g_dec_trace) != cudaSuccess) return 1;
    return cudaMemset(addr, 0, sizeof(sq::g_dec_trace)) == cudaSuccess ? 0 : 1;
}
#endif
