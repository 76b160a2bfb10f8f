// INT8 GEMM / batched matmul on the 5th-generation tensor cores (sm_100a):
//   acc[t, o] = sum_j A[t, j] * B[o, j]      (Eq. 2's integer factor, INT32 exact)
// with the dequantisation of Eq. 2 (+ bias, ReLU, re-quantisation) fused into the epilogue.
//
// Persistent kernel, one CTA per SM.  With CG = 1 every CTA owns 128 x BLOCK_N tiles; with
// CG = 2 (tcgen05 cta_group::2) the two CTAs of a cluster own a 256 x BLOCK_N tile together:
// each loads its own 128 rows of A and its own half of B, the even CTA issues one MMA for
// both, and each CTA's tensor memory receives its 128 rows of the accumulator.  Pairing cuts
// the shared-memory fill traffic per MMA by a third; no TMA multicast is involved.
// Roles inside a CTA:
//   warp 4 (one lane) : TMA producer -- streams 128-byte-wide K slices of A and B into a
//                       ring of shared-memory stages (128B swizzle), mbarrier-tracked;
//   warp 5 (one lane) : issues tcgen05.mma.kind::i8 (K = 32 per instruction), accumulating
//                       in tensor memory (TMEM), two accumulator slots;
//   warps 0-3         : epilogue -- tcgen05.ld the finished slot, dequantise, store, while
//                       the MMA warp already fills the other slot with the next tile.
// Every wait is bounded: on expiry the CTA records SQ_ERR_TIMEOUT in the status word, lets
// outstanding copies land, frees its TMEM and returns.
#include "sq_kernels.h"
#include "sq_tcgen05.cuh"

namespace sq {

namespace {

using namespace tc;


// EW: epilogue warps, 4 (one per TMEM lane quarter) or 8 (two per quarter, each taking half the
// columns -- for short reductions, where draining the accumulator is the bottleneck).
template <int BLOCK_N, int CG, int EW>
struct Cfg {
    static constexpr int NUM_THREADS = EW * 32 + 64;  // + TMA producer warp + MMA/TMEM warp
    static constexpr int EPI_THREADS = EW * 32;
    static constexpr int B_ROWS = BLOCK_N / CG;  // rows of B this CTA loads per K slice
    static constexpr int A_BYTES = BLOCK_M * BLOCK_K;
    static constexpr int B_BYTES = B_ROWS * BLOCK_K;
    static constexpr int STAGE_BYTES = A_BYTES + B_BYTES;
    static constexpr int STAGING_BYTES = EW * 32 * 128;  // per epilogue warp: 32 rows x 128 bytes
    static constexpr int STAGES = ((EW == 8 ? 176 : 192) * 1024) / STAGE_BYTES;
    // column stride between the two accumulator slots (power of two keeps the allocation simple)
    static constexpr int SLOT_COLS = BLOCK_N <= 32 ? 32 : BLOCK_N <= 64 ? 64 : BLOCK_N <= 128 ? 128 : 256;
    static constexpr int TMEM_COLS = 2 * SLOT_COLS;
    static constexpr int EPI_BYTES = BLOCK_N * 3 * 4;  // per column: w_scale, requant, bias as fp32
    static constexpr int SMEM_BYTES = 1024 /*alignment slack*/ + STAGES * STAGE_BYTES + STAGING_BYTES +
                                      EPI_BYTES + (2 * STAGES + 4) * 8 + 64;
    static_assert(SMEM_BYTES <= 227 * 1024, "shared memory budget");
    static_assert(BLOCK_N % (16 * CG) == 0 && BLOCK_N <= 256, "MMA N constraint");
    static_assert(B_ROWS % 8 == 0, "B tile must be whole 8-row swizzle groups");
};

// Tuning build only (python -m paper_2211_10438_b200.build --trace: -DSQ_GEMM_TRACE): the MMA warp of every
// even CTA records, in SM cycles, what it spends per tile -- index arithmetic before the tile, the wait for
// the accumulator slot, the loop over the K blocks -- and, once, cycles and nanoseconds from its first MMA to
// its last commit (their ratio is the SM clock the launch actually ran at); epilogue warp 0 records how long
// it takes to drain the fourth tile's slot.  sq_debug_gemm_trace() copies the table of the last launch out.
#ifdef SQ_GEMM_TRACE
constexpr int kGemmTraceTiles = 16;
__device__ unsigned long long g_gemm_trace[160][kGemmTraceTiles + 1][4];
__device__ __forceinline__ unsigned long long global_timer_ns() {
    unsigned long long t;
    asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
    return t;
}
#endif

struct Params {
    int64_t M, N, K;
    int heads, batch;
    int num_m, num_n;  // tiles per matrix (num_m counts tiles of 128*CG rows)
    uint32_t total_tiles, per_mat;  // tiles over all matrices / per matrix (after causal compaction)
    int causal_compact;             // per-matrix tiles are enumerated through causal_prefix (num_m <= 32)
    uint32_t causal_prefix[33];     // first compact tile index of every m tile
    int num_kb;
    int b_is_kn;
    int causal;  // attention: A = Q (skip score tiles above the diagonal) or A = P (skip K slices right of it)
    // coordinate slot (1..3) of the row / head / batch dimension in each tensor map
    int a_slot_row, a_slot_head, a_slot_batch;
    int b_slot_row, b_slot_head, b_slot_batch;
    const float* x_scale; int x_per_row;
    const float* w_scale; int w_per_col;
    float alpha;
    const void* bias; int bias_is_bf16;
    int relu;
    const float* requant_mul; int requant_per_col;
    float* row_absmax_out;
    const void* residual; int64_t ld_res;  // [M, N] of the output type, added after the output rounding (plain GEMMs)
    void* C; int out_dt;
    int64_t c_stride_batch, c_stride_head, c_stride_row;
    int c_tma;  // C leaves through TMA stores (needs 16-byte aligned base and strides)
    int c_slot_row, c_slot_head, c_slot_batch;
    uint32_t* status;
    // K split of the last, partly filled wave of tiles (plain GEMMs only; split == 1: none).
    // Units [0, full_tiles) are whole tiles; unit full_tiles + t * split + i is K piece i of tile
    // full_tiles + t.  A piece parks its INT32 accumulators in its slot of `part`; the CTA that
    // arrives last for a tile (per CTA of a pair: `counters`) adds the others and runs the epilogue.
    uint32_t full_tiles, total_units;
    int split, kb_per_piece;
    int32_t* part;
    uint32_t* counters;
    // N split of the last wave, for reductions too short for the K split (nsplit == 1: none): unit
    // full_tiles + t * nsplit + i is column part i (BLOCK_N / nsplit wide, the whole K range) of tile
    // full_tiles + t.  No exchange is needed; the A tile is simply fetched once per part.
    int nsplit;
    // Long reductions of a plain GEMM: the band of A rows (8 m-tiles x K) is read again by every column of tiles and
    // by every wave, the weight tiles only by the pairs that work on them at the same time -- A is loaded with an
    // evict-last L2 policy, B with evict-first, so that the waves after the first find A in L2 instead of in HBM.
    int l2_hints;
};

// unit id -> tile and K-block range; piece < 0 for a whole tile (kb1 is then the tile's own count);
// npart >= 0: the unit is column part npart of its tile (whole K range)
template <bool NS>
__device__ __forceinline__ void unit_of(uint32_t u, const Params& p, uint32_t& tile, int& kb0, int& kb1, int& piece,
                                        int& npart) {
    npart = -1;
    if (u < p.full_tiles) {
        tile = u; kb0 = 0; kb1 = -1; piece = -1;
        return;
    }
    const uint32_t r = u - p.full_tiles;
    if (NS) {
        const uint32_t t = r / (uint32_t)p.nsplit;
        npart = (int)(r - t * (uint32_t)p.nsplit);
        tile = p.full_tiles + t; kb0 = 0; kb1 = -1; piece = -1;
        return;
    }
    const uint32_t t = r / (uint32_t)p.split;
    piece = (int)(r - t * (uint32_t)p.split);
    tile = p.full_tiles + t;
    kb0 = piece * p.kb_per_piece;
    kb1 = min(p.num_kb, kb0 + p.kb_per_piece);
}

// tile id -> (batch*heads index, m tile, n tile).  Within one matrix, tiles are visited in
// bands of G m-tiles so that the CTAs running at the same time share A and B tiles in L2.
// (32-bit arithmetic: with a single K slice per tile this runs on the critical path of the
// single-lane producer and MMA roles.)  For causal score matrices only the tiles on or below the
// diagonal are enumerated, so every CTA gets the same share of real work.
__device__ __forceinline__ void tile_coords(uint32_t tile, const Params& p, int& bh, int& mi, int& ni) {
    const uint32_t b = tile / p.per_mat;
    const uint32_t t = tile - b * p.per_mat;
    bh = (int)b;
    if (p.causal_compact) {
        int m = 0;
        while (t >= p.causal_prefix[m + 1]) ++m;
        mi = m;
        ni = (int)(t - p.causal_prefix[m]);
        return;
    }
    constexpr uint32_t G = 8;
    const uint32_t band_tiles = G * (uint32_t)p.num_n;
    const uint32_t band = t / band_tiles;
    const uint32_t band_h = min(G, (uint32_t)p.num_m - band * G);
    const uint32_t r = t - band * band_tiles;
    const uint32_t q = r / band_h;
    mi = (int)(band * G + (r - q * band_h));
    ni = (int)q;
}

// Causal attention: a score tile whose first key lies beyond the tile's last query is never
// needed (softmax masks it), and for P.V the K slices beyond the last query hold only zeros.
__device__ __forceinline__ bool tile_skipped(const Params& p, int mi, int ni, int tile_m, int block_n) {
    return p.causal && !p.b_is_kn && (int64_t)ni * block_n > (int64_t)(mi + 1) * tile_m - 1;
}
__device__ __forceinline__ int tile_num_kb(const Params& p, int mi, int tile_m) {
    if (p.causal && p.b_is_kn) return min(p.num_kb, (int)(((int64_t)(mi + 1) * tile_m + BLOCK_K - 1) / BLOCK_K));
    return p.num_kb;
}

// ------------------------------------------------------------------------------------
// Epilogue of one 128 x BLOCK_N accumulator slot: Eq. 2 and the output conversions.
// Called by the 128 epilogue threads; thread = one accumulator row (TMEM lane).
// Output leaves through shared memory: each warp stages 32 rows x 128 bytes (128B swizzle,
// conflict-free 16-byte writes) and one lane issues a TMA store, which also clips the M and N
// tails.  If C is not 16-byte aligned the rows are written directly instead.
// ------------------------------------------------------------------------------------
// FIX: this CTA arrived last for a K-split tile: the other pieces' partial sums (fix_count slots,
// fix_stride ints apart, fix_base already at this thread's row) are added to the accumulators first.
template <int BLOCK_N, bool FIX = false, bool EW8 = false, bool PLAIN16 = false>
__device__ __forceinline__ void epilogue_slot(const Params& p, const CUtensorMap* tmap_c, uint8_t* stg,
                                              uint32_t taddr, int64_t row, int row0_warp, int64_t col0, int b,
                                              int h, int64_t c_off, float xs, const float* s_wscale,
                                              const float* s_bias, const float* s_requant, int lane,
                                              int cc_begin, int cc_end, const int32_t* fix_base = nullptr,
                                              int fix_count = 0, int fix_mine = 0, size_t fix_stride = 0) {
    // PLAIN16: the instantiation for the plain linear layer -- 16-bit output through staged TMA stores, vector
    // scales / bias, no residual, no row maxima.  The generic body carries every output type and option in one
    // unrolled loop; its code size alone (instruction fetch, 255 registers) made a slot take 11 000 cycles
    // where this one takes under 7 000.
    const int out_dt = PLAIN16 ? (p.out_dt == SQ_F16 ? (int)SQ_F16 : (int)SQ_BF16) : p.out_dt;
    const bool c_tma = PLAIN16 || p.c_tma;
    const void* const residual = PLAIN16 ? nullptr : p.residual;
    float* const row_absmax_out = PLAIN16 ? nullptr : p.row_absmax_out;
    const bool row_ok = row < p.M;
    float row_max = 0.0f;
    // 32-column chunks per 128-byte staging row: 1 (int32), 2 (fp16/bf16), 4 (int8)
    const int chunks_per_store = out_dt == SQ_I32 ? 1 : (out_dt == SQ_I8 ? 4 : 2);
    const int pieces = 8 / chunks_per_store;  // 16-byte pieces one chunk contributes to the row
    int cc_coord[4] = {0, 0, 0, 0};
    cc_coord[p.c_slot_row] = row0_warp; cc_coord[p.c_slot_head] = h; cc_coord[p.c_slot_batch] = b;
    const bool scalar_scale = !PLAIN16 && p.w_scale == nullptr && p.bias == nullptr;  // attention BMMs: y = acc * alpha
#pragma unroll 1
    for (int cc = cc_begin; cc < cc_end; ++cc) {
        uint32_t r[32];
        tmem_ld32(taddr + cc * 32, r);  // warp-collective: executed by every lane
        tmem_ld_wait();
        if (FIX) {
            for (int o = 0; o < fix_count; ++o) {
                if (o == fix_mine) continue;
                // slot layout [4-column group][row][4]: a thread's 16 bytes, a warp's 512 contiguous bytes
                const int4* src = reinterpret_cast<const int4*>(fix_base + (size_t)o * fix_stride) + (size_t)(cc * 8) * BLOCK_M;
                int4 t[8];
#pragma unroll
                for (int v = 0; v < 8; ++v) t[v] = __ldcg(src + (size_t)v * BLOCK_M);
#pragma unroll
                for (int v = 0; v < 8; ++v) {
                    r[4 * v] += (uint32_t)t[v].x; r[4 * v + 1] += (uint32_t)t[v].y;
                    r[4 * v + 2] += (uint32_t)t[v].z; r[4 * v + 3] += (uint32_t)t[v].w;
                }
            }
        }
        const int64_t ncols = p.N - (col0 + cc * 32);  // valid columns in this chunk
        // ---- Eq. 2 on the chunk; w[] receives the packed output words ----
        uint32_t w[32];
        int nwords;
        if (out_dt == SQ_I32) {
#pragma unroll
            for (int j = 0; j < 32; ++j) w[j] = r[j];
            nwords = 32;
        } else {
            float y[32];
            if (scalar_scale) {
#pragma unroll
                for (int j = 0; j < 32; ++j) {
                    float v = __fmul_rn(__int2float_rn((int32_t)r[j]), xs);  // == fma(acc, xs * 1, 0)
                    if (p.relu) v = fmaxf(v, 0.0f);
                    y[j] = v;
                }
            } else {
#pragma unroll
                for (int j = 0; j < 32; ++j) {
                    const float sc = __fmul_rn(xs, s_wscale[cc * 32 + j]);
                    float v = __fmaf_rn(__int2float_rn((int32_t)r[j]), sc, s_bias[cc * 32 + j]);
                    if (p.relu) v = fmaxf(v, 0.0f);
                    y[j] = v;
                }
            }
            if (row_absmax_out) {
#pragma unroll
                for (int j = 0; j < 32; ++j)
                    if (j < ncols) row_max = fmaxf(row_max, fabsf(y[j]));
            }
            if (residual && !c_tma) {
                // the block's residual connection: round y to the output type first, then add the
                // residual element in fp32 (the final rounding below is the 16-bit add's rounding)
                const uint4* rrow = reinterpret_cast<const uint4*>(
                    static_cast<const uint16_t*>(residual) + (row_ok ? row : 0) * p.ld_res + col0 + cc * 32);
#pragma unroll
                for (int v = 0; v < 4; ++v) {
                    if (row_ok && 8 * v < ncols) {  // N is a multiple of 8: whole vectors only
                        const uint4 rv = __ldg(rrow + v);
                        float rf[8];
                        if (out_dt == SQ_BF16) {
                            unpack8<__nv_bfloat16>(rv, rf);
#pragma unroll
                            for (int k = 0; k < 8; ++k)
                                y[8 * v + k] = __bfloat162float(__float2bfloat16_rn(y[8 * v + k])) + rf[k];
                        } else {
                            unpack8<__half>(rv, rf);
#pragma unroll
                            for (int k = 0; k < 8; ++k)
                                y[8 * v + k] = __half2float(__float2half_rn(y[8 * v + k])) + rf[k];
                        }
                    }
                }
            }
            if (out_dt == SQ_I8) {
#pragma unroll
                for (int v = 0; v < 8; ++v)
                    w[v] = pack4(quant_code(y[4 * v], s_requant[cc * 32 + 4 * v]),
                                 quant_code(y[4 * v + 1], s_requant[cc * 32 + 4 * v + 1]),
                                 quant_code(y[4 * v + 2], s_requant[cc * 32 + 4 * v + 2]),
                                 quant_code(y[4 * v + 3], s_requant[cc * 32 + 4 * v + 3]));
                nwords = 8;
            } else if (out_dt == SQ_BF16) {
#pragma unroll
                for (int v = 0; v < 16; ++v) {
                    __nv_bfloat162 t = __halves2bfloat162(__float2bfloat16_rn(y[2 * v]), __float2bfloat16_rn(y[2 * v + 1]));
                    w[v] = *reinterpret_cast<uint32_t*>(&t);
                }
                nwords = 16;
            } else {
#pragma unroll
                for (int v = 0; v < 16; ++v) {
                    __half2 t = __halves2half2(__float2half_rn(y[2 * v]), __float2half_rn(y[2 * v + 1]));
                    w[v] = *reinterpret_cast<uint32_t*>(&t);
                }
                nwords = 16;
            }
        }
        if (c_tma) {
            // ---- staged TMA store: lane = row of the 32 x 128-byte staging tile ----
            const int sub = cc % chunks_per_store;
            uint8_t* buf = stg;
            if (sub == 0) {  // the previous store must have finished READING the staging tile
                if (lane == 0) tma_store_wait_read();
                __syncwarp();
            }
            uint8_t* srow = buf + lane * 128;
#pragma unroll
            for (int v = 0; v < 8; ++v) {
                if (v < pieces) {
                    const int j = sub * pieces + v;  // 16-byte piece index inside the 128-byte row
                    *reinterpret_cast<uint4*>(srow + ((j ^ (lane & 7)) << 4)) =
                        make_uint4(w[4 * v], w[4 * v + 1], w[4 * v + 2], w[4 * v + 3]);
                }
            }
            if (sub == chunks_per_store - 1) {
                const int64_t gcol = col0 + (int64_t)(cc - sub) * 32;  // first column of the staged group
                if (residual) {
                    // The residual connection, on the staged tile (32 rows x 64 rounded outputs): the
                    // warp walks it in the layout of the global rows -- 8 lanes per row, 16 bytes per
                    // lane -- so that the residual arrives in whole 128-byte lines, adds in fp32 and
                    // rounds again (the 16-bit add's rounding).
                    __syncwarp();
                    const int piece_c = lane & 7;
                    const int64_t rcol = gcol + piece_c * 8;
                    constexpr int RB = EW8 ? 4 : 8;  // loads in flight per batch (register budget)
#pragma unroll 1
                    for (int i0 = 0; i0 < 8; i0 += RB) {
                    uint4 rv[RB];
#pragma unroll
                    for (int i = 0; i < RB; ++i) {
                        const int64_t rr = (int64_t)row0_warp + 4 * (i0 + i) + (lane >> 3);
                        rv[i] = (rr < p.M && rcol < p.N)  // N is a multiple of 8: whole vectors only
                                    ? __ldg(reinterpret_cast<const uint4*>(static_cast<const uint16_t*>(residual) +
                                                                           rr * p.ld_res + rcol))
                                    : make_uint4(0u, 0u, 0u, 0u);
                    }
#pragma unroll
                    for (int i = 0; i < RB; ++i) {
                        const int r = 4 * (i0 + i) + (lane >> 3);
                        uint4* cell = reinterpret_cast<uint4*>(buf + r * 128 + ((piece_c ^ (r & 7)) << 4));
                        float a[8], b[8];
                        uint4 o;
                        if (out_dt == SQ_BF16) {
                            unpack8<__nv_bfloat16>(*cell, a);
                            unpack8<__nv_bfloat16>(rv[i], b);
                            __nv_bfloat162 t0 = __halves2bfloat162(__float2bfloat16_rn(a[0] + b[0]), __float2bfloat16_rn(a[1] + b[1]));
                            __nv_bfloat162 t1 = __halves2bfloat162(__float2bfloat16_rn(a[2] + b[2]), __float2bfloat16_rn(a[3] + b[3]));
                            __nv_bfloat162 t2 = __halves2bfloat162(__float2bfloat16_rn(a[4] + b[4]), __float2bfloat16_rn(a[5] + b[5]));
                            __nv_bfloat162 t3 = __halves2bfloat162(__float2bfloat16_rn(a[6] + b[6]), __float2bfloat16_rn(a[7] + b[7]));
                            o = make_uint4(*reinterpret_cast<uint32_t*>(&t0), *reinterpret_cast<uint32_t*>(&t1),
                                           *reinterpret_cast<uint32_t*>(&t2), *reinterpret_cast<uint32_t*>(&t3));
                        } else {
                            unpack8<__half>(*cell, a);
                            unpack8<__half>(rv[i], b);
                            __half2 t0 = __halves2half2(__float2half_rn(a[0] + b[0]), __float2half_rn(a[1] + b[1]));
                            __half2 t1 = __halves2half2(__float2half_rn(a[2] + b[2]), __float2half_rn(a[3] + b[3]));
                            __half2 t2 = __halves2half2(__float2half_rn(a[4] + b[4]), __float2half_rn(a[5] + b[5]));
                            __half2 t3 = __halves2half2(__float2half_rn(a[6] + b[6]), __float2half_rn(a[7] + b[7]));
                            o = make_uint4(*reinterpret_cast<uint32_t*>(&t0), *reinterpret_cast<uint32_t*>(&t1),
                                           *reinterpret_cast<uint32_t*>(&t2), *reinterpret_cast<uint32_t*>(&t3));
                        }
                        *cell = o;
                    }
                    }
                }
                asm volatile("fence.proxy.async.shared::cta;" ::: "memory");  // generic writes -> async proxy
                __syncwarp();
#ifndef SQ_GEMM_ISSUE_ONLY
                if (lane == 0 && gcol < p.N && row0_warp < p.M) {
                    cc_coord[0] = (int)gcol;
                    tma_store_4d(tmap_c, buf, cc_coord[0], cc_coord[1], cc_coord[2], cc_coord[3]);
                }
#endif
            }
            continue;
        }
        // ---- direct stores (unaligned C) ----
        if (!row_ok || ncols <= 0) continue;
        const bool full = ncols >= 32;
        if (out_dt == SQ_I32) {
            int32_t* out = static_cast<int32_t*>(p.C) + c_off + cc * 32;
#pragma unroll
            for (int j = 0; j < 32; ++j)
                if (full || j < ncols) out[j] = (int32_t)w[j];
        } else if (out_dt == SQ_I8) {
            int8_t* out = static_cast<int8_t*>(p.C) + c_off + cc * 32;
#pragma unroll
            for (int j = 0; j < 32; ++j)
                if (full || j < ncols) out[j] = (int8_t)((w[j >> 2] >> (8 * (j & 3))) & 0xff);
        } else {
            uint16_t* out = static_cast<uint16_t*>(p.C) + c_off + cc * 32;
#pragma unroll
            for (int j = 0; j < 32; ++j)
                if (full || j < ncols) out[j] = (uint16_t)((w[j >> 1] >> (16 * (j & 1))) & 0xffff);
        }
        (void)nwords;
    }
    if (row_absmax_out && row_ok) atomic_max_nonneg(row_absmax_out + row, row_max);
}

// ------------------------------------------------------------------------------------
// The kernel
// ------------------------------------------------------------------------------------
template <int BLOCK_N, int CG, int EW, bool NS = false, bool PLAIN16 = false>
__global__ void __launch_bounds__(EW * 32 + 64, 1)
gemm_i8_kernel(const __grid_constant__ CUtensorMap tmap_a, const __grid_constant__ CUtensorMap tmap_b,
               const __grid_constant__ CUtensorMap tmap_c, const __grid_constant__ CUtensorMap tmap_bp, const Params p) {
    using C = Cfg<BLOCK_N, CG, EW>;
    extern __shared__ uint8_t smem_raw[];
    // identical layout in both CTAs of a pair (the MMA addresses both with one descriptor)
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
    uint8_t* stage_base = smem;
    uint8_t* staging = smem + C::STAGES * C::STAGE_BYTES;  // 1024-byte aligned: swizzle pattern matches TMA's
    float* epi_f = reinterpret_cast<float*>(staging + C::STAGING_BYTES);
    uint64_t* full_bar = reinterpret_cast<uint64_t*>(reinterpret_cast<uint8_t*>(epi_f) + C::EPI_BYTES);
    uint64_t* empty_bar = full_bar + C::STAGES;
    uint64_t* tmem_full = empty_bar + C::STAGES;
    uint64_t* tmem_empty = tmem_full + 2;
    uint32_t* tmem_holder = reinterpret_cast<uint32_t*>(tmem_empty + 2);
    volatile uint32_t* abort_flag = tmem_holder + 1;
    volatile uint32_t* epi_go = tmem_holder + 2;
    volatile uint32_t* epi_last = tmem_holder + 3;

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int rank = CG == 1 ? 0 : (int)cluster_ctarank();  // 0 = even CTA: issues the MMAs
    const uint32_t first_tile = blockIdx.x / CG, tile_step = gridDim.x / CG;

    if (threadIdx.x == EW * 32) {
        asm volatile("prefetch.tensormap [%0];" ::"l"(&tmap_a) : "memory");
        asm volatile("prefetch.tensormap [%0];" ::"l"(&tmap_b) : "memory");
        if (p.c_tma) asm volatile("prefetch.tensormap [%0];" ::"l"(&tmap_c) : "memory");
        for (int s = 0; s < C::STAGES; ++s) {
            mbar_init(full_bar + s, 1);   // the even CTA's arrive.expect_tx
            mbar_init(empty_bar + s, 1);  // one tcgen05.commit
        }
        for (int s = 0; s < 2; ++s) {
            mbar_init(tmem_full + s, 1);
            mbar_init(tmem_empty + s, C::EPI_THREADS * CG);  // epilogue threads of the whole group
        }
        *abort_flag = 0u;
        *epi_go = 0u;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    if (warp == EW + 1) tmem_alloc<CG>(tmem_holder, C::TMEM_COLS);  // whole warp (in both CTAs of a pair)
    tcgen05_fence_before();
    if (CG == 1) __syncthreads(); else cluster_sync_all();  // peers' barriers are live before any remote signal
    tcgen05_fence_after();
    const uint32_t tmem_base = *tmem_holder;
    pdl_wait();               // set-up overlapped the previous kernel's tail; its outputs are visible from here on
    pdl_launch_dependents();

    if (warp == EW) {
        // ============================ TMA producer ============================
        if (lane == 0) {
            int stage = 0;
            uint32_t phase = 0;
            bool ok = true;
            const uint64_t keep_a = l2_policy_evict_last(), stream_b = l2_policy_evict_first();
            for (uint32_t u = first_tile; ok && u < p.total_units; u += tile_step) {
                uint32_t tile;
                int kb0, kb1, piece, npart;
                unit_of<NS>(u, p, tile, kb0, kb1, piece, npart);
                int bh, mi, ni;
                tile_coords(tile, p, bh, mi, ni);
                if (tile_skipped(p, mi, ni, BLOCK_M * CG, BLOCK_N)) continue;
                if (piece < 0) kb1 = tile_num_kb(p, mi, BLOCK_M * CG);
                const int b = bh / p.heads, h = bh - b * p.heads;
                int ca[4] = {0, 0, 0, 0}, cb[4] = {0, 0, 0, 0};
                ca[p.a_slot_row] = (mi * CG + rank) * BLOCK_M; ca[p.a_slot_head] = h; ca[p.a_slot_batch] = b;
                cb[p.b_slot_head] = h; cb[p.b_slot_batch] = b;
                // this CTA's share of the B tile (of the column part, whose own map has a smaller box)
                const int part_rows = (NS && npart >= 0) ? C::B_ROWS / p.nsplit : C::B_ROWS;
                const int b_row0 = ni * BLOCK_N + ((NS && npart >= 0) ? npart * (BLOCK_N / p.nsplit) : 0) + rank * part_rows;
                const CUtensorMap* mapb = (NS && npart >= 0) ? &tmap_bp : &tmap_b;
                const uint32_t stage_tx = (uint32_t)(C::A_BYTES + part_rows * BLOCK_K) * CG;
                for (int kb = kb0; kb < kb1; ++kb) {
                    if (!(ok = mbar_wait(empty_bar + stage, phase ^ 1u, abort_flag, p.status, 1))) break;
                    uint8_t* sa = stage_base + stage * C::STAGE_BYTES;
                    uint8_t* sb = sa + C::A_BYTES;
#ifdef SQ_GEMM_ISSUE_ONLY
                    // Ceiling build (python -m paper_2211_10438_b200.build --issue-only): no operand is
                    // loaded and no result stored, the MMAs run on whatever shared memory holds -- what the
                    // tensor pipe sustains when nothing else limits it.  Results are meaningless.
                    if (rank == 0) mbar_arrive(full_bar + stage);
                    if (++stage == C::STAGES) { stage = 0; phase ^= 1u; }
                    continue;
#endif
                    if (rank == 0) mbar_expect_tx(full_bar + stage, stage_tx);
                    ca[0] = kb * BLOCK_K;
                    if (p.l2_hints) {  // (plain GEMMs only: B is stored [N, K])
                        cb[0] = kb * BLOCK_K;
                        cb[p.b_slot_row] = b_row0;
                        tma_load_4d_hint<CG>(sa, &tmap_a, full_bar + stage, ca[0], ca[1], ca[2], ca[3], keep_a);
                        tma_load_4d_hint<CG>(sb, mapb, full_bar + stage, cb[0], cb[1], cb[2], cb[3], stream_b);
                        if (++stage == C::STAGES) { stage = 0; phase ^= 1u; }
                        continue;
                    }
                    tma_load_4d<CG>(sa, &tmap_a, full_bar + stage, ca[0], ca[1], ca[2], ca[3]);
                    if (p.b_is_kn) {  // B stored [K, N]: x walks N, the row slot walks K
                        cb[0] = b_row0;
                        cb[p.b_slot_row] = kb * BLOCK_K;
                    } else {
                        cb[0] = kb * BLOCK_K;
                        cb[p.b_slot_row] = b_row0;
                    }
                    tma_load_4d<CG>(sb, mapb, full_bar + stage, cb[0], cb[1], cb[2], cb[3]);
                    if (++stage == C::STAGES) { stage = 0; phase ^= 1u; }
                }
            }
        }
    } else if (warp == EW + 1) {
        // ============================ MMA issuer (even CTA only) ==============
        // The WHOLE warp walks the units and waits on the barriers, converged; one elected lane issues the MMAs
        // and commits.  Everything the MMA instruction takes is then warp-uniform to the compiler (under a
        // `lane == 0` branch it is not, and every operand is first moved to a uniform register, lane by lane).
        if (rank == 0) {
            const uint32_t idesc = make_idesc(BLOCK_M * CG, BLOCK_N, p.b_is_kn);
            // The loop over the K blocks takes about as long as the tensor pipe needs for them (four MMAs
            // of 128 cycles): it is kept short -- descriptors as running low words, barriers by their
            // shared-memory addresses, the slow path of a wait out of line -- so that the warp gets ahead of
            // the pipe and the epilogue warps' instructions, which share its scheduler, cannot hold it up.
            constexpr uint32_t kStage16 = (uint32_t)C::STAGE_BYTES >> 4;
            const uint32_t a_lo0 = smem_desc_lo(smem_u32(stage_base), 16);
            const uint32_t b_lo0 = smem_desc_lo(smem_u32(stage_base) + (uint32_t)C::A_BYTES, p.b_is_kn ? 16384u : 16u);
            // descriptor step between consecutive K=32 slices inside a stage (in 16-byte units)
            const uint32_t a_k16 = (uint32_t)UMMA_K >> 4;
            const uint32_t b_k16 = (p.b_is_kn ? (uint32_t)(UMMA_K * 128) : (uint32_t)UMMA_K) >> 4;
            const uint32_t full0 = smem_u32(full_bar), empty0 = smem_u32(empty_bar);
            const uint32_t tmem_full0 = smem_u32(tmem_full), tmem_empty0 = smem_u32(tmem_empty);
            int stage = 0;
            uint32_t phase = 0;
            int slot = 0;
            uint32_t slot_phase = 0;
            bool ok = true;
#ifdef SQ_GEMM_TRACE
            int trace_tile = 0;
            long long trace_prev_end = clock64(), trace_first = 0;
            unsigned long long trace_first_ns = 0;
#endif
            for (uint32_t u = first_tile; ok && u < p.total_units; u += tile_step) {
                uint32_t tile;
                int kb0, kb1, piece, npart;
                unit_of<NS>(u, p, tile, kb0, kb1, piece, npart);
                // This lane is never more than about one MMA ahead of the tensor pipe: whatever it computes
                // between two tiles is time the pipe idles.  A tile's coordinates (three dependent integer
                // divisions, several hundred cycles) matter to this role only under a causal mask.
                if (p.causal) {
                    int bh, mi, ni;
                    tile_coords(tile, p, bh, mi, ni);
                    if (tile_skipped(p, mi, ni, BLOCK_M * CG, BLOCK_N)) continue;
                    if (piece < 0) kb1 = tile_num_kb(p, mi, BLOCK_M * CG);
                } else if (piece < 0) {
                    kb1 = p.num_kb;
                }
                const uint32_t idesc_u = (NS && npart >= 0) ? make_idesc(BLOCK_M * CG, BLOCK_N / p.nsplit, p.b_is_kn) : idesc;
#ifdef SQ_GEMM_TRACE
                const long long trace_decoded = clock64();
#endif
                if (!(ok = mbar_wait_warp(tmem_empty + slot, tmem_empty0 + (uint32_t)slot * 8u, slot_phase ^ 1u, abort_flag,
                                          p.status, 2)))
                    break;
                tcgen05_fence_after();
                const uint32_t d_tmem = tmem_base + (uint32_t)(slot * C::SLOT_COLS);
                uint32_t accumulate = 0u;  // the tile's first MMA overwrites the slot
#ifdef SQ_GEMM_TRACE
                const long long trace_start = clock64();
                if (trace_tile == 0) { trace_first = trace_start; trace_first_ns = global_timer_ns(); }
#endif
                for (int kb = kb0; kb < kb1; ++kb) {
                    if (!(ok = mbar_wait_warp(full_bar + stage, full0 + (uint32_t)stage * 8u, phase, abort_flag, p.status, 3)))
                        break;
                    tcgen05_fence_after();
                    const uint32_t a_lo = a_lo0 + (uint32_t)stage * kStage16;
                    const uint32_t b_lo = b_lo0 + (uint32_t)stage * kStage16;
                    if (elect_one()) {
                        umma_i8_lo<CG>(d_tmem, a_lo, b_lo, idesc_u, accumulate);
#pragma unroll
                        for (int k = 1; k < BLOCK_K / UMMA_K; ++k)
                            umma_i8_lo<CG>(d_tmem, a_lo + k * a_k16, b_lo + k * b_k16, idesc_u, 1u);
                        umma_commit_u32<CG>(empty0 + (uint32_t)stage * 8u);  // frees the stage (in both CTAs) once these MMAs retire
                    }
                    accumulate = 1u;
                    if (++stage == C::STAGES) { stage = 0; phase ^= 1u; }
                }
                if (!ok) break;
                if (elect_one()) umma_commit_u32<CG>(tmem_full0 + (uint32_t)slot * 8u);  // accumulator complete -> epilogue (of both CTAs)
#ifdef SQ_GEMM_TRACE
                {
                    const long long trace_end = clock64();
                    if (lane == 0) {
                        if (trace_tile < kGemmTraceTiles) {
                            unsigned long long* tr = g_gemm_trace[blockIdx.x][trace_tile];
                            tr[0] = (unsigned long long)(trace_decoded - trace_prev_end);
                            tr[1] = (unsigned long long)(trace_start - trace_decoded);
                            tr[2] = (unsigned long long)(trace_end - trace_start);
                            tr[3] = (unsigned long long)(kb1 - kb0);
                        }
                        unsigned long long* tr = g_gemm_trace[blockIdx.x][kGemmTraceTiles];
                        tr[0] = (unsigned long long)(trace_end - trace_first);
                        tr[1] = global_timer_ns() - trace_first_ns;
                    }
                    ++trace_tile;
                    trace_prev_end = trace_end;
                }
#endif
                slot ^= 1;
                if (slot == 0) slot_phase ^= 1u;
            }
        }
    } else {
        // ============================ epilogue (warps 0 .. EW-1) ===============
        // warp w reads TMEM lanes 32*(w%4).. (hardware rule) and the column half w/4 of the tile
        float* s_wscale = epi_f;
        float* s_requant = epi_f + BLOCK_N;
        float* s_bias = epi_f + 2 * BLOCK_N;
        const int et = threadIdx.x;
        const int quarter = warp & 3, half = warp >> 2;
        int slot = 0;
        uint32_t slot_phase = 0;
#ifdef SQ_GEMM_TRACE
        int trace_tile = 0;
        long long trace_go = 0;
#endif
        for (uint32_t u = first_tile; u < p.total_units; u += tile_step) {
            uint32_t tile;
            int kb0, kb1, piece, npart;
            unit_of<NS>(u, p, tile, kb0, kb1, piece, npart);
            int bh, mi, ni;
            tile_coords(tile, p, bh, mi, ni);
            if (tile_skipped(p, mi, ni, BLOCK_M * CG, BLOCK_N)) continue;
            const int b = bh / p.heads, h = bh - b * p.heads;
            const int width = (NS && npart >= 0) ? BLOCK_N / p.nsplit : BLOCK_N;  // columns of this unit
            const int64_t col0 = (int64_t)ni * BLOCK_N + ((NS && npart >= 0) ? npart * width : 0);
            // stage this tile's per-column constants
            for (int c = et; c < width; c += C::EPI_THREADS) {
                const int64_t col = col0 + c;
                const bool in = col < p.N;
                float ws = 1.0f, rq = 1.0f, bs = 0.0f;
                if (in) {
                    if (p.w_scale) ws = __ldg(p.w_scale + (p.w_per_col ? col : 0));
                    if (p.bias)
                        bs = p.bias_is_bf16 ? __bfloat162float(static_cast<const __nv_bfloat16*>(p.bias)[col])
                                            : __half2float(static_cast<const __half*>(p.bias)[col]);
                    if (p.requant_mul) rq = __ldg(p.requant_mul + (p.requant_per_col ? col : 0));
                }
                s_wscale[c] = ws; s_bias[c] = bs; s_requant[c] = rq;
            }
            if (!PLAIN16 && p.residual) {
                // pull this thread's row of the residual tile into L2 while the tile's MMAs still run:
                // under a saturated memory system a demand load in the epilogue waits microseconds
                const int64_t prow = ((int64_t)mi * CG + rank) * BLOCK_M + quarter * 32 + lane;
                if (prow < p.M) {
                    const char* base = reinterpret_cast<const char*>(static_cast<const uint16_t*>(p.residual) + prow * p.ld_res + col0);
                    const int64_t bytes = 2 * min((int64_t)width, p.N - col0);
                    for (int64_t off = half * 128; off < bytes; off += (EW == 8 ? 256 : 128))
                        asm volatile("prefetch.global.L2 [%0];" ::"l"(base + off));
                }
            }
            // this thread's row and its activation step: requested while the tile's MMAs still run (read behind the
            // wait, the load is a dependent trip to L2 in every tile's epilogue)
            const int64_t row = ((int64_t)mi * CG + rank) * BLOCK_M + quarter * 32 + lane;
            float xs = p.alpha;
            if (p.x_scale) xs = __ldg(p.x_scale + ((p.x_per_row && row < p.M) ? row : 0));
            if (et == 0)
                *epi_go = mbar_wait(tmem_full + slot, slot_phase, abort_flag, p.status, 4) ? 1u : 0u;
            epi_bar_sync<C::EPI_THREADS>();  // constants staged; outcome of the wait visible to all epilogue threads
            if (*epi_go == 0u) break;
            tcgen05_fence_after();
#ifdef SQ_GEMM_TRACE
            trace_go = clock64();
#endif

            const int64_t c_off = (int64_t)b * p.c_stride_batch + (int64_t)h * p.c_stride_head +
                                  row * p.c_stride_row + col0;
            const uint32_t taddr = tmem_base + ((uint32_t)(quarter * 32) << 16) + (uint32_t)(slot * C::SLOT_COLS);
            const int row0_warp = (mi * CG + rank) * BLOCK_M + quarter * 32;
            // split the tile's 32-column chunks between the two warps of this lane quarter, in whole
            // store groups (a staged TMA store covers 128 bytes of a row = 1, 2 or 4 chunks)
            const int cps = PLAIN16 ? 2 : (p.out_dt == SQ_I32 ? 1 : (p.out_dt == SQ_I8 ? 4 : 2));
            const int groups = (width / 32 + cps - 1) / cps;
            const int g_split = EW == 8 ? (groups + 1) / 2 : groups;
            const int cc_begin = half == 0 ? 0 : g_split * cps;
            const int cc_end = half == 0 ? min(g_split * cps, width / 32) : width / 32;
            if (EW == 8 || piece < 0) {  // (the eight-warp configuration serves short reductions: never split)
                epilogue_slot<BLOCK_N, false, EW == 8, PLAIN16>(p, &tmap_c, staging + warp * (32 * 128), taddr, row, row0_warp, col0, b, h,
                                       c_off, xs, s_wscale, s_bias, s_requant, lane, cc_begin, cc_end);
            } else {
                // K piece of a split tile: park the accumulators, then see who is last
                constexpr size_t kTileInts = (size_t)BLOCK_M * BLOCK_N;
                const uint32_t rem = tile - p.full_tiles;
                // slot layout [4-column group][row of this CTA][4]: a thread stores 16 bytes, a warp 512 contiguous bytes
                int32_t* tile_slots = p.part + ((size_t)rem * p.split * CG + rank) * kTileInts +
                                      (size_t)(quarter * 32 + lane) * 4;  // piece 0, this CTA, this row
                int32_t* mine = tile_slots + (size_t)piece * CG * kTileInts;
                for (int cc = cc_begin; cc < cc_end; ++cc) {
                    uint32_t r[32];
                    tmem_ld32(taddr + cc * 32, r);
                    tmem_ld_wait();
#pragma unroll
                    for (int v = 0; v < 8; ++v)
                        __stcg(reinterpret_cast<int4*>(mine) + (size_t)(cc * 8 + v) * BLOCK_M,
                               make_int4((int)r[4 * v], (int)r[4 * v + 1], (int)r[4 * v + 2], (int)r[4 * v + 3]));
                }
                __threadfence();
                epi_bar_sync<C::EPI_THREADS>();
                if (et == 0)
                    *epi_last = atomicAdd(p.counters + rem * CG + rank, 1u) == (uint32_t)(p.split - 1) ? 1u : 0u;
                epi_bar_sync<C::EPI_THREADS>();
                if (*epi_last != 0u) {
                    __threadfence();
                    epilogue_slot<BLOCK_N, true, false, PLAIN16>(p, &tmap_c, staging + warp * (32 * 128), taddr, row, row0_warp, col0, b,
                                                 h, c_off, xs, s_wscale, s_bias, s_requant, lane, cc_begin, cc_end,
                                                 tile_slots, p.split, piece, (size_t)CG * kTileInts);
                    if (et == 0) p.counters[rem * CG + rank] = 0u;  // hand the counter back zeroed
                }
            }

#ifdef SQ_GEMM_TRACE
            if (threadIdx.x == 0 && trace_tile == 3) g_gemm_trace[blockIdx.x][kGemmTraceTiles][2] = (unsigned long long)(clock64() - trace_go);
            ++trace_tile;
#endif
            // accumulator slot drained: hand it back to the MMA warp (in the even CTA)
            tcgen05_fence_before();
            if (CG == 1) mbar_arrive(tmem_empty + slot); else mbar_arrive_even_cta(tmem_empty + slot);
            slot ^= 1;
            if (slot == 0) slot_phase ^= 1u;
            epi_bar_sync<C::EPI_THREADS>();  // nobody still reads the staged constants when the next tile overwrites them
        }
        if (p.c_tma && lane == 0) tma_store_wait_all();  // this warp's stores have landed before the CTA exits
    }

    // ---------------------------------- teardown ------------------------------------
    __syncwarp();
    if (*abort_flag) __nanosleep(1000000);  // let copies / MMAs in flight land before freeing
    tcgen05_fence_before();
    if (CG == 1) __syncthreads(); else cluster_sync_all();  // the peer may still signal this CTA's barriers
    if (warp == EW + 1) {
        tcgen05_fence_after();
        tmem_dealloc<CG>(tmem_base, C::TMEM_COLS);
    }
}

// ------------------------------------------------------------------------------------
// Host side: tensor maps + launch
// ------------------------------------------------------------------------------------
// K split of the last wave.  With T tiles on G resident CTA groups the last R = T mod G tiles keep
// only part of the machine busy.  Cutting each of them into s K pieces spreads them over up to
// R * s groups, at the price of parking and re-reading INT32 partial sums (128 KB per CTA and
// piece, which a single SM reads at only ~50 GB/s).  Measured on B200: it pays for long
// reductions only (a 256 x 256 tile of K = 20480 takes 66 us: 156 -> 144 us on 2048 x 5120 x 20480,
// 291 -> 271 us on 2048 x 7168 x 28672), loses for K = 5120 (tile 16 us) at every s, and loses badly
// when the pieces need more than one round.  Hence: K >= 12288, s in {4, 3, 2} with R * s <= G
// and at least 16 K blocks per piece; and, when all tiles together fill at most half of the
// groups, every tile is cut into up to 8 pieces of at least 8 K blocks.
// Also tried for K < 12288: equal contiguous ranges of (tile, K block) pairs per group ("stream-K",
// at most two owners per tile).  Bit-exact, but slower wherever it applied (2048 x 21504 x 7168:
// 204 -> 275 us; 256 x 21504 x 7168: 49 -> 54 us): groups that run side by side then work on tiles
// far apart in the visiting order, so the weight tiles they stream no longer coincide in L2 (74
// pairs x 1.8 MB live at once), and with few tokens a partly filled wave already runs faster per
// tile because one SM's copy rate, not HBM, is the limit there.
struct SplitPlan { uint32_t full; int split; int kb_per_piece; };
inline SplitPlan plan_split(int64_t total_tiles, int num_kb, int groups, int64_t K, int tile_m, int tile_n) {
    SplitPlan pl{(uint32_t)total_tiles, 1, num_kb};
    (void)tile_m; (void)tile_n;
    if (groups <= 0 || total_tiles <= 0) return pl;
    if (K < 12288) return pl;
    if (2 * total_tiles <= groups) {
        // a single wave that fills at most half of the machine (few tokens against a narrow weight):
        // every tile is cut (7168 x 28672, 128 tokens: 92 -> 60 us with 128 x 256 tiles)
        for (int s = (int)std::min<int64_t>(8, groups / total_tiles); s >= 2; --s) {
            const int per = (num_kb + s - 1) / s;
            if (per < 8 || (num_kb + per - 1) / per != s) continue;
            pl.split = s;
            pl.kb_per_piece = per;
            pl.full = 0;
            return pl;
        }
        return pl;
    }
    const int64_t R = total_tiles % groups;
    if (R == 0) return pl;
    for (int s = 4; s >= 2; --s) {
        const int per = (num_kb + s - 1) / s;
        if (R * s > groups || per < 16 || (num_kb + per - 1) / per != s) continue;
        pl.split = s;
        pl.kb_per_piece = per;
        pl.full = (uint32_t)(total_tiles - R);
        break;
    }
    return pl;
}
template <int BLOCK_N, int CG>
inline size_t split_workspace_bytes(const SplitPlan& pl, int64_t total_tiles) {
    if (pl.split <= 1) return kWsHeader;
    return kWsHeader + kDecCounterBytes +
           (size_t)(total_tiles - pl.full) * pl.split * CG * BLOCK_M * BLOCK_N * sizeof(int32_t);
}

template <int BLOCK_N, int CG, int EW>
sq_status launch_ew(const GemmArgs& a, cudaStream_t st) {
    using C = Cfg<BLOCK_N, CG, EW>;
    Params p;
    p.M = a.M; p.N = a.N; p.K = a.K;
    p.heads = (int)a.heads; p.batch = (int)a.batch;
    p.num_m = (int)((a.M + BLOCK_M * CG - 1) / (BLOCK_M * CG));
    p.num_n = (int)((a.N + BLOCK_N - 1) / BLOCK_N);
    // tiles per matrix; for causal score matrices only those on or below the diagonal
    p.causal_compact = 0;
    p.per_mat = (uint32_t)p.num_m * (uint32_t)p.num_n;
    if (a.causal && !a.b_is_kn && p.num_m <= 32) {
        p.causal_compact = 1;
        uint32_t acc = 0;
        for (int mi = 0; mi < p.num_m; ++mi) {
            p.causal_prefix[mi] = acc;
            const int64_t last_query = (int64_t)(mi + 1) * BLOCK_M * CG - 1;
            acc += (uint32_t)std::min<int64_t>(p.num_n, last_query / BLOCK_N + 1);
        }
        p.causal_prefix[p.num_m] = acc;
        p.per_mat = acc;
    }
    const int64_t total = (int64_t)p.per_mat * a.heads * a.batch;
    if (total >= (int64_t)1 << 31) return SQ_ERR_UNSUPPORTED;
    p.total_tiles = (uint32_t)total;
    p.num_kb = (int)((a.K + BLOCK_K - 1) / BLOCK_K);
    p.b_is_kn = a.b_is_kn;
    p.causal = a.causal;
    CUtensorMap ma, mb;
    if (!make_map(&ma, a.A, 1, a.K, a.M, a.heads, a.batch, a.strideA[2], a.strideA[1], a.strideA[0], BLOCK_K,
                  BLOCK_M, &p.a_slot_row, &p.a_slot_head, &p.a_slot_batch))
        return SQ_ERR_CUDA;
    const bool okb =
        a.b_is_kn ? make_map(&mb, a.B, 1, a.N, a.K, a.heads, a.batch, a.strideB[2], a.strideB[1], a.strideB[0],
                             C::B_ROWS, BLOCK_K, &p.b_slot_row, &p.b_slot_head, &p.b_slot_batch)
                  : make_map(&mb, a.B, 1, a.K, a.N, a.heads, a.batch, a.strideB[2], a.strideB[1], a.strideB[0],
                             BLOCK_K, C::B_ROWS, &p.b_slot_row, &p.b_slot_head, &p.b_slot_batch);
    if (!okb) return SQ_ERR_CUDA;
    p.x_scale = a.x_scale; p.x_per_row = a.x_per_row;
    p.w_scale = a.w_scale; p.w_per_col = a.w_per_col;
    p.alpha = a.alpha;
    p.bias = a.bias; p.bias_is_bf16 = a.bias_dt == SQ_BF16;
    p.relu = a.relu;
    p.requant_mul = a.requant_mul; p.requant_per_col = a.requant_per_col;
    p.row_absmax_out = a.row_absmax_out;
    p.residual = a.residual; p.ld_res = a.ld_res;
    p.C = a.C; p.out_dt = (int)a.out_dt;
    p.c_stride_batch = a.strideC[0]; p.c_stride_head = a.strideC[1]; p.c_stride_row = a.strideC[2];
    const int esz = a.out_dt == SQ_I32 ? 4 : (a.out_dt == SQ_I8 ? 1 : 2);
    const int vec_elems = 16 / esz;
    p.c_tma = aligned16(a.C) && a.strideC[0] % vec_elems == 0 && a.strideC[1] % vec_elems == 0 &&
              a.strideC[2] % vec_elems == 0;
    p.c_slot_row = 1; p.c_slot_head = 2; p.c_slot_batch = 3;
    CUtensorMap mc = ma;  // placeholder when C is written directly
    if (p.c_tma && !make_map(&mc, a.C, esz, a.N, a.M, a.heads, a.batch, a.strideC[2], a.strideC[1], a.strideC[0],
                             128 / esz, 32, &p.c_slot_row, &p.c_slot_head, &p.c_slot_batch))
        return SQ_ERR_CUDA;
    p.status = a.status;

    // Variants of the main configuration, each an instantiation of its own so that the others pay nothing for
    // it: the N split of the last wave, and the plain linear layer's epilogue (16-bit output through staged
    // TMA stores, vector scales or bias, no residual, no row maxima).
    constexpr bool kMain = BLOCK_N == 256 && CG == 2 && EW == 4;
    constexpr bool kCanSplitN = kMain;
    const bool plain16 = kMain && (a.out_dt == SQ_F16 || a.out_dt == SQ_BF16) && p.c_tma && a.residual == nullptr &&
                         a.row_absmax_out == nullptr && (a.w_scale != nullptr || a.bias != nullptr);
    static bool attr_set[64] = {false};  // once per device
    int dev = 0;
    SQ_CUDA_OK(cudaGetDevice(&dev));
    if (dev < 0 || dev >= 64 || !attr_set[dev]) {
        SQ_CUDA_OK(cudaFuncSetAttribute(gemm_i8_kernel<BLOCK_N, CG, EW, false, false>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                        C::SMEM_BYTES));
        if (kMain) {
            SQ_CUDA_OK(cudaFuncSetAttribute(gemm_i8_kernel<BLOCK_N, CG, EW, kMain, false>,
                                            cudaFuncAttributeMaxDynamicSharedMemorySize, C::SMEM_BYTES));
            SQ_CUDA_OK(cudaFuncSetAttribute(gemm_i8_kernel<BLOCK_N, CG, EW, false, kMain>,
                                            cudaFuncAttributeMaxDynamicSharedMemorySize, C::SMEM_BYTES));
            SQ_CUDA_OK(cudaFuncSetAttribute(gemm_i8_kernel<BLOCK_N, CG, EW, kMain, kMain>,
                                            cudaFuncAttributeMaxDynamicSharedMemorySize, C::SMEM_BYTES));
        }
        if (dev >= 0 && dev < 64) attr_set[dev] = true;
    }
    // K split of the last wave: plain GEMMs only, and only with the scratch it needs
    p.full_tiles = p.total_tiles; p.total_units = p.total_tiles; p.split = 1; p.kb_per_piece = p.num_kb;
    p.part = nullptr; p.counters = nullptr;
    if (EW == 4 && a.batch == 1 && a.heads == 1 && !a.causal && !a.b_is_kn) {
        const SplitPlan pl = plan_split(p.total_tiles, p.num_kb, sm_count() / CG, a.K, BLOCK_M * CG, BLOCK_N);
        if (pl.split > 1 && (p.total_tiles - pl.full) * CG <= kDecCounterBytes / 4 &&
            a.ws_bytes >= split_workspace_bytes<BLOCK_N, CG>(pl, p.total_tiles)) {
            p.full_tiles = pl.full; p.split = pl.split; p.kb_per_piece = pl.kb_per_piece;
            p.total_units = pl.full + (p.total_tiles - pl.full) * (uint32_t)pl.split;
            char* ws = reinterpret_cast<char*>(a.status);
            p.counters = reinterpret_cast<uint32_t*>(ws + kWsHeader);
            p.part = reinterpret_cast<int32_t*>(ws + kWsHeader + kDecCounterBytes);
        }
    }
    // N split of the last wave: plain GEMMs whose reduction is too short for the K split.  With R tiles left
    // over after the full waves, cutting each into 2 or 4 column parts that still fit ONE round shortens the
    // last wave to a half or a quarter of a tile time; the parts need no exchange, only the A tile again.
    // Measured on B200 (full-range codes, same GPU back to back, split withheld -> taken): 2048 x 15360 x 5120
    // 105.4 -> 103.9 us, 2048 x 21504 x 7168 198.2 -> 195.2, 8192 x 28672 x 7168 1019 -> 1011.
    p.nsplit = 1;
    CUtensorMap mbp = mb;  // placeholder unless the split is taken
    if (kCanSplitN && p.split == 1 && a.batch == 1 && a.heads == 1 && !a.causal && !a.b_is_kn) {
        const int64_t G = sm_count() / CG;
        const int64_t R = (int64_t)p.total_tiles % G;
        const int max_ns = a.out_dt == SQ_I8 ? 2 : 4;  // a staged store row is 128 bytes: a part must fill it
#ifdef SQ_GEMM_NO_NSPLIT  // tuning build (python -m paper_2211_10438_b200.build --no-nsplit): the split withheld, for A/B timing
        const int ns = 1;
        (void)max_ns;
#else
        const int ns = (p.total_tiles > G && R > 0) ? ((4 * R <= G && max_ns >= 4) ? 4 : (2 * R <= G ? 2 : 1)) : 1;
#endif
        if (ns > 1) {
            if (!make_map(&mbp, a.B, 1, a.K, a.N, a.heads, a.batch, a.strideB[2], a.strideB[1], a.strideB[0], BLOCK_K,
                          C::B_ROWS / ns, &p.b_slot_row, &p.b_slot_head, &p.b_slot_batch))
                return SQ_ERR_CUDA;
            p.nsplit = ns;
            p.full_tiles = (uint32_t)(p.total_tiles - R);
            p.total_units = p.full_tiles + (uint32_t)R * (uint32_t)ns;
        }
    }
    // A single band of m-tiles (A is then re-read by every wave, B streamed exactly once), A well inside the 126 MB L2,
    // and a second wave to find it there.  Measured on B200: 2048 x 5120 x 20480 147.1 -> 143.8 us, DRAM reads 217 -> 183 MB
    // (147 MB of operands); with several bands (8192 x 20480 x 20480) the weights come round once per band and the hints cost 1 %.
#ifdef SQ_GEMM_NO_L2_HINTS  // tuning build (-DSQ_GEMM_NO_L2_HINTS)
    p.l2_hints = 0;
    if (false)
#endif
    p.l2_hints = (a.batch == 1 && a.heads == 1 && !a.causal && !a.b_is_kn && a.K >= 8192 && a.M <= 8 * BLOCK_M * CG &&
                  a.M * a.K <= (48LL << 20) && (int64_t)p.total_tiles > sm_count() / CG)
                     ? 1 : 0;
    const int groups = (int)std::min<int64_t>((int64_t)p.total_units, sm_count() / CG);
    const dim3 grid((unsigned)(groups * CG)), block(C::NUM_THREADS);
    if (kMain && p.nsplit > 1 && plain16)
        return launch_pdl(gemm_i8_kernel<BLOCK_N, CG, EW, kMain, kMain>, grid, block, (size_t)C::SMEM_BYTES, st, CG, ma, mb, mc, mbp, p);
    if (kMain && p.nsplit > 1)
        return launch_pdl(gemm_i8_kernel<BLOCK_N, CG, EW, kMain, false>, grid, block, (size_t)C::SMEM_BYTES, st, CG, ma, mb, mc, mbp, p);
    if (kMain && plain16)
        return launch_pdl(gemm_i8_kernel<BLOCK_N, CG, EW, false, kMain>, grid, block, (size_t)C::SMEM_BYTES, st, CG, ma, mb, mc, mbp, p);
    return launch_pdl(gemm_i8_kernel<BLOCK_N, CG, EW, false, false>, grid, block, (size_t)C::SMEM_BYTES, st, CG, ma, mb, mc, mbp, p);
}

// Short reductions (few K slices per tile) are bound by draining the accumulators: give them
// eight epilogue warps; long ones keep four, which leaves the MMA and TMA lanes more issue slots.
template <int BLOCK_N, int CG>
sq_status launch(const GemmArgs& a, cudaStream_t st) {
    return a.K <= 1024 ? launch_ew<BLOCK_N, CG, 8>(a, st) : launch_ew<BLOCK_N, CG, 4>(a, st);
}

}  // namespace

namespace {
// One warp waits on a barrier that never completes; the bounded wait must give up and report.
__global__ void bounded_wait_selftest_kernel(uint32_t* status, uint32_t budget) {
    __shared__ uint64_t bar;
    __shared__ uint32_t abort_flag;
    if (threadIdx.x == 0) {
        tc::mbar_init(&bar, 1);
        abort_flag = 0u;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncthreads();
    if (threadIdx.x == 0) tc::mbar_wait(&bar, 0u, &abort_flag, status, 15u, budget);
    __syncthreads();
}
}  // namespace

sq_status bounded_wait_selftest(uint32_t* status, uint32_t budget, cudaStream_t st) {
    bounded_wait_selftest_kernel<<<1, 32, 0, st>>>(status, budget);
    return launch_status();
}

static bool narrow_single_row_tiles(int64_t N) { return (N + 127) / 128 <= (int64_t)sm_count(); }

// Scratch a plain GEMM of this shape can use for the K split of its last wave (the tile
// configuration follows gemm_i8's dispatch); with less the split is simply not taken.
size_t gemm_workspace_bytes(int64_t M, int64_t N, int64_t K) {
    if (N <= 128 || K <= 1024) return kWsHeader;  // those configurations never split
    const int num_kb = (int)((K + BLOCK_K - 1) / BLOCK_K);
    if (M <= 128) {  // single CTAs, one row of 128 x 128 or 128 x 256 tiles
        if (narrow_single_row_tiles(N)) {
            const int64_t tiles = (N + 127) / 128;
            return split_workspace_bytes<128, 1>(plan_split(tiles, num_kb, sm_count(), K, BLOCK_M, 128), tiles);
        }
        const int64_t tiles = (N + 255) / 256;
        return split_workspace_bytes<256, 1>(plan_split(tiles, num_kb, sm_count(), K, BLOCK_M, 256), tiles);
    }
    const int64_t tiles = ((M + 2 * BLOCK_M - 1) / (2 * BLOCK_M)) * ((N + 255) / 256);
    if (tiles >= (int64_t)1 << 31) return kWsHeader;
    const SplitPlan pl = plan_split(tiles, num_kb, sm_count() / 2, K, 2 * BLOCK_M, 256);
    return split_workspace_bytes<256, 2>(pl, tiles);
}

sq_status gemm_i8(const GemmArgs& a, cudaStream_t st) {
    if (decode_supports(a)) return decode_gemm(a, a.status, a.ws_bytes, st);
    // [K, N]-stored B is limited to one 128-byte swizzle row of N per tile
    if (a.b_is_kn || a.N <= 128) return launch<128, 1>(a, st);
    // Up to 128 tokens every tile is one row of tiles: 128 output channels per tile instead of 256
    // whenever those still fit one wave (N <= 128 * SMs), so that twice as many SMs stream weights
    // (12288 x 12288, 128 tokens: 46 -> 35 us; 15360 x 5120: 22 -> 18 us).
    if (a.M <= 128) return narrow_single_row_tiles(a.N) ? launch<128, 1>(a, st) : launch<256, 1>(a, st);
    // CTA pairs with 256 x 256 tiles.  Narrower pair tiles (192, 128 columns) were measured: they
    // even out the last wave of some shapes but move more operand bytes per MAC and lose overall.
    return launch<256, 2>(a, st);
}

}  // namespace sq

#ifdef SQ_GEMM_TRACE
// [160 CTAs][16 tiles + 1][4] 64-bit words: per tile (index arithmetic, wait for the accumulator slot, K loop:
// SM cycles; K blocks); last row: cycles and nanoseconds from the CTA's first MMA to its last commit, cycles
// epilogue warp 0 took to drain the fourth tile's slot, 0.  Copies the table out and clears it.
extern "C" int sq_debug_gemm_trace(unsigned long long* host_out) {
    const size_t bytes = sizeof(unsigned long long) * 160 * (sq::kGemmTraceTiles + 1) * 4;
    if (cudaMemcpyFromSymbol(host_out, sq::g_gemm_trace, bytes) != cudaSuccess) return 1;
    void* dev = nullptr;
    if (cudaGetSymbolAddress(&dev, sq::g_gemm_trace) != cudaSuccess || cudaMemset(dev, 0, bytes) != cudaSuccess) return 1;
    return 0;
}
#endif
