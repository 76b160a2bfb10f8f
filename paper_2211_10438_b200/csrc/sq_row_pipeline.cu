// Fused LayerNorm + smooth + absmax + INT8 quantise (and the plain quantiser) as a persistent,
// bulk-copy-fed pipeline: the HBM-bound runtime stage in front of every W8A8 GEMM.
//
//   * one CTA per SM, 512 threads (384 for the LayerNorm variants of hidden sizes 7168 and 12288)
//     split into groups of GROUP threads; a group owns one row (token) at a time and walks the
//     rows assigned to it.  A thread holds 80 to 128 values of its row: per-row costs (three
//     reductions, barrier, ring bookkeeping, the scalar statistics) are paid once per thread and
//     row, so few threads per row keep the instruction count per element low;
//   * rows arrive through a ring of shared-memory stages filled by cp.async.bulk (one bulk
//     copy per row, completion on an mbarrier), so the next rows stream in from HBM while
//     the current one is being reduced and quantised;
//   * the folded LayerNorm parameters gamma_hat / beta_hat live on the SM for the whole kernel -- in
//     shared memory as 16-bit values, or (hidden sizes 4096, 7168, 9216, 14336, 20480) as fp32 in
//     tensor memory, which saves unpacking them for every row; a row is unpacked once into
//     registers, so HBM sees 2 bytes in + 1 byte out per element and nothing else;
//   * reductions are warp shuffles + one named barrier each: one for the statistics (per-thread
//     mean and squared deviations merged with the parallel-variance update; rows with a ragged
//     tail take the sum first and the deviations second), one for the absolute maximum.
// Arithmetic is the normative fp32 sequence: n = fma(x, rstd, -(mu*rstd)),
// y = fma(n, gamma_hat, beta_hat), Delta = max(|y|, 1e-5)/127, q = round(y * (1/Delta)).
// The kernel is instruction-issue sensitive (about 12 instructions per element at 3 bytes of
// HBM traffic per element), hence the two-wide fp32 instructions (same rounding per half as the
// scalar ones), the single-FMA rounding, byte-permute packing, vector loads of the reduction
// partials and multiplications by 1/C in the statistics.
// Tried and measured no faster: gamma_hat / beta_hat as 16-BIT values in each thread's own
// tensor-memory lane, which frees their shared memory for a second ring stage at hidden sizes 8192
// to 20480 -- bit-identical output, 0.79 instead of 0.81 of the copy bandwidth at 20480 and 0.82
// instead of 0.87 at 12288, so the bytes in flight are not what limits those shapes (the
// instructions are: the fp32 form above removes two of them per element); 256- and 320-thread CTAs with 128 to 160 values per thread at 20480 (too
// few warps to cover the reductions); 640 threads with 64 values per thread; fp32 copies of
// gamma_hat / beta_hat in shared memory, which take the two unpacks per element out of the inner
// loop but double the bytes every row reads back from shared memory (65536 x 7168: 0.96 -> 0.71).
#include "sq_common.cuh"
#include "sq_bulk.cuh"
#include "sq_kernels.h"
#include "sq_tcgen05.cuh"

namespace sq {

namespace {

constexpr int CTA_THREADS = 512;
#ifdef SQ_LN_NO_TM  // tuning build (-DSQ_LN_NO_TM): LayerNorm parameters stay in shared memory at every hidden size
constexpr bool kLnTensorMemory = false;
#else
constexpr bool kLnTensorMemory = true;
#endif

using namespace bulk;
template <int GROUP, int CTA = CTA_THREADS>
__device__ __forceinline__ void group_sync(int g) {
    if (GROUP == CTA) __syncthreads();
    else asm volatile("bar.sync %0, %1;" ::"r"(g + 1), "n"(GROUP) : "memory");
}
// All GROUP threads get the reduction of v; `red` holds GROUP/32 floats owned by this call site.
template <bool IS_MAX, int GROUP, int CTA = CTA_THREADS>
__device__ __forceinline__ float group_reduce(float v, float* red, int g, int gwarp, int lane) {
    // non-negative floats order like their bit patterns: one redux instruction per level
    v = IS_MAX ? __uint_as_float(__reduce_max_sync(0xffffffffu, __float_as_uint(v))) : warp_sum(v);
    constexpr int NW = GROUP / 32;
    if constexpr (NW == 1) return v;  // one warp per row: every lane already holds the result
    if (lane == 0) red[gwarp] = v;
    group_sync<GROUP, CTA>(g);
    // every thread folds the NW partials in the same order (identical result in all threads);
    // `red` is 16-byte aligned, so the partials come in with vector loads
    constexpr int NWP = (NW + 3) & ~3;
    float p[NWP];
    if constexpr (NW > 2) {
#pragma unroll
        for (int i = 0; i < NWP / 4; ++i) {
            const float4 q = reinterpret_cast<const float4*>(red)[i];
            p[4 * i] = q.x; p[4 * i + 1] = q.y; p[4 * i + 2] = q.z; p[4 * i + 3] = q.w;
        }
    } else {
        const float2 q = *reinterpret_cast<const float2*>(red);
        p[0] = q.x; p[1] = q.y;
    }
    float r = p[0];
#pragma unroll
    for (int i = 1; i < NW; ++i) r = IS_MAX ? fmaxf(r, p[i]) : r + p[i];
    return r;
}

// Mean and sum of squared deviations of a row whose threads all hold the same number of values
// (n_lane each): every thread brings the statistics of its own values, pairs are merged with the
// parallel-variance update (equal counts: mean = (a + b) / 2, M2 = M2a + M2b + (a - b)^2 * n / 2,
// written symmetrically so that both lanes of a pair compute identical bits), warps are merged in
// a fixed order by every thread.  One barrier instead of the two of "mean, then deviations".
template <int GROUP, int CTA>
__device__ __forceinline__ void group_merge_stats(float& mean, float& m2, float n_lane, float* red_mean, float* red_m2,
                                                  int g, int gwarp, int lane) {
    float n = n_lane;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        const float om = __shfl_xor_sync(0xffffffffu, mean, o), o2 = __shfl_xor_sync(0xffffffffu, m2, o);
        const float d = mean - om;
        m2 = (m2 + o2) + (d * d) * (n * 0.5f);
        mean = (mean + om) * 0.5f;
        n += n;
    }
    constexpr int NW = GROUP / 32;
    if constexpr (NW == 1) return;
    if (lane == 0) { red_mean[gwarp] = mean; red_m2[gwarp] = m2; }
    group_sync<GROUP, CTA>(g);
    constexpr int NWP = (NW + 3) & ~3;
    float pm[NWP], p2[NWP];
#pragma unroll
    for (int i = 0; i < NWP / 4; ++i) {
        const float4 a = reinterpret_cast<const float4*>(red_mean)[i], b = reinterpret_cast<const float4*>(red_m2)[i];
        pm[4 * i] = a.x; pm[4 * i + 1] = a.y; pm[4 * i + 2] = a.z; pm[4 * i + 3] = a.w;
        p2[4 * i] = b.x; p2[4 * i + 1] = b.y; p2[4 * i + 2] = b.z; p2[4 * i + 3] = b.w;
    }
    mean = pm[0]; m2 = p2[0];
#pragma unroll
    for (int i = 1; i < NW; ++i) {  // i warps merged so far, one more of the same size
        const float d = pm[i] - mean;
        mean = fmaf(d, 1.0f / (float)(i + 1), mean);
        m2 = (m2 + p2[i]) + (d * d) * (n * ((float)i / (float)(i + 1)));
    }
}

// One thread's bounded wait for a row's bulk copy.  An expiry is recorded in the device status word
// (when the caller gave a workspace to hold one) as SQ_ERR_TIMEOUT | 5 << 8; the group then stops.
__device__ __forceinline__ bool wait_row(uint64_t* bar, uint32_t parity, uint32_t* status,
                                         uint32_t budget = bulk::kWaitCycles) {
    const bool ok = mbar_wait_bounded(bar, parity, budget);
    if (!ok && status != nullptr) atomicCAS(status, 0u, (uint32_t)SQ_ERR_TIMEOUT | (5u << 8));
    return ok;
}

// Self-test of that wait: a barrier nothing will ever complete, a small cycle budget.
__global__ void row_wait_selftest_kernel(uint32_t* status, uint32_t budget) {
    __shared__ uint64_t bar;
    if (threadIdx.x == 0) {
        mbar_init(&bar, 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        wait_row(&bar, 0u, status, budget);
    }
}

// Sixteen 32-bit words per thread to / from tensor memory (lane = thread of the warp's lane quarter).
__device__ __forceinline__ void tm_st16(uint32_t taddr, const uint32_t (&r)[16]) {
    asm volatile(
        "tcgen05.st.sync.aligned.32x32b.x16.b32 [%0], "
        "{%1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, %16};"
        ::"r"(taddr), "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7]), "r"(r[8]),
          "r"(r[9]), "r"(r[10]), "r"(r[11]), "r"(r[12]), "r"(r[13]), "r"(r[14]), "r"(r[15])
        : "memory");
}
__device__ __forceinline__ void tm_ld16(uint32_t taddr, uint32_t (&r)[16]) {
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x16.b32 "
        "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15}, [%16];"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
          "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15])
        : "r"(taddr)
        : "memory");
}
__device__ __forceinline__ void tm_ld8(uint32_t taddr, uint32_t (&r)[8]) {
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x8.b32 {%0, %1, %2, %3, %4, %5, %6, %7}, [%8];"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7])
        : "r"(taddr)
        : "memory");
}
__device__ __forceinline__ void tm_ld_wait8(uint32_t (&r)[8]) {
    asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
#pragma unroll
    for (int i = 0; i < 8; ++i) asm volatile("" : "+r"(r[i]));
}
// The loaded words may be used only behind the wait: route them through an empty statement placed after it.
__device__ __forceinline__ void tm_ld_wait16(uint32_t (&r)[16]) {
    asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
#pragma unroll
    for (int i = 0; i < 16; ++i) asm volatile("" : "+r"(r[i]));
}

// EXACT: the row has exactly GROUP * V vectors, so no per-vector bounds checks are needed.
// TM (LayerNorm, EXACT): the folded parameters do not sit in shared memory as 16-bit values that every row
// unpacks again (two integer instructions per element, a fifth of all the kernel issues) but in TENSOR
// MEMORY as fp32, written once per CTA: a thread's 16 V words (gamma and beta of its V vectors) live in its
// own lane, and the threads of all groups that hold the same columns share them (warps W and W + 4k of
// a lane quarter hold the same columns unless the group has eight warps, which then take two column
// ranges).  The values are the unpacked 16-bit parameters, so the arithmetic is unchanged bit for bit;
// the 4 C bytes of shared memory go to more ring stages.
// MUL (never together with LN): every element is first multiplied by a per-column fp32 factor --
// s_j when weights are folded (Eq. 3), 1/s_j for an activation whose producer cannot absorb it.
// The factors live in shared memory for the CTA's lifetime, in the space LayerNorm's parameters
// would take (4 bytes per column either way).
template <typename T, int GROUP, int V, bool LN, bool EXACT, bool MUL = false, int CTA = CTA_THREADS, int TMW = 0>
__global__ void __launch_bounds__(CTA, 1)
row_pipe_kernel(const T* __restrict__ X, int64_t M, int C, const T* __restrict__ gamma,
                const T* __restrict__ beta, const float* __restrict__ col_mul, float eps, int mode, int stages,
                int8_t* __restrict__ Xq,
                float* __restrict__ scale, float* __restrict__ absmax_word, float* __restrict__ stats,
                int stats_are_input, uint32_t* __restrict__ status) {
    constexpr int G = CTA / GROUP;  // rows in flight per CTA
    constexpr int NW = GROUP / 32;
    constexpr bool TM = TMW != 0;   // parameters in tensor memory, read TMW (8 or 16) words at a time
    static_assert(TMW == 0 || TMW == 8 || TMW == 16, "tensor-memory read width");
    extern __shared__ __align__(128) uint8_t smem[];
    const int row_bytes = C * 2;
    const int nvec = C >> 3;
    static_assert(!TM || (LN && EXACT && !MUL && 16 * V * (NW == 8 ? 2 : 1) <= 512 && (NW == 1 || NW == 2 || NW == 4 || NW == 8)),
                  "tensor-memory parameters: LayerNorm on exact rows, one or two column ranges of 16 V words");
    uint8_t* s_gamma = smem;                                   // [C] T   (LN only, not TM)
    uint8_t* s_beta = smem + (LN ? row_bytes : 0);             // [C] T   (LN only, not TM)
    const float* s_mul = reinterpret_cast<const float*>(smem); // [C] fp32 (MUL only)
    uint8_t* s_rows = smem + (((LN && !TM) || MUL) ? 2 * row_bytes : 0);  // [G][stages][C] T
    uint64_t* full = reinterpret_cast<uint64_t*>(s_rows + (size_t)G * stages * row_bytes);  // [G][stages]
    constexpr int NWP = (NW + 3) & ~3;  // partial slots padded to whole 16-byte vectors
    float* s_red = reinterpret_cast<float*>(
        (reinterpret_cast<uintptr_t>(full + G * stages) + 15) & ~(uintptr_t)15);           // [G][3][NWP]

    const int tid = threadIdx.x;
    const int g = tid / GROUP, gt = tid % GROUP, gwarp = gt >> 5, lane = tid & 31;
    // rows go round the CTAs first and round a CTA's groups second: a handful of rows (one token per
    // sequence at the generation stage) then sit on as many SMs instead of sharing one
    const int64_t first = (int64_t)g * gridDim.x + blockIdx.x;
    const int64_t stride = (int64_t)gridDim.x * G;
    uint64_t* my_full = full + g * stages;
    uint8_t* my_rows = s_rows + (size_t)g * stages * row_bytes;
    float* red = s_red + g * 3 * NWP;
    volatile uint32_t* my_flag = reinterpret_cast<volatile uint32_t*>(s_red + G * 3 * NWP) + g;
    uint32_t* tmem_holder = const_cast<uint32_t*>(reinterpret_cast<volatile uint32_t*>(s_red + G * 3 * NWP) + G);
    constexpr uint32_t kTmCols = 16 * V * (NW == 8 ? 2 : 1) <= 256 ? 256 : 512;  // a power of two that holds the column ranges
    if (TM && tid < 32) tc::tmem_alloc<1>(tmem_holder, kTmCols);  // warp 0; freed at the end of the kernel

    if (gt == 0) {
        for (int s = 0; s < stages; ++s) mbar_init(my_full + s, 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    pdl_wait();               // the producer of X (and of the statistics / absmax word) has completed
    pdl_launch_dependents();  // the next kernel may be scheduled as this one's CTAs drain
    if (gt == 0) {
        // prologue: fill the ring
        for (int s = 0; s < stages; ++s) {
            const int64_t r = first + (int64_t)s * stride;
            if (r < M) {
                mbar_expect_tx(my_full + s, (uint32_t)row_bytes);
                bulk_load(my_rows + (size_t)s * row_bytes, X + r * C, (uint32_t)row_bytes, my_full + s);
            }
        }
    }
    if (MUL) {
        const float4* m4 = reinterpret_cast<const float4*>(col_mul);
        for (int v = tid; v < 2 * nvec; v += CTA) reinterpret_cast<float4*>(smem)[v] = __ldg(m4 + v);
    }
    if (LN && !TM) {  // parameters: global -> shared once per CTA
        const uint4* g4 = reinterpret_cast<const uint4*>(gamma);
        const uint4* b4 = reinterpret_cast<const uint4*>(beta);
        for (int v = tid; v < nvec; v += CTA) {
            reinterpret_cast<uint4*>(s_gamma)[v] = __ldg(g4 + v);
            reinterpret_cast<uint4*>(s_beta)[v] = beta ? __ldg(b4 + v) : make_uint4(0u, 0u, 0u, 0u);
        }
    }
    uint32_t tm_addr = 0;
    if (TM) {
        tc::tcgen05_fence_before();
        __syncthreads();  // the allocation's address is in shared memory
        tc::tcgen05_fence_after();
        const int warp = tid >> 5;
        // this thread's lane quarter and, for eight-warp groups, the column range of its half of the group
        tm_addr = *tmem_holder + ((uint32_t)((warp & 3) * 32) << 16) + (uint32_t)((NW == 8 ? (gwarp >> 2) : 0) * 16 * V);
        if (warp < (NW == 8 ? 8 : 4)) {  // one writer per lane quarter and column range
            const uint4* g4 = reinterpret_cast<const uint4*>(gamma);
            const uint4* b4 = reinterpret_cast<const uint4*>(beta);
#pragma unroll
            for (int i = 0; i < V; ++i) {
                const int v = gt + i * GROUP;
                float2 ga[4], be[4];
                unpack8_pairs<T>(__ldg(g4 + v), ga);
                unpack8_pairs<T>(beta ? __ldg(b4 + v) : make_uint4(0u, 0u, 0u, 0u), be);
                uint32_t w[16];
#pragma unroll
                for (int j = 0; j < 4; ++j) {  // words: gamma, beta of pairs 0, 1, then of pairs 2, 3 (eight words per half vector)
                    const int o = 8 * (j >> 1) + 2 * (j & 1);
                    w[o] = __float_as_uint(ga[j].x); w[o + 1] = __float_as_uint(ga[j].y);
                    w[o + 4] = __float_as_uint(be[j].x); w[o + 5] = __float_as_uint(be[j].y);
                }
                tm_st16(tm_addr + 16 * i, w);
            }
            asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory");
        }
        tc::tcgen05_fence_before();
    }
    __syncthreads();
    if (TM) tc::tcgen05_fence_after();

    float tensor_delta = 0.0f;
    if (mode == ROW_GIVEN_SCALE) tensor_delta = __ldg(scale);
    else if (mode == ROW_FROM_ABSMAX_WORD) {
        tensor_delta = step_size(__ldg(absmax_word));
        if (blockIdx.x == 0 && tid == 0) scale[0] = tensor_delta;
    }
    const float inv_C = __fdiv_rn(1.0f, (float)C);
    float group_max = 0.0f;  // ROW_ABSMAX_ONLY: one atomic per group at the end

    int s = 0;
    uint32_t parity = 0;
    for (int64_t row = first; row < M; row += stride) {
        // One thread waits (bounded) for the row's bulk copy; its outcome reaches the group through
        // shared memory so that every thread takes the same branch.
        if (gt == 0) {
            *my_flag = wait_row(my_full + s, parity, status) ? 1u : 0u;
        }
        group_sync<GROUP, CTA>(g);
        if (*my_flag == 0u) break;  // the copy never landed: stop this group
        const uint4* srow = reinterpret_cast<const uint4*>(my_rows + (size_t)s * row_bytes);
        uint4 raw[V];
#pragma unroll
        for (int i = 0; i < V; ++i) {
            const int v = gt + i * GROUP;
            raw[i] = (EXACT || v < nvec) ? srow[v] : make_uint4(0u, 0u, 0u, 0u);
        }
        // After the next group-wide barrier everyone holds the row in registers and the stage can
        // be refilled with the row `stages` iterations ahead.
        bool refilled = false;
        auto refill = [&]() {
            if (!refilled && gt == 0) {
                const int64_t nxt = row + (int64_t)stages * stride;
                if (nxt < M) {
                    mbar_expect_tx(my_full + s, (uint32_t)row_bytes);
                    bulk_load(my_rows + (size_t)s * row_bytes, X + nxt * C, (uint32_t)row_bytes, my_full + s);
                }
            }
            refilled = true;
        };
        if ((LN && stats_are_input) || (!LN && mode != ROW_DYNAMIC && mode != ROW_ABSMAX_ONLY)) {
            group_sync<GROUP, CTA>(g);  // no reduction follows on this path: synchronise explicitly
            refill();
        }

        float m = 0.0f;
        // LayerNorm and the column multiplier change the values and keep them as fp32; the plain
        // quantiser keeps the packed 16-bit row (half the registers: rows of up to 81 920 elements
        // fit) and unpacks a vector only when it is rounded.
        constexpr bool FP32_ROW = LN || MUL;
        float2 y[FP32_ROW ? V : 1][4];  // pairs: the two-wide fp32 instructions take them as they are
        if (FP32_ROW) {
#pragma unroll
            for (int i = 0; i < V; ++i) unpack8_pairs<T>(raw[i], y[FP32_ROW ? i : 0]);
        }
        if (LN) {
            float mu, rstd;
            if (stats_are_input) {
                mu = stats[2 * row];
                rstd = stats[2 * row + 1];
            } else {
                float2 sum2[2] = {make_float2(0.f, 0.f), make_float2(0.f, 0.f)};
#pragma unroll
                for (int i = 0; i < V; ++i) {  // zero-filled vectors add nothing
                    const float2* f = y[FP32_ROW ? i : 0];
                    sum2[0] = __fadd2_rn(sum2[0], __fadd2_rn(f[0], f[1]));
                    sum2[1] = __fadd2_rn(sum2[1], __fadd2_rn(f[2], f[3]));
                }
                const float sum = (sum2[0].x + sum2[0].y) + (sum2[1].x + sum2[1].y);
                if constexpr (!EXACT) {
                    mu = group_reduce<false, GROUP, CTA>(sum, red, g, gwarp, lane) * inv_C;
                    refill();
                } else {
                    mu = sum * (1.0f / (float)(8 * V));  // this thread's own mean first
                }
                const float2 nmu2 = make_float2(-mu, -mu);
                float2 ss2[2] = {make_float2(0.f, 0.f), make_float2(0.f, 0.f)};
#pragma unroll
                for (int i = 0; i < V; ++i) {
                    if (EXACT || gt + i * GROUP < nvec) {
#pragma unroll
                        for (int j = 0; j < 4; ++j) {
                            const float2 d = __fadd2_rn(y[FP32_ROW ? i : 0][j], nmu2);
                            ss2[j & 1] = __ffma2_rn(d, d, ss2[j & 1]);
                        }
                    }
                }
                float ss = (ss2[0].x + ss2[0].y) + (ss2[1].x + ss2[1].y);
                if constexpr (!EXACT) {
                    ss = group_reduce<false, GROUP, CTA>(ss, red + NWP, g, gwarp, lane);
                } else {
                    group_merge_stats<GROUP, CTA>(mu, ss, (float)(8 * V), red, red + NWP, g, gwarp, lane);
                    refill();
                }
                const float var = ss * inv_C;
                rstd = rsqrt_refined(var + eps);
                if (stats != nullptr && gt == 0) {
                    stats[2 * row] = mu;
                    stats[2 * row + 1] = rstd;
                }
            }
            const float shift = -__fmul_rn(mu, rstd);
            const float2 rstd2 = make_float2(rstd, rstd), shift2 = make_float2(shift, shift);
            if constexpr (TM) {
                // TMW words at a time (a vector's 16, or half a vector's 8 where registers are short), the next
                // read on its way while this one is used; a half vector holds gamma, beta of two pairs
                constexpr int NP = TMW / 4;  // pairs per read
                uint32_t gb[2][TMW == 0 ? 8 : TMW];
                auto ld = [&](int k, uint32_t (&r)[TMW == 0 ? 8 : TMW]) {
                    if constexpr (TMW == 16) tm_ld16(tm_addr + 16 * k, r); else tm_ld8(tm_addr + 8 * k, r);
                };
                auto ld_wait = [&](uint32_t (&r)[TMW == 0 ? 8 : TMW]) {
                    if constexpr (TMW == 16) tm_ld_wait16(r); else tm_ld_wait8(r);
                };
                constexpr int READS = 16 * V / (TMW == 0 ? 8 : TMW);
                ld(0, gb[0]);
#pragma unroll
                for (int k = 0; k < READS; ++k) {
                    uint32_t (&cur)[TMW == 0 ? 8 : TMW] = gb[k & 1];
                    ld_wait(cur);
                    if (k + 1 < READS) ld(k + 1, gb[(k + 1) & 1]);
#pragma unroll
                    for (int jj = 0; jj < NP; ++jj) {
                        const int i = (k * NP + jj) >> 2, j = (k * NP + jj) & 3;
                        const int o = 8 * (jj >> 1) + 2 * (jj & 1);  // word of this pair's gamma inside the read
                        const float2 ga = make_float2(__uint_as_float(cur[o]), __uint_as_float(cur[o + 1]));
                        const float2 be = make_float2(__uint_as_float(cur[o + 4]), __uint_as_float(cur[o + 5]));
                        const float2 t = __ffma2_rn(__ffma2_rn(y[FP32_ROW ? i : 0][j], rstd2, shift2), ga, be);
                        y[FP32_ROW ? i : 0][j] = t;
                        m = fmaxf(m, fmaxf(fabsf(t.x), fabsf(t.y)));
                    }
                }
            } else {
#pragma unroll
            for (int i = 0; i < V; ++i) {
                const int v = gt + i * GROUP;
                if (EXACT || v < nvec) {
                    float2 ga[4], be[4];
                    unpack8_pairs<T>(reinterpret_cast<const uint4*>(s_gamma)[v], ga);
                    unpack8_pairs<T>(reinterpret_cast<const uint4*>(s_beta)[v], be);
#pragma unroll
                    for (int j = 0; j < 4; ++j) {
                        // (x * rstd + shift) * gamma + beta, each product-sum rounded once
                        const float2 t = __ffma2_rn(__ffma2_rn(y[FP32_ROW ? i : 0][j], rstd2, shift2), ga[j], be[j]);
                        y[FP32_ROW ? i : 0][j] = t;
                        m = fmaxf(m, fmaxf(fabsf(t.x), fabsf(t.y)));
                    }
                }
            }
            }
        } else if (MUL) {
#pragma unroll
            for (int i = 0; i < V; ++i) {
                const int v = gt + i * GROUP;
                if (EXACT || v < nvec) {
                    const float4 m0 = reinterpret_cast<const float4*>(s_mul)[2 * v];
                    const float4 m1 = reinterpret_cast<const float4*>(s_mul)[2 * v + 1];
                    float2* f = y[FP32_ROW ? i : 0];
                    f[0] = __fmul2_rn(f[0], make_float2(m0.x, m0.y));
                    f[1] = __fmul2_rn(f[1], make_float2(m0.z, m0.w));
                    f[2] = __fmul2_rn(f[2], make_float2(m1.x, m1.y));
                    f[3] = __fmul2_rn(f[3], make_float2(m1.z, m1.w));
#pragma unroll
                    for (int j = 0; j < 4; ++j) m = fmaxf(m, fmaxf(fabsf(f[j].x), fabsf(f[j].y)));
                }
            }
        } else if (mode == ROW_DYNAMIC || mode == ROW_ABSMAX_ONLY) {
            uint32_t pm = 0u;  // packed running max of |x|: exact in fp16/bf16
#pragma unroll
            for (int i = 0; i < V; ++i) {
                pm = Act<T>::absmax2(pm, raw[i].x); pm = Act<T>::absmax2(pm, raw[i].y);
                pm = Act<T>::absmax2(pm, raw[i].z); pm = Act<T>::absmax2(pm, raw[i].w);
            }
            m = Act<T>::hmax_of2(pm);
        }

        float delta = tensor_delta;
        if (mode == ROW_DYNAMIC || mode == ROW_ABSMAX_ONLY) {
            m = group_reduce<true, GROUP, CTA>(m, red + 2 * NWP, g, gwarp, lane);
            refill();
            if (mode == ROW_ABSMAX_ONLY) {
                group_max = fmaxf(group_max, m);
                if (++s == stages) { s = 0; parity ^= 1u; }
                continue;
            }
            delta = step_size(m);
            if (gt == 0) scale[row] = delta;
        } else if (mode == ROW_GIVEN_ROW_ABSMAX) {  // the row's maximum was agreed on elsewhere (all ranks' slices)
            delta = step_size(__ldg(absmax_word + row));
            if (gt == 0) scale[row] = delta;
        }
        const float inv = recip_step(delta);
        uint2* qrow = reinterpret_cast<uint2*>(Xq + row * C);
        if (mode == ROW_GIVEN_SCALE || mode == ROW_GIVEN_ROW_ABSMAX) {  // a given step may be exceeded: saturate
#pragma unroll
            for (int i = 0; i < V; ++i) {
                const int v = gt + i * GROUP;
                if (EXACT || v < nvec) {
                    if (FP32_ROW) {
                        qrow[v] = quant8_pairs<true>(y[FP32_ROW ? i : 0], inv);
                    } else {
                        float2 f[4];
                        unpack8_pairs<T>(raw[i], f);
                        qrow[v] = quant8_pairs<true>(f, inv);
                    }
                }
            }
        } else {  // |y| <= absmax by construction: |y * inv| < 127.5, no clamp needed
#pragma unroll
            for (int i = 0; i < V; ++i) {
                const int v = gt + i * GROUP;
                if (EXACT || v < nvec) {
                    if (FP32_ROW) {
                        qrow[v] = quant8_pairs<false>(y[FP32_ROW ? i : 0], inv);
                    } else {
                        float2 f[4];
                        unpack8_pairs<T>(raw[i], f);
                        qrow[v] = quant8_pairs<false>(f, inv);
                    }
                }
            }
        }
        if (++s == stages) { s = 0; parity ^= 1u; }
    }
    if (mode == ROW_ABSMAX_ONLY && gt == 0) atomic_max_nonneg(absmax_word, group_max);
    (void)parity;
    if (TM) {  // every group is done with the parameters (whether it finished or gave up)
        tc::tcgen05_fence_before();
        __syncthreads();
        if (tid < 32) {
            tc::tcgen05_fence_after();
            tc::tmem_dealloc<1>(*tmem_holder, kTmCols);
        }
    }
}

template <typename T, int GROUP, int V, bool LN, bool EXACT = false, bool MUL = false, int CTA = CTA_THREADS, int TMW = 0>
sq_status launch_pipe(const void* X, int64_t M, int64_t C, const void* gamma, const void* beta, const float* col_mul, float eps,
                      int mode, int8_t* Xq, float* scale, float* absmax_word, float* stats, int stats_are_input,
                      uint32_t* status, cudaStream_t st) {
    constexpr int G = CTA / GROUP;
    constexpr bool TM = TMW != 0;
    const size_t row_bytes = (size_t)C * 2;
    const size_t fixed = (((LN && !TM) || MUL) ? 2 * row_bytes : 0) + 2048 /*barriers + reduction scratch*/;
    const size_t budget = 220 * 1024;
    if (budget < fixed + G * row_bytes) return SQ_ERR_UNSUPPORTED;
    int stages = (int)((budget - fixed) / (G * row_bytes));
    stages = std::min(stages, 8);
    const size_t smem = (((LN && !TM) || MUL) ? 2 * row_bytes : 0) + (size_t)G * stages * row_bytes + (size_t)G * stages * 8 +
                        (size_t)G * 3 * ((GROUP / 32 + 3) & ~3) * 4 + (size_t)G * 4 + 4 + 144;
    auto kern = row_pipe_kernel<T, GROUP, V, LN, EXACT, MUL, CTA, TMW>;
    static bool attr_set[64] = {false};
    int dev = 0;
    SQ_CUDA_OK(cudaGetDevice(&dev));
    if (dev < 0 || dev >= 64 || !attr_set[dev]) {
        SQ_CUDA_OK(cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, 226 * 1024));
        if (dev >= 0 && dev < 64) attr_set[dev] = true;
    }
    const int grid = (int)std::min<int64_t>(M, sm_count());
    return launch_pdl(kern, dim3((unsigned)grid), dim3(CTA), smem, st, 1, static_cast<const T*>(X), M,
                      (int)C, static_cast<const T*>(gamma), static_cast<const T*>(beta), col_mul, eps, mode, stages, Xq, scale,
                      absmax_word, stats, stats_are_input, status);
}

template <typename T, bool LN>
sq_status dispatch_pipe(const void* X, int64_t M, int64_t C, const void* gamma, const void* beta, float eps,
                        int mode, int8_t* Xq, float* scale, float* absmax_word, float* stats,
                        int stats_are_input, uint32_t* status, cudaStream_t st) {
    const int64_t nvec = C / 8;
#define SQ_PIPE(GROUP, V)                                                                                  \
    return launch_pipe<T, GROUP, V, LN>(X, M, C, gamma, beta, nullptr, eps, mode, Xq, scale, absmax_word, stats, \
                                        stats_are_input, status, st)
#define SQ_PIPE_EXACT(GROUP, V)                                                                            \
    if (nvec == (GROUP) * (V))                                                                             \
        return launch_pipe<T, GROUP, V, LN, true>(X, M, C, gamma, beta, nullptr, eps, mode, Xq, scale, absmax_word, \
                                                  stats, stats_are_input, status, st)
    // the hidden sizes of the model shapes this library is benchmarked on divide evenly
    if constexpr (LN) {
        // LayerNorm is bound by instruction issue and by the three reductions a row costs: 384
        // threads leave room for 112 to 128 fp32 values per thread, so a row needs only two or
        // three warps (measured: 0.79 -> 0.89 of the copy bandwidth at 7168, 0.75 -> 0.91 at 12288)
#define SQ_PIPE_LN384(GROUP, V)                                                                                  \
        if (nvec == (GROUP) * (V))                                                                               \
            return launch_pipe<T, GROUP, V, LN, true, false, 384>(X, M, C, gamma, beta, nullptr, eps, mode, Xq, scale, \
                                                                  absmax_word, stats, stats_are_input, status, st)
        // Parameters in tensor memory where it measured faster (fraction of the 6534 GB/s copy bandwidth, shared
        // memory -> tensor memory): 32768 x 4096 0.84 -> 0.86 with whole-vector reads; with half-vector reads
        // 16384 x 14336 0.85 -> 0.92, 16384 x 20480 0.83 -> 0.89-0.92 and 8192 x 7168 43.1 -> 37.2 us (65536 x 7168
        // unchanged at 0.90); 5120 and 8192 lose 4-5 % and stay as they were; groups of three warps (12288)
        // would need three column ranges, more than tensor memory has, and 12288 as 128 x 12 gains 3 % at 16384 rows
        // but loses 7 % at 4096.
#define SQ_PIPE_LN_TM(GROUP, V, CTA, TMW)                                                                        \
        if (nvec == (GROUP) * (V))                                                                               \
            return launch_pipe<T, GROUP, V, LN, true, false, CTA, (LN && kLnTensorMemory) ? TMW : 0>(X, M, C, gamma, beta, nullptr, eps, mode, Xq, \
                                                                                scale, absmax_word, stats, stats_are_input, status, st)
        SQ_PIPE_LN_TM(32, 16, 384, 16);           // 4096
        SQ_PIPE_LN_TM(64, 14, 384, 8);            // 7168
        SQ_PIPE_LN_TM(128, 9, 384, 16);           // 9216: four-warp groups (three-warp ones cannot share columns), 0.82 -> 0.90
        SQ_PIPE_LN_TM(128, 14, 384, 8);           // 14336
        SQ_PIPE_LN_TM(256, 10, CTA_THREADS, 8);   // 20480
#undef SQ_PIPE_LN_TM
        SQ_PIPE_LN384(64, 16);   // 8192
        SQ_PIPE_LN384(96, 16);   // 12288
#undef SQ_PIPE_LN384
    }
    SQ_PIPE_EXACT(64, 8);    // 4096
    SQ_PIPE_EXACT(64, 10);   // 5120
    SQ_PIPE_EXACT(128, 7);   // 7168
    SQ_PIPE_EXACT(256, 6);   // 12288
    SQ_PIPE_EXACT(256, 10);  // 20480
    SQ_PIPE_EXACT(512, 7);   // 28672
#undef SQ_PIPE_EXACT
    if constexpr (LN) {
#define SQ_PIPE_LN384_ANY(GROUP, V)                                                                              \
        if (nvec <= (GROUP) * (V))                                                                               \
            return launch_pipe<T, GROUP, V, LN, false, false, 384>(X, M, C, gamma, beta, nullptr, eps, mode, Xq, scale, \
                                                                   absmax_word, stats, stats_are_input, status, st)
        SQ_PIPE_LN384_ANY(64, 16);   // C <= 8192
        SQ_PIPE_LN384_ANY(96, 16);   // C <= 12288
        SQ_PIPE_LN384_ANY(128, 14);  // C <= 14336
#undef SQ_PIPE_LN384_ANY
    }
    if (nvec <= 64 * 8) SQ_PIPE(64, 8);      // C <= 4096
    if (nvec <= 64 * 10) SQ_PIPE(64, 10);    // C <= 5120
    if (nvec <= 128 * 8) SQ_PIPE(128, 8);    // C <= 8192   (7168)
    if (nvec <= 128 * 10) SQ_PIPE(128, 10);  // C <= 10240
    if (nvec <= 256 * 8) SQ_PIPE(256, 8);    // C <= 16384  (12288)
    if (nvec <= 256 * 10) SQ_PIPE(256, 10);  // C <= 20480
    if (nvec <= 512 * 8 || LN) SQ_PIPE(512, 8);  // C <= 32768  (28672)
    if constexpr (!LN) {                         // wider rows: plain quantiser only (the row stays packed in registers)
        if (nvec <= 512 * 12) SQ_PIPE(512, 12);  // C <= 49152
        if (nvec <= 512 * 16) SQ_PIPE(512, 16);  // C <= 65536
        SQ_PIPE(512, 20);                        // C <= 81920
    }
    return SQ_ERR_UNSUPPORTED;
#undef SQ_PIPE
}

// Column-multiplier variant (weights folded with s, activations scaled by 1/s): the generic ladder
// only -- these calls are offline or rare, so the bounds-check-free instantiations are not built.
template <typename T>
sq_status dispatch_pipe_mul(const void* X, int64_t M, int64_t C, const float* col_mul, int mode, int8_t* Xq,
                            float* scale, float* absmax_word, uint32_t* status, cudaStream_t st) {
    const int64_t nvec = C / 8;
#define SQ_PIPE(GROUP, V)                                                                                       \
    return launch_pipe<T, GROUP, V, false, false, true>(X, M, C, nullptr, nullptr, col_mul, 0.f, mode, Xq, scale, \
                                                        absmax_word, nullptr, 0, status, st)
    if (nvec <= 64 * 10) SQ_PIPE(64, 10);    // C <= 5120
    if (nvec <= 128 * 10) SQ_PIPE(128, 10);  // C <= 10240
    if (nvec <= 256 * 10) SQ_PIPE(256, 10);  // C <= 20480
    SQ_PIPE(512, 8);                         // C <= 32768
#undef SQ_PIPE
}

}  // namespace

sq_status row_wait_selftest(uint32_t* status, uint32_t budget, cudaStream_t st) {
    row_wait_selftest_kernel<<<1, 32, 0, st>>>(status, budget);
    return launch_status();
}

bool row_pipeline_supports(int64_t M, int64_t C, bool ln, bool has_col_mul) {
    // LayerNorm and column-multiplied rows are held as fp32 (up to 32 768 elements); the plain
    // quantiser holds the packed row (up to 81 920)
    const int64_t max_vec = (ln || has_col_mul) ? 512 * 8 : 512 * 20;
    return M > 0 && C % 8 == 0 && C / 8 <= max_vec;
}

sq_status row_pipeline(const void* X, sq_dtype dt, int64_t M, int64_t C, const float* col_mul, const void* gamma,
                       const void* beta, float eps, bool ln, int mode, int8_t* Xq, float* scale, float* absmax_word,
                       float* stats, int stats_are_input, uint32_t* status, cudaStream_t st) {
    if (col_mul != nullptr && !ln)
        return dt == SQ_F16 ? dispatch_pipe_mul<__half>(X, M, C, col_mul, mode, Xq, scale, absmax_word, status, st)
                            : dispatch_pipe_mul<__nv_bfloat16>(X, M, C, col_mul, mode, Xq, scale, absmax_word, status, st);
    if (dt == SQ_F16)
        return ln ? dispatch_pipe<__half, true>(X, M, C, gamma, beta, eps, mode, Xq, scale, absmax_word, stats,
                                                stats_are_input, status, st)
                  : dispatch_pipe<__half, false>(X, M, C, nullptr, nullptr, 0.f, mode, Xq, scale, absmax_word,
                                                 nullptr, 0, status, st);
    return ln ? dispatch_pipe<__nv_bfloat16, true>(X, M, C, gamma, beta, eps, mode, Xq, scale, absmax_word, stats,
                                                   stats_are_input, status, st)
              : dispatch_pipe<__nv_bfloat16, false>(X, M, C, nullptr, nullptr, 0.f, mode, Xq, scale, absmax_word,
                                                    nullptr, 0, status, st);
}

}  // namespace sq
