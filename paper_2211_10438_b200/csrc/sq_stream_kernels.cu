// HBM-bound streaming kernels of the SmoothQuant hot path:
//   calibration column-absmax (Section 4), smoothing factor (Eq. 4), LayerNorm folding
//   (Eq. 3), activation / weight quantisation (Eq. 1) and the fused LayerNorm + quantise.
// All are one pass over their input with 16-byte loads; a row is held in registers between
// its statistics pass and its quantise pass, so each element is read from HBM once.
#include <cooperative_groups.h>

#include "sq_bulk.cuh"
#include "sq_common.cuh"
#include "sq_kernels.h"

namespace cg = cooperative_groups;

namespace sq {

int sm_count() {
    static int cached[64] = {0};
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return kNumSMsB200;
    if (cached[dev] == 0) {
        int n = 0;
        if (cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || n <= 0)
            n = kNumSMsB200;
        cached[dev] = n;
    }
    return cached[dev];
}

// =======================================================================================
// Calibration: absmax[j] = max(absmax[j], max_t |X[t, j]|)        (Section 4)
// Block = 32 column-vectors (256 columns) x 8 row lanes; each thread walks down its rows
// with 4 independent 16-byte loads in flight and keeps a packed running maximum.
// =======================================================================================
template <typename T>
__global__ void __launch_bounds__(256)
col_absmax_vec_kernel(const T* __restrict__ X, int64_t rows, int64_t cols, int64_t ld,
                      float* __restrict__ absmax) {
    const int tx = threadIdx.x & 31, ty = threadIdx.x >> 5;
    const int64_t vcol = (int64_t)blockIdx.x * 32 + tx;  // 8-column vector index
    const bool active = vcol * 8 < cols;
    const int64_t row_step = (int64_t)gridDim.y * 8;
    uint4 m = make_uint4(0u, 0u, 0u, 0u);
    if (active) {
        const uint4* base = reinterpret_cast<const uint4*>(X + vcol * 8);
        const int64_t ldv = ld / 8;
        int64_t r = (int64_t)blockIdx.y * 8 + ty;
        for (; r + 3 * row_step < rows; r += 4 * row_step) {
            uint4 v0 = __ldcs(base + r * ldv);
            uint4 v1 = __ldcs(base + (r + row_step) * ldv);
            uint4 v2 = __ldcs(base + (r + 2 * row_step) * ldv);
            uint4 v3 = __ldcs(base + (r + 3 * row_step) * ldv);
#define SQ_ACC(v)                                                                          \
    m.x = Act<T>::absmax2(m.x, v.x); m.y = Act<T>::absmax2(m.y, v.y);                       \
    m.z = Act<T>::absmax2(m.z, v.z); m.w = Act<T>::absmax2(m.w, v.w);
            SQ_ACC(v0) SQ_ACC(v1) SQ_ACC(v2) SQ_ACC(v3)
        }
        for (; r < rows; r += row_step) {
            uint4 v0 = __ldcs(base + r * ldv);
            SQ_ACC(v0)
        }
#undef SQ_ACC
    }
    __shared__ uint4 sm[8][32];
    sm[ty][tx] = m;
    __syncthreads();
    if (ty == 0 && active) {
#pragma unroll
        for (int i = 1; i < 8; ++i) {
            uint4 o = sm[i][tx];
            m.x = Act<T>::absmax2(m.x, o.x); m.y = Act<T>::absmax2(m.y, o.y);
            m.z = Act<T>::absmax2(m.z, o.z); m.w = Act<T>::absmax2(m.w, o.w);
        }
        float f[8];
        unpack8<T>(m, f);
#pragma unroll
        for (int i = 0; i < 8; ++i) atomic_max_nonneg(absmax + vcol * 8 + i, f[i]);
    }
}

template <typename T>
__global__ void col_absmax_scalar_kernel(const T* __restrict__ X, int64_t rows, int64_t cols,
                                         int64_t ld, float* __restrict__ absmax) {
    const int64_t j = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (j >= cols) return;
    float m = 0.0f;
    for (int64_t r = blockIdx.y; r < rows; r += gridDim.y)
        m = fmaxf(m, fabsf(Act<T>::to_float(X[r * ld + j])));
    atomic_max_nonneg(absmax + j, m);
}

// The same reduction as a stream for large calibration batches: the columns are cut into slabs of
// at most 640 vectors (5120 columns), the rows into gridDim.x / n_slabs parts; a CTA owns one slab
// of one part.  Its 8 groups of 64 threads each walk their own rows: a row's slab segment (up to
// 10 KB, contiguous) arrives by one bulk copy into the group's ring, every thread folds its 10
// vectors into packed running maxima, and only at the end do the groups meet in shared memory and
// issue one atomic max per column and CTA.  One named barrier per row and group: passing the
// barrier of row k proves that everybody finished reading row k - 1, whose stage is then refilled.
// A bulk copy that never lands (bounded wait) poisons the CTA's columns with NaN.
constexpr int CAL_THREADS = 512, CAL_GROUP = 64, CAL_V = 10, CAL_G = CAL_THREADS / CAL_GROUP;
template <typename T>
__global__ void __launch_bounds__(CAL_THREADS, 1)
col_absmax_stream_kernel(const T* __restrict__ X, int64_t rows, int64_t nvec, int64_t ld, int slab_vecs, int n_slabs,
                         int stages, float* __restrict__ absmax) {
    using namespace bulk;
    extern __shared__ __align__(128) uint8_t cal_smem[];
    const int tid = threadIdx.x, g = tid / CAL_GROUP, gt = tid % CAL_GROUP;
    const int slab = blockIdx.x % n_slabs, part = blockIdx.x / n_slabs, parts = gridDim.x / n_slabs;
    const int64_t v0 = (int64_t)slab * slab_vecs;
    const int nv = (int)min((int64_t)slab_vecs, nvec - v0);  // vectors of this slab
    const uint32_t seg_bytes = (uint32_t)nv * 16u;
    const size_t stage_bytes = (size_t)slab_vecs * 16;
    uint8_t* ring = cal_smem + (size_t)g * stages * stage_bytes;
    uint64_t* full = reinterpret_cast<uint64_t*>(cal_smem + (size_t)CAL_G * stages * stage_bytes) + g * stages;
    volatile uint32_t* flags = reinterpret_cast<volatile uint32_t*>(
        reinterpret_cast<uint64_t*>(cal_smem + (size_t)CAL_G * stages * stage_bytes) + CAL_G * stages);
    volatile uint32_t* my_flag = flags + g;
    volatile uint32_t* bad = flags + CAL_G;
    if (tid == 0) *bad = 0u;
    if (gt == 0) {
        for (int s = 0; s < stages; ++s) mbar_init(full + s, 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    __syncthreads();
    const int64_t first = (int64_t)part * CAL_G + g, stride = (int64_t)parts * CAL_G;
    const T* src = X + v0 * 8;
    if (gt == 0) {
        for (int s = 0; s < stages; ++s) {
            const int64_t r = first + s * stride;
            if (r < rows) {
                mbar_expect_tx(full + s, seg_bytes);
                bulk_load(ring + (size_t)s * stage_bytes, src + r * ld, seg_bytes, full + s);
            }
        }
    }
    uint4 cm[CAL_V];
#pragma unroll
    for (int i = 0; i < CAL_V; ++i) cm[i] = make_uint4(0u, 0u, 0u, 0u);
    int s = 0, prev = -1;
    uint32_t parity = 0;
    int64_t prev_row = 0;
    for (int64_t row = first; row < rows; row += stride) {
        if (gt == 0) {
            const bool ok = mbar_wait_bounded(full + s, parity);
            *my_flag = ok ? 1u : 0u;
        }
        asm volatile("bar.sync %0, %1;" ::"r"(g + 1), "n"(CAL_GROUP) : "memory");
        if (*my_flag == 0u) { *bad = 1u; break; }
        if (gt == 0 && prev >= 0) {  // everybody is past the reads of the previous row: refill its stage
            const int64_t nxt = prev_row + (int64_t)stages * stride;
            if (nxt < rows) {
                mbar_expect_tx(full + prev, seg_bytes);
                bulk_load(ring + (size_t)prev * stage_bytes, src + nxt * ld, seg_bytes, full + prev);
            }
        }
        const uint4* seg = reinterpret_cast<const uint4*>(ring + (size_t)s * stage_bytes);
#pragma unroll
        for (int i = 0; i < CAL_V; ++i) {
            const int v = gt + i * CAL_GROUP;
            if (v < nv) {
                const uint4 x = seg[v];
                cm[i].x = Act<T>::absmax2(cm[i].x, x.x); cm[i].y = Act<T>::absmax2(cm[i].y, x.y);
                cm[i].z = Act<T>::absmax2(cm[i].z, x.z); cm[i].w = Act<T>::absmax2(cm[i].w, x.w);
            }
        }
        prev = s; prev_row = row;
        if (++s == stages) { s = 0; parity ^= 1u; }
    }
    __syncthreads();  // every group is done with its ring: the space becomes [group][vector] scratch
    uint4* scratch = reinterpret_cast<uint4*>(cal_smem);
#pragma unroll
    for (int i = 0; i < CAL_V; ++i) {
        const int v = gt + i * CAL_GROUP;
        if (v < nv) scratch[(size_t)g * slab_vecs + v] = cm[i];
    }
    __syncthreads();
    const bool poisoned = *bad != 0u;
    for (int v = tid; v < nv; v += CAL_THREADS) {
        uint4 m = scratch[v];
#pragma unroll
        for (int o = 1; o < CAL_G; ++o) {
            const uint4 x = scratch[(size_t)o * slab_vecs + v];
            m.x = Act<T>::absmax2(m.x, x.x); m.y = Act<T>::absmax2(m.y, x.y);
            m.z = Act<T>::absmax2(m.z, x.z); m.w = Act<T>::absmax2(m.w, x.w);
        }
        float f[8];
        unpack8<T>(m, f);
#pragma unroll
        for (int i = 0; i < 8; ++i)
            atomic_max_nonneg(absmax + (v0 + v) * 8 + i, poisoned ? __uint_as_float(0x7fc00000u) : f[i]);
    }
}

template <typename T>
static sq_status calib_absmax_t(const void* X, int64_t rows, int64_t cols, int64_t ld, float* a,
                                cudaStream_t st) {
    const T* x = static_cast<const T*>(X);
    const int sms = sm_count();
    // (from about 256 MB per call the stream wins -- 16384 x 20480: 120 -> 101 us; below, its ring fill and
    // its final meeting of the groups cost more than they save, and a batch that fits L2 favours plain loads)
    if (aligned16(X) && cols % 8 == 0 && ld % 8 == 0 && cols >= 2048 && rows * cols >= ((int64_t)1 << 27)) {
        const int64_t nvec = cols / 8;
        const int n_slabs = (int)((nvec + CAL_GROUP * CAL_V - 1) / (CAL_GROUP * CAL_V));
        if (n_slabs <= sms) {
            const int slab_vecs = (int)((nvec + n_slabs - 1) / n_slabs);
            const int parts = (int)std::max<int64_t>(1, std::min<int64_t>(sms / n_slabs, (rows + CAL_G - 1) / CAL_G));
            const size_t stage_all = (size_t)CAL_G * slab_vecs * 16;
            const int stages = (int)std::min<size_t>(4, (size_t)(200 * 1024) / stage_all);  // >= 2: a slab is at most 10 KB
            const size_t smem = stage_all * stages + (size_t)CAL_G * stages * 8 + (CAL_G + 1) * 4 + 64;
            auto kern = col_absmax_stream_kernel<T>;
            static bool attr_set[64] = {false};
            int dev = 0;
            SQ_CUDA_OK(cudaGetDevice(&dev));
            if (dev < 0 || dev >= 64 || !attr_set[dev]) {
                SQ_CUDA_OK(cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, 226 * 1024));
                if (dev >= 0 && dev < 64) attr_set[dev] = true;
            }
            kern<<<dim3((unsigned)(parts * n_slabs)), CAL_THREADS, smem, st>>>(x, rows, nvec, ld, slab_vecs, n_slabs, stages, a);
            return launch_status();
        }
    }
    if (aligned16(X) && cols % 8 == 0 && ld % 8 == 0) {
        const int64_t gx = (cols / 8 + 31) / 32;
        // enough row slices for ~8 resident CTAs per SM, but at least 32 rows per slice
        int64_t gy = (8LL * sms + gx - 1) / gx;
        gy = std::max<int64_t>(1, std::min<int64_t>(gy, (rows + 31) / 32));
        gy = std::min<int64_t>(gy, 65535);
        col_absmax_vec_kernel<T><<<dim3((unsigned)gx, (unsigned)gy), 256, 0, st>>>(x, rows, cols, ld, a);
    } else {
        const int64_t gx = (cols + 255) / 256;
        int64_t gy = std::max<int64_t>(1, std::min<int64_t>((4LL * sms + gx - 1) / gx, rows));
        gy = std::min<int64_t>(gy, 65535);
        col_absmax_scalar_kernel<T><<<dim3((unsigned)gx, (unsigned)gy), 256, 0, st>>>(x, rows, cols, ld, a);
    }
    return launch_status();
}

sq_status calib_absmax(const void* X, sq_dtype dt, int64_t rows, int64_t cols, int64_t ld, float* a,
                       cudaStream_t st) {
    return dt == SQ_F16 ? calib_absmax_t<__half>(X, rows, cols, ld, a, st)
                        : calib_absmax_t<__nv_bfloat16>(X, rows, cols, ld, a, st);
}

// =======================================================================================
// Static-step calibration with the largest tokens set aside (Section 5.2: the top 2 % of tokens
// are clipped when the static step sizes are calibrated for GLM-130B): per-token |max| of every
// calibration token, then the exact (n_clip + 1)-th largest of them.
// =======================================================================================
template <typename T>
__global__ void __launch_bounds__(256)
token_absmax_kernel(const T* __restrict__ X, int64_t M, int64_t C, int64_t ld, float* __restrict__ out) {
    // one warp per token; packed |x| / max on 16-bit pairs is exact
    const int lane = threadIdx.x & 31;
    const int64_t row = (int64_t)blockIdx.x * 8 + (threadIdx.x >> 5);
    if (row >= M) return;
    const uint4* src = reinterpret_cast<const uint4*>(X + row * ld);
    const int64_t nvec = C / 8;
    uint4 m = make_uint4(0u, 0u, 0u, 0u);
    for (int64_t v = lane; v < nvec; v += 32) {
        const uint4 x = __ldcs(src + v);
        m.x = Act<T>::absmax2(m.x, x.x); m.y = Act<T>::absmax2(m.y, x.y);
        m.z = Act<T>::absmax2(m.z, x.z); m.w = Act<T>::absmax2(m.w, x.w);
    }
    float f[8];
    unpack8<T>(m, f);
    float r = fmaxf(fmaxf(fmaxf(f[0], f[1]), fmaxf(f[2], f[3])), fmaxf(fmaxf(f[4], f[5]), fmaxf(f[6], f[7])));
    r = warp_max(r);
    if (lane == 0) out[row] = r;
}

// Exact selection among T non-negative floats: their bit patterns order like the values, so four
// passes of an 8-bit histogram (most significant byte first) pin the pattern of the element of
// descending rank k.  One CTA; T is a calibration set's token count (10^4 .. 10^7).
__global__ void __launch_bounds__(1024)
select_rank_kernel(const float* __restrict__ vals, int64_t T, int64_t k, float* __restrict__ absmax_out,
                   float* __restrict__ step_out) {
    __shared__ uint32_t hist[256];
    __shared__ uint32_t s_prefix, s_k;
    const uint32_t* u = reinterpret_cast<const uint32_t*>(vals);
    if (threadIdx.x == 0) { s_prefix = 0u; s_k = (uint32_t)k; }
    for (int pass = 0; pass < 4; ++pass) {
        const int shift = 24 - 8 * pass;
        const uint32_t mask = pass == 0 ? 0u : (0xffffffffu << (shift + 8));
        if (threadIdx.x < 256) hist[threadIdx.x] = 0u;
        __syncthreads();
        const uint32_t prefix = s_prefix;
        for (int64_t i = threadIdx.x; i < T; i += blockDim.x) {
            const uint32_t x = u[i];
            if ((x & mask) == prefix) atomicAdd(&hist[(x >> shift) & 255u], 1u);
        }
        __syncthreads();
        if (threadIdx.x == 0) {
            uint32_t kk = s_k, bin = 255u;
            for (;; --bin) {  // from the largest byte down; the counts of this pass sum to more than kk
                if (hist[bin] > kk || bin == 0u) break;
                kk -= hist[bin];
            }
            s_k = kk;
            s_prefix = prefix | (bin << shift);
        }
        __syncthreads();
    }
    if (threadIdx.x == 0) {
        const float a = __uint_as_float(s_prefix);
        absmax_out[0] = a;
        if (step_out) step_out[0] = step_size(a);
    }
}

sq_status token_absmax(const void* X, sq_dtype dt, int64_t M, int64_t C, int64_t ld, float* out, cudaStream_t st) {
    const unsigned grid = (unsigned)((M + 7) / 8);
    if (dt == SQ_F16)
        token_absmax_kernel<__half><<<grid, 256, 0, st>>>(static_cast<const __half*>(X), M, C, ld, out);
    else
        token_absmax_kernel<__nv_bfloat16><<<grid, 256, 0, st>>>(static_cast<const __nv_bfloat16*>(X), M, C, ld, out);
    return launch_status();
}

sq_status clipped_absmax(const float* token_absmax, int64_t T, int64_t n_clip, float* absmax_out, float* step_out,
                         cudaStream_t st) {
    const int64_t k = std::max<int64_t>(0, std::min<int64_t>(n_clip, T - 1));  // at least one token is kept
    select_rank_kernel<<<1, 1024, 0, st>>>(token_absmax, T, k, absmax_out, step_out);
    return launch_status();
}

// =======================================================================================
// Eq. 4 and the LayerNorm fold of Eq. 3 (tiny, offline)
// =======================================================================================
__global__ void smooth_scales_kernel(const float* __restrict__ ax, const float* __restrict__ aw,
                                     int64_t C, float alpha, float* __restrict__ s,
                                     float* __restrict__ s_inv) {
    const int64_t j = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (j >= C) return;
    const double a = (double)alpha;
    const double x = (double)fmaxf(ax[j], kAbsmaxFloor), w = (double)fmaxf(aw[j], kAbsmaxFloor);
    const float sj = __double2float_rn(__ddiv_rn(pow(x, a), pow(w, 1.0 - a)));
    s[j] = sj;
    if (s_inv != nullptr) s_inv[j] = __fdiv_rn(1.0f, sj);
}

sq_status smooth_scales(const float* ax, const float* aw, int64_t C, float alpha, float* s, float* s_inv,
                        cudaStream_t st) {
    smooth_scales_kernel<<<(unsigned)((C + 127) / 128), 128, 0, st>>>(ax, aw, C, alpha, s, s_inv);
    return launch_status();
}

template <typename T>
__global__ void fold_ln_kernel(const T* __restrict__ gamma, const T* __restrict__ beta,
                               const float* __restrict__ s, int64_t C, T* __restrict__ gout,
                               T* __restrict__ bout) {
    const int64_t j = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (j >= C) return;
    const float sj = s[j];
    gout[j] = Act<T>::from_float(__fdiv_rn(Act<T>::to_float(gamma[j]), sj));
    if (beta != nullptr) bout[j] = Act<T>::from_float(__fdiv_rn(Act<T>::to_float(beta[j]), sj));
}

sq_status fold_ln_weight(const void* g, const void* b, sq_dtype dt, const float* s, int64_t C,
                         void* go, void* bo, cudaStream_t st) {
    const unsigned grid = (unsigned)((C + 127) / 128);
    if (dt == SQ_F16)
        fold_ln_kernel<__half><<<grid, 128, 0, st>>>((const __half*)g, (const __half*)b, s, C,
                                                     (__half*)go, (__half*)bo);
    else
        fold_ln_kernel<__nv_bfloat16><<<grid, 128, 0, st>>>(
            (const __nv_bfloat16*)g, (const __nv_bfloat16*)b, s, C, (__nv_bfloat16*)go,
            (__nv_bfloat16*)bo);
    return launch_status();
}

// =======================================================================================
// Row kernel: one CTA (or one cluster of CTAs for very wide rows) per row -- a token, or an
// output channel of W.  The row's 16-byte vectors are spread over the threads and kept in
// registers (up to VPT per thread), so the row is read from HBM exactly once.
//   LN        : apply the folded LayerNorm first (two-pass statistics in registers)
//   HAS_MUL   : multiply by a per-column fp32 vector first (1/s, or s for weights)
//   CLUSTER   : CTAs sharing one row; partial statistics meet through distributed smem
//   mode      : how the step size is obtained, see RowMode
// =======================================================================================
template <bool IS_MAX, int CLUSTER>
__device__ __forceinline__ float row_reduce(float v, float* red, float* xchg) {
    v = block_reduce<IS_MAX>(v, red);
    if (CLUSTER > 1) {
        cg::cluster_group cluster = cg::this_cluster();
        cluster.sync();  // every CTA of the row is done reading the previous exchange value
        if (threadIdx.x == 0) *xchg = v;
        cluster.sync();
        float r = IS_MAX ? 0.0f : 0.0f;
#pragma unroll
        for (int i = 0; i < CLUSTER; ++i) {  // same order in every CTA: identical result
            const float o = *cluster.map_shared_rank(xchg, i);
            r = IS_MAX ? fmaxf(r, o) : r + o;
        }
        v = r;
    }
    return v;
}

template <typename T, int VPT, bool LN, bool HAS_MUL, int CLUSTER>
__global__ void __launch_bounds__(VPT <= 4 ? 256 : 512)
row_quant_kernel(const T* __restrict__ X, int64_t M, int64_t C, const float* __restrict__ col_mul,
                 const T* __restrict__ gamma, const T* __restrict__ beta, float eps, int mode,
                 int8_t* __restrict__ Xq, float* __restrict__ scale, float* __restrict__ absmax_word,
                 float* __restrict__ stats /*[2M]: mu, rstd*/, int stats_are_input) {
    __shared__ float red[33];
    __shared__ float xchg;
    const int64_t row = blockIdx.x / CLUSTER;
    const int rank = blockIdx.x % CLUSTER;
    const int nvec_row = (int)(C >> 3);
    // this CTA's slice of the row's vectors
    const int per_cta = (nvec_row + CLUSTER - 1) / CLUSTER;
    const int v_begin = rank * per_cta;
    const int nvec = max(0, min(per_cta, nvec_row - v_begin));
    const int tid = threadIdx.x, nthr = blockDim.x;
    const uint4* xrow = reinterpret_cast<const uint4*>(X + row * C) + v_begin;
    const bool lead = rank == 0 && tid == 0;

    uint4 raw[VPT];
#pragma unroll
    for (int i = 0; i < VPT; ++i) {
        const int v = tid + i * nthr;
        raw[i] = v < nvec ? __ldcs(xrow + v) : make_uint4(0u, 0u, 0u, 0u);
    }

    float mu = 0.0f, rstd = 1.0f;
    if (LN) {
        if (stats_are_input) {
            mu = stats[2 * row];
            rstd = stats[2 * row + 1];
        } else {
            float s = 0.0f;
#pragma unroll
            for (int i = 0; i < VPT; ++i) {
                float f[8];
                unpack8<T>(raw[i], f);  // zero-filled vectors add nothing
                s += ((f[0] + f[1]) + (f[2] + f[3])) + ((f[4] + f[5]) + (f[6] + f[7]));
            }
            mu = row_reduce<false, CLUSTER>(s, red, &xchg) / (float)C;
            float ss = 0.0f;
#pragma unroll
            for (int i = 0; i < VPT; ++i) {
                if (tid + i * nthr < nvec) {
                    float f[8];
                    unpack8<T>(raw[i], f);
#pragma unroll
                    for (int k = 0; k < 8; ++k) {
                        const float d = f[k] - mu;
                        ss = fmaf(d, d, ss);
                    }
                }
            }
            const float var = row_reduce<false, CLUSTER>(ss, red, &xchg) / (float)C;
            rstd = __fdiv_rn(1.0f, __fsqrt_rn(var + eps));
            if (stats != nullptr && lead) {
                stats[2 * row] = mu;
                stats[2 * row + 1] = rstd;
            }
        }
    }

    // values of this thread's vector i, after LayerNorm / column multiplier
    auto transform = [&](int i, float (&f)[8]) {
        unpack8<T>(raw[i], f);
        const int v = v_begin + tid + i * nthr;
        if (LN) {
            const uint4 g4 = __ldg(reinterpret_cast<const uint4*>(gamma) + v);
            float g[8], b[8];
            unpack8<T>(g4, g);
            if (beta != nullptr) {
                const uint4 b4 = __ldg(reinterpret_cast<const uint4*>(beta) + v);
                unpack8<T>(b4, b);
            } else {
#pragma unroll
                for (int k = 0; k < 8; ++k) b[k] = 0.0f;
            }
            const float shift = -__fmul_rn(mu, rstd);
#pragma unroll
            for (int k = 0; k < 8; ++k) f[k] = __fmaf_rn(__fmaf_rn(f[k], rstd, shift), g[k], b[k]);
        }
        if (HAS_MUL) {
            const float4 m0 = __ldg(reinterpret_cast<const float4*>(col_mul) + 2 * v);
            const float4 m1 = __ldg(reinterpret_cast<const float4*>(col_mul) + 2 * v + 1);
            f[0] = __fmul_rn(f[0], m0.x); f[1] = __fmul_rn(f[1], m0.y);
            f[2] = __fmul_rn(f[2], m0.z); f[3] = __fmul_rn(f[3], m0.w);
            f[4] = __fmul_rn(f[4], m1.x); f[5] = __fmul_rn(f[5], m1.y);
            f[6] = __fmul_rn(f[6], m1.z); f[7] = __fmul_rn(f[7], m1.w);
        }
    };

    float delta;
    if (mode == ROW_DYNAMIC || mode == ROW_ABSMAX_ONLY) {
        float m = 0.0f;
        if (!LN && !HAS_MUL) {
            uint32_t pm = 0u;  // packed running max of |x|: exact in fp16/bf16
#pragma unroll
            for (int i = 0; i < VPT; ++i) {
                pm = Act<T>::absmax2(pm, raw[i].x); pm = Act<T>::absmax2(pm, raw[i].y);
                pm = Act<T>::absmax2(pm, raw[i].z); pm = Act<T>::absmax2(pm, raw[i].w);
            }
            m = Act<T>::hmax_of2(pm);
        } else {
#pragma unroll
            for (int i = 0; i < VPT; ++i) {
                if (tid + i * nthr < nvec) {
                    float f[8];
                    transform(i, f);
#pragma unroll
                    for (int k = 0; k < 8; ++k) m = fmaxf(m, fabsf(f[k]));
                }
            }
        }
        m = row_reduce<true, CLUSTER>(m, red, &xchg);
        if (mode == ROW_ABSMAX_ONLY) {
            if (lead) atomic_max_nonneg(absmax_word, m);
            if (CLUSTER > 1) cg::this_cluster().sync();  // peers may still read this CTA's smem
            return;
        }
        delta = step_size(m);
        if (lead) scale[row] = delta;
    } else if (mode == ROW_GIVEN_SCALE) {
        delta = __ldg(scale);
    } else if (mode == ROW_GIVEN_ROW_ABSMAX) {
        delta = step_size(__ldg(absmax_word + row));
        if (lead) scale[row] = delta;
    } else {  // ROW_FROM_ABSMAX_WORD
        delta = step_size(__ldg(absmax_word));
        if (row == 0 && lead) scale[0] = delta;
    }
    const float inv = recip_step(delta);

    uint2* qrow = reinterpret_cast<uint2*>(Xq + row * C) + v_begin;
#pragma unroll
    for (int i = 0; i < VPT; ++i) {
        const int v = tid + i * nthr;
        if (v < nvec) {
            float f[8];
            transform(i, f);
            __stcs(qrow + v, quant8(f, inv));
        }
    }
    if (CLUSTER > 1) cg::this_cluster().sync();  // keep smem alive until every peer has read it
}

template <typename T, int VPT, bool LN, bool HAS_MUL, int CLUSTER>
static void launch_row_kernel(int64_t M, int threads, cudaStream_t st, const T* x, int64_t C,
                              const float* col_mul, const T* g, const T* b, float eps, int mode,
                              int8_t* Xq, float* scale, float* absmax_word, float* stats,
                              int stats_are_input) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)(M * CLUSTER));
    cfg.blockDim = dim3((unsigned)threads);
    cfg.dynamicSmemBytes = 0;
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = CLUSTER;
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    cfg.attrs = attr;
    cfg.numAttrs = CLUSTER > 1 ? 1 : 0;
    cudaLaunchKernelEx(&cfg, row_quant_kernel<T, VPT, LN, HAS_MUL, CLUSTER>, x, M, C, col_mul, g, b, eps,
                       mode, Xq, scale, absmax_word, stats, stats_are_input);
}

template <typename T, bool LN, bool HAS_MUL>
static sq_status launch_rows(const void* X, int64_t M, int64_t C, const float* col_mul,
                             const void* gamma, const void* beta, float eps, int mode, int8_t* Xq,
                             float* scale, float* absmax_word, float* stats, int stats_are_input,
                             cudaStream_t st) {
    const int64_t nvec = C / 8;
    const T* x = static_cast<const T*>(X);
    const T* g = static_cast<const T*>(gamma);
    const T* b = static_cast<const T*>(beta);
#define SQ_LAUNCH(V, CL, THREADS)                                                               \
    launch_row_kernel<T, V, LN, HAS_MUL, CL>(M, THREADS, st, x, C, col_mul, g, b, eps, mode, Xq, \
                                             scale, absmax_word, stats, stats_are_input)
    // 256-thread CTAs for ordinary rows (several rows resident per SM), 512 for wide ones,
    // a cluster of 2 or 4 CTAs beyond 65536 elements
    if (nvec <= 512) {
        const int threads = (int)std::max<int64_t>(32, ((nvec + 1) / 2 + 31) / 32 * 32);
        SQ_LAUNCH(2, 1, threads);
    } else if (nvec <= 1024) SQ_LAUNCH(4, 1, 256);
    else if (nvec <= 4096) SQ_LAUNCH(8, 1, 512);
    else if (nvec <= 8192) SQ_LAUNCH(16, 1, 512);
    else if (nvec <= 16384) SQ_LAUNCH(16, 2, 512);
    else if (nvec <= 32768) SQ_LAUNCH(16, 4, 512);
    else return SQ_ERR_UNSUPPORTED;  // rows wider than 262144 elements
#undef SQ_LAUNCH
    return launch_status();
}

// An empty kernel launched WITHOUT the programmatic-serialisation attribute: it starts only when
// everything queued before it on the stream has completed and is visible.  Placed after a kernel
// whose output a later dependent launch reads BEFORE its programmatic-dependency wait (the
// decode-shaped GEMM prefetches weights that early), it closes that window.
__global__ void full_dependency_kernel() {}

sq_status stream_full_dependency(cudaStream_t st) {
    full_dependency_kernel<<<1, 32, 0, st>>>();
    return launch_status();
}

sq_status row_quant(const void* X, sq_dtype dt, int64_t M, int64_t C, const float* col_mul,
                    const void* gamma, const void* beta, float eps, bool ln, int mode, int8_t* Xq,
                    float* scale, float* absmax_word, float* stats, int stats_are_input,
                    uint32_t* status, cudaStream_t st) {
    // the bulk-copy pipeline takes rows up to 32 768 elements (81 920 for the plain quantiser);
    // LayerNorm never comes with a column multiplier
    if (row_pipeline_supports(M, C, ln, col_mul != nullptr) && !(ln && col_mul != nullptr))
        return row_pipeline(X, dt, M, C, col_mul, gamma, beta, eps, ln, mode, Xq, scale, absmax_word, stats,
                            stats_are_input, status, st);
#define SQ_DISPATCH(T)                                                                           \
    (ln ? launch_rows<T, true, false>(X, M, C, nullptr, gamma, beta, eps, mode, Xq, scale,       \
                                      absmax_word, stats, stats_are_input, st)                   \
        : (col_mul ? launch_rows<T, false, true>(X, M, C, col_mul, nullptr, nullptr, 0.f, mode,  \
                                                 Xq, scale, absmax_word, nullptr, 0, st)         \
                   : launch_rows<T, false, false>(X, M, C, nullptr, nullptr, nullptr, 0.f, mode, \
                                                  Xq, scale, absmax_word, nullptr, 0, st)))
    return dt == SQ_F16 ? SQ_DISPATCH(__half) : SQ_DISPATCH(__nv_bfloat16);
#undef SQ_DISPATCH
}

// =======================================================================================
// Attention plumbing: causal softmax + fixed-step quantisation of P; residual add.
// One warp per score row; the row (S <= 4096) is held in registers.
// =======================================================================================
template <typename T, int VPL>
__global__ void __launch_bounds__(256)
softmax_quant_p_kernel(const T* __restrict__ scores, int64_t n_rows, int S, int8_t* __restrict__ Pq) {
    const int lane = threadIdx.x & 31;
    const int64_t r = (int64_t)blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
    if (r >= n_rows) return;
    const int i = (int)(r % S);  // query position: keys j <= i are visible
    const uint4* srow = reinterpret_cast<const uint4*>(scores + r * S);
    const int nvec = S >> 3;
    // Only the vectors that hold a visible key (8 * vi <= i) are loaded and exponentiated; the
    // rest of the row is written as zeros.  exp(s - max) is evaluated as exp2(s * log2(e) -
    // max * log2(e)) and the division by the row sum as one reciprocal per row.
    float f[VPL][8];
    float mx = -INFINITY;
#pragma unroll
    for (int v = 0; v < VPL; ++v) {
        const int vi = lane + 32 * v;
        if (vi < nvec && vi * 8 <= i) {
            unpack8<T>(__ldcs(srow + vi), f[v]);
#pragma unroll
            for (int k = 0; k < 8; ++k) {
                if (vi * 8 + k > i) f[v][k] = -INFINITY;
                mx = fmaxf(mx, f[v][k]);
            }
        }
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, o));
    const float kLog2e = 1.4426950408889634f;
    const float shift = -mx * kLog2e;
    float sum = 0.0f;
#pragma unroll
    for (int v = 0; v < VPL; ++v) {
        const int vi = lane + 32 * v;
        if (vi < nvec && vi * 8 <= i) {
#pragma unroll
            for (int k = 0; k < 8; ++k) {
                f[v][k] = exp2f(fmaf(f[v][k], kLog2e, shift));  // exp2(-inf) = 0 for masked positions
                sum += f[v][k];
            }
        }
    }
    sum = warp_sum(sum);
    const float inv = __fdiv_rn(1.0f, sum);
    uint2* prow = reinterpret_cast<uint2*>(Pq + r * S);
#pragma unroll
    for (int v = 0; v < VPL; ++v) {
        const int vi = lane + 32 * v;
        if (vi < nvec) {
            if (vi * 8 <= i) {
                float p[8];
#pragma unroll
                for (int k = 0; k < 8; ++k) p[k] = f[v][k] * inv;
                __stcs(prow + vi, quant8<false>(p, 127.0f));  // p <= 1: the code cannot exceed 127
            } else {
                __stcs(prow + vi, make_uint2(0u, 0u));
            }
        }
    }
}

sq_status softmax_quant_p(const void* scores, sq_dtype dt, int64_t n_mat, int64_t S, int8_t* Pq,
                          cudaStream_t st) {
    const int64_t n_rows = n_mat * S;
    const int vpl = (int)((S / 8 + 31) / 32);
    if (vpl > 16) return SQ_ERR_UNSUPPORTED;  // S > 4096
    const unsigned grid = (unsigned)((n_rows + 7) / 8);
#define SQ_SM(T, V) softmax_quant_p_kernel<T, V><<<grid, 256, 0, st>>>((const T*)scores, n_rows, (int)S, Pq)
#define SQ_SM_T(T)                                                                        \
    do {                                                                                  \
        if (vpl <= 1) SQ_SM(T, 1); else if (vpl <= 2) SQ_SM(T, 2); else if (vpl <= 4) SQ_SM(T, 4); \
        else if (vpl <= 8) SQ_SM(T, 8); else SQ_SM(T, 16);                                \
    } while (0)
    if (dt == SQ_F16) SQ_SM_T(__half); else SQ_SM_T(__nv_bfloat16);
#undef SQ_SM_T
#undef SQ_SM
    return launch_status();
}

template <typename T>
__global__ void residual_add_kernel(const uint4* __restrict__ a, const uint4* __restrict__ b,
                                    int64_t nvec, uint4* __restrict__ out) {
    pdl_wait();  // a and b come from the kernels in front
    pdl_launch_dependents();
    for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < nvec;
         i += (int64_t)gridDim.x * blockDim.x) {
        float fa[8], fb[8];
        unpack8<T>(a[i], fa);
        unpack8<T>(b[i], fb);
        __align__(16) T r[8];
#pragma unroll
        for (int k = 0; k < 8; ++k) r[k] = Act<T>::from_float(__fadd_rn(fa[k], fb[k]));
        out[i] = *reinterpret_cast<uint4*>(r);
    }
}

// Eq. 2 on a matrix of INT32 accumulators that already sits in memory: the epilogue of the GEMM
// kernels as a pass of its own.  Tensor-parallel row-parallel layers need it: every rank's GEMM
// leaves raw partial sums, the ranks add them exactly as integers, and the sum is dequantised once.
// Same arithmetic, operation for operation, as the fused epilogues.  One thread = 8 columns.
template <typename T>
__global__ void __launch_bounds__(256)
dequant_acc_kernel(const DequantArgs a) {
    pdl_wait();
    pdl_launch_dependents();
    const int64_t nvec = a.N >> 3;
    const int64_t total = a.M * nvec;
    for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < total; i += (int64_t)gridDim.x * blockDim.x) {
        const int64_t row = i / nvec, col = (i - row * nvec) << 3;
        const int4* src = reinterpret_cast<const int4*>(a.acc + row * a.ld_acc + col);
        const int4 lo = __ldcs(src), hi = __ldcs(src + 1);
        const int32_t acc[8] = {lo.x, lo.y, lo.z, lo.w, hi.x, hi.y, hi.z, hi.w};
        const float xs = __ldg(a.x_scale + (a.x_per_row ? row : 0));
        float y[8];
#pragma unroll
        for (int k = 0; k < 8; ++k) {
            const float ws = __ldg(a.w_scale + (a.w_per_col ? col + k : 0));
            const float bs = a.bias == nullptr ? 0.0f
                             : (a.bias_dt == SQ_BF16 ? __bfloat162float(static_cast<const __nv_bfloat16*>(a.bias)[col + k])
                                                     : __half2float(static_cast<const __half*>(a.bias)[col + k]));
            float v = __fmaf_rn(__int2float_rn(acc[k]), __fmul_rn(xs, ws), bs);
            if (a.relu) v = fmaxf(v, 0.0f);
            y[k] = v;
        }
        if (a.out_dt == SQ_I8) {
            uint32_t c[8];
#pragma unroll
            for (int k = 0; k < 8; ++k) c[k] = quant_code(y[k], __ldg(a.requant_mul + (a.requant_per_col ? col + k : 0)));
            *reinterpret_cast<uint2*>(static_cast<int8_t*>(a.Y) + row * a.ldy + col) =
                make_uint2(pack4(c[0], c[1], c[2], c[3]), pack4(c[4], c[5], c[6], c[7]));
        } else {
            if (a.residual != nullptr) {  // round to the output type, then the residual add (rounded by the store)
                float r[8];
                unpack8<T>(__ldg(reinterpret_cast<const uint4*>(static_cast<const T*>(a.residual) + row * a.ld_res + col)), r);
#pragma unroll
                for (int k = 0; k < 8; ++k) y[k] = __fadd_rn(Act<T>::to_float(Act<T>::from_float(y[k])), r[k]);
            }
            __align__(16) T o[8];
#pragma unroll
            for (int k = 0; k < 8; ++k) o[k] = Act<T>::from_float(y[k]);
            *reinterpret_cast<uint4*>(static_cast<T*>(a.Y) + row * a.ldy + col) = *reinterpret_cast<const uint4*>(o);
        }
    }
}

sq_status dequant_acc(const DequantArgs& a, cudaStream_t st) {
    const int64_t total = a.M * (a.N >> 3);
    const unsigned grid = (unsigned)std::min<int64_t>((total + 255) / 256, 16LL * sm_count());
    if (a.out_dt == SQ_BF16)
        return launch_pdl(dequant_acc_kernel<__nv_bfloat16>, dim3(grid), dim3(256), 0, st, 1, a);
    return launch_pdl(dequant_acc_kernel<__half>, dim3(grid), dim3(256), 0, st, 1, a);  // also SQ_I8 (T unused there)
}

sq_status residual_add(const void* a, const void* b, sq_dtype dt, int64_t n, void* out,
                       cudaStream_t st) {
    const int64_t nvec = n / 8;
    const unsigned grid = (unsigned)std::min<int64_t>((nvec + 255) / 256, 8LL * sm_count());
    if (dt == SQ_F16)
        return launch_pdl(residual_add_kernel<__half>, dim3(grid), dim3(256), 0, st, 1, (const uint4*)a, (const uint4*)b, nvec,
                          (uint4*)out);
    return launch_pdl(residual_add_kernel<__nv_bfloat16>, dim3(grid), dim3(256), 0, st, 1, (const uint4*)a, (const uint4*)b,
                      nvec, (uint4*)out);
}

}  // namespace sq
