// Generation-stage attention over an INT8 key/value cache, and the kernel that fills the cache.
//
// The paper's Discussion notes that quantised activations also shrink the KV cache; in the
// precision mapping of Fig. 6 the newest token's attention is then
//     s_j = (q . K_j) * alpha_qk  (INT8 x INT8 -> INT32),  p = softmax(s),  P_j = round(127 p_j),
//     out = (sum_j P_j V_j) * alpha_pv  (INT8 x INT8 -> INT32)  -> INT8 or 16-bit float.
// One query row per (sequence, head) makes this a pair of matrix-vector products: 2 * L * d bytes
// of cache are read for 4 * L * d integer operations, so the kernel is bound by HBM, not by the
// tensor cores, and is built around keeping bulk copies in flight:
//   * K cache [B, H, L_max, 128]: one key per 128-byte row.  V cache [B, H, L_max/4, 128, 4]: four
//     consecutive positions of one channel share a 32-bit word, which is exactly the operand
//     dp4a wants for a reduction over positions -- no transposition at read time.
//   * every warp owns a private ring of 4 KB stages fed by cp.async.bulk (32 keys per stage,
//     completion on an mbarrier, bounded waits); its stream of tiles runs through its K tiles
//     and straight on into its V tiles, so V is already arriving while the softmax is computed.
//   * a sequence can be split over a thread-block cluster (1..8 CTAs): the CTAs exchange the
//     integer score maximum, the exponential sums and the INT32 partial outputs through
//     distributed shared memory.  Integer partials add exactly; the exponential sum is taken in
//     rank order, so a given launch configuration is deterministic.
// Tried and measured slower: taking the grid's batch index as a rank in the order of decreasing
// length (longest streams first, so that the last wave holds the shortest) -- the rank costs every
// CTA three barriers and a pass over the lengths, more than the evened tail returns (batch 16:
// 103 -> 106 us, batch 64: 355 -> 368 us).
#include <climits>

#include "sq_common.cuh"
#include "sq_bulk.cuh"
#include "sq_kernels.h"

namespace sq {

namespace {

constexpr int KV_D = 128;                    // head dimension (bytes per key row)
constexpr int KV_TILE = 32;                  // keys per ring stage
constexpr int KV_TILE_BYTES = KV_TILE * KV_D;
constexpr int KV_WARPS = 4;
constexpr int KV_THREADS = KV_WARPS * 32;
#ifndef SQ_KV_STAGES  // tuning builds may override it: python -m paper_2211_10438_b200.build --variant NAME -DSQ_KV_STAGES=4
#define SQ_KV_STAGES 2
#endif
constexpr int KV_STAGES = SQ_KV_STAGES;                 // ring stages per warp (two: four to six CTAs fit an SM, by the score buffer; deeper rings with fewer CTAs measured slower)
constexpr int KV_MAX_CLUSTER = 8;
constexpr float kLog2e = 1.4426950408889634f;

using namespace bulk;
__device__ __forceinline__ uint32_t cluster_rank() {
    uint32_t r;
    asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
    return r;
}
// every thread of every CTA of the cluster; orders shared-memory writes before it against reads after it
__device__ __forceinline__ void cluster_sync() {
    asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory");
    asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");
}
// the 32-bit word at the same shared-memory offset in CTA `rank` of this cluster
__device__ __forceinline__ uint32_t ld_cluster_u32(const void* local, uint32_t rank) {
    uint32_t remote, v;
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(remote) : "r"(smem_u32(local)), "r"(rank));
    asm volatile("ld.shared::cluster.u32 %0, [%1];" : "=r"(v) : "r"(remote) : "memory");
    return v;
}
__device__ __forceinline__ float ex2_approx(float x) {
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}

struct KvParams {
    const int8_t* q;        // [B, ldq]; head h at columns h*128 ..
    int64_t ldq;
    int8_t* kc;             // [B, H, lmax, 128]
    int8_t* vc;             // [B, H, lmax/4, 128, 4]
    const int8_t* k_new;    // nullable: [B, ld_new] k / v codes of the newest token, not yet cached;
    const int8_t* v_new;    // head h at columns h*128 ..
    int64_t ld_new;
    const int32_t* lens;    // [B]
    int64_t lmax;
    int H;
    int max_len;            // host-known upper bound of lens[]
    int cap;                // keys one CTA can hold (multiple of 32)
    int cluster;
    float c1;               // alpha_qk * log2(e)
    float alpha_pv;
    const float* requant_mul;
    void* out;
    int out_dt;
    int64_t ldo;
    uint32_t* status;
};

__host__ __device__ constexpr size_t kv_smem_bytes(int cap) {
    return (size_t)KV_WARPS * KV_STAGES * KV_TILE_BYTES  // rings
           + (size_t)cap * 4                              // INT32 scores, then fp32 exponentials
           + (size_t)cap                                  // P codes
           + KV_D                                         // q
           + (size_t)KV_WARPS * KV_D * 4                  // per-warp INT32 partial outputs
           + (size_t)KV_D * 4                             // this CTA's partial output
           + (size_t)KV_WARPS * KV_STAGES * 8             // mbarriers
           + 64;                                          // per-warp scratch, exchanged scalars
}

__global__ void __launch_bounds__(KV_THREADS)
kv_decode_attention_kernel(const KvParams p) {
    extern __shared__ __align__(128) uint8_t smem[];
    uint8_t* ring = smem;
    int32_t* scores = reinterpret_cast<int32_t*>(ring + KV_WARPS * KV_STAGES * KV_TILE_BYTES);
    uint32_t* pbar = reinterpret_cast<uint32_t*>(scores + p.cap);
    uint8_t* q_s = reinterpret_cast<uint8_t*>(pbar) + p.cap;
    int32_t* wpart = reinterpret_cast<int32_t*>(q_s + KV_D);
    int32_t* x_part = wpart + KV_WARPS * KV_D;
    uint64_t* bars = reinterpret_cast<uint64_t*>(x_part + KV_D);
    uint32_t* wred = reinterpret_cast<uint32_t*>(bars + KV_WARPS * KV_STAGES);  // [KV_WARPS]
    int32_t* x_max = reinterpret_cast<int32_t*>(wred + KV_WARPS);
    float* x_sum = reinterpret_cast<float*>(x_max + 1);

    const int tid = threadIdx.x, lane = tid & 31, w = tid >> 5;
    const uint32_t crank = cluster_rank();
    const int C = p.cluster;
    const int h = blockIdx.y, b = blockIdx.z;

    if (tid == 0) {
        for (int i = 0; i < KV_WARPS * KV_STAGES; ++i) mbar_init(bars + i, 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    pdl_wait();  // q, the cache and the lengths may come from the preceding launch
    pdl_launch_dependents();
    // Everything this CTA reads besides the cache is requested here, at once: the sequence length, the new
    // token's key and value rows, the re-quantisation factor.  Read where they are used, each of them is a
    // dependent trip to L2 or HBM (about a microsecond) on a path that is nothing but latency at short contexts.
    const size_t new_off = (size_t)b * p.ld_new + (size_t)h * KV_D;
    uint4 k_new_row = make_uint4(0u, 0u, 0u, 0u);
    uint32_t v_new_word = 0u;
    int8_t v_new_byte = 0;
    if (p.k_new != nullptr) {
        if (w == 0 && lane < KV_D / 16) k_new_row = __ldg(reinterpret_cast<const uint4*>(p.k_new + new_off) + lane);
        if (w == 0) v_new_word = __ldg(reinterpret_cast<const uint32_t*>(p.v_new + new_off) + lane);
        v_new_byte = __ldg(p.v_new + new_off + tid);
    }
    const float requant = (p.out_dt == SQ_I8 && crank == 0) ? __ldg(p.requant_mul) : 1.0f;
    int len = __ldg(p.lens + b);
    const bool truncated = len > p.max_len;
    if (truncated) {  // the caller's bound was wrong: say so, and stay inside what was sized
        if (tid == 0 && crank == 0) atomicCAS(p.status, 0u, (uint32_t)SQ_ERR_SHAPE | (40u << 8));
        len = p.max_len;
    }
    const size_t out_off = (size_t)b * p.ldo + (size_t)h * KV_D + tid;
    if (len <= 0) {  // nothing cached: define the output as zero (same branch in every CTA of the cluster)
        if (crank == 0) {
            if (p.out_dt == SQ_I8) reinterpret_cast<int8_t*>(p.out)[out_off] = 0;
            else reinterpret_cast<uint16_t*>(p.out)[out_off] = 0;
        }
        return;
    }
    if (tid < KV_D / 16)
        reinterpret_cast<uint4*>(q_s)[tid] = __ldg(reinterpret_cast<const uint4*>(p.q + (size_t)b * p.ldq + (size_t)h * KV_D) + tid);

    // this CTA's share of the positions, in whole tiles
    const int chunk = ((len + C - 1) / C + KV_TILE - 1) / KV_TILE * KV_TILE;
    const int key0 = (int)crank * chunk;
    const int n = max(0, min(len - key0, chunk));
    // With k_new / v_new the newest position (len - 1) is not in the cache yet: the CTA that owns
    // it takes its key and value from the new rows, stores them for later steps, and streams only
    // the positions before it.  A truncated sequence appends nothing: position max_len - 1 holds a
    // valid earlier key and value, which the newest token's must not overwrite; the output is then
    // the attention over the first max_len cached positions.
    const bool owns_new = !truncated && p.k_new != nullptr && n > 0 && key0 + n == len;
    const int nc = owns_new ? n - 1 : n;  // positions of this CTA that come from the cache
    const int nt = (nc + KV_TILE - 1) / KV_TILE;
    const int ntw = nt > w ? (nt - w + KV_WARPS - 1) / KV_WARPS : 0;  // tiles of this warp, per operand
    const int total = 2 * ntw;                                        // K tiles, then V tiles
    const size_t base = (((size_t)b * p.H + h) * (size_t)p.lmax + (size_t)key0) * KV_D;
    uint8_t* my_ring = ring + (size_t)w * KV_STAGES * KV_TILE_BYTES;
    uint64_t* my_bars = bars + w * KV_STAGES;
    __syncthreads();  // barriers initialised, q in place

    auto issue = [&](int u) {  // lane 0: start the copy of this warp's u-th tile
        const bool is_v = u >= ntw;
        const int t = w + KV_WARPS * (is_v ? u - ntw : u);
        const int rows = min(KV_TILE, nc - KV_TILE * t);
        const uint32_t bytes = is_v ? (uint32_t)((rows + 3) / 4) * 4u * KV_D : (uint32_t)rows * KV_D;
        const int8_t* src = (is_v ? p.vc : p.kc) + base + (size_t)t * KV_TILE_BYTES;
        const int slot = u % KV_STAGES;
        mbar_expect_tx(my_bars + slot, bytes);
        bulk_load(my_ring + (size_t)slot * KV_TILE_BYTES, src, bytes, my_bars + slot);
    };
    auto wait_tile = [&](int u) -> bool {  // warp-uniform result
        uint32_t ok = 1;
        if (lane == 0) {
            ok = mbar_wait_bounded(my_bars + (u % KV_STAGES), (uint32_t)(u / KV_STAGES) & 1u) ? 1u : 0u;
            if (!ok) atomicCAS(p.status, 0u, (uint32_t)SQ_ERR_TIMEOUT | (41u << 8));
        }
        return __shfl_sync(0xffffffffu, ok, 0) != 0;
    };
    if (lane == 0)
        for (int u = 0; u < min(KV_STAGES, total); ++u) issue(u);

    // ---- phase 1: scores of this CTA's keys (lane = key of the tile), running integer maximum ----
    bool ok = true;
    int vmax = INT_MIN;
    for (int u = 0; u < ntw; ++u) {
        if (!(ok = wait_tile(u))) break;
        const int t = w + KV_WARPS * u;
        const int rows = min(KV_TILE, nc - KV_TILE * t);
        const uint8_t* row = my_ring + (size_t)(u % KV_STAGES) * KV_TILE_BYTES + lane * KV_D;
        int acc = 0;
#pragma unroll
        for (int i = 0; i < KV_D / 16; ++i) {
            const int pc = i ^ (lane & 7);  // rotate the pieces across lanes: conflict-free 16-byte reads
            const uint4 kv = *reinterpret_cast<const uint4*>(row + pc * 16);
            const uint4 qv = *reinterpret_cast<const uint4*>(q_s + pc * 16);
            acc = __dp4a((int)kv.x, (int)qv.x, acc);
            acc = __dp4a((int)kv.y, (int)qv.y, acc);
            acc = __dp4a((int)kv.z, (int)qv.z, acc);
            acc = __dp4a((int)kv.w, (int)qv.w, acc);
        }
        if (lane < rows) {
            scores[KV_TILE * t + lane] = acc;
            vmax = max(vmax, acc);
        }
        __syncwarp();
        if (lane == 0 && u + KV_STAGES < total) issue(u + KV_STAGES);
    }
    if (owns_new && w == 0) {  // score of the newest position from its own key row
        int acc = 0;
        if (lane < KV_D / 16) {
            const uint4 kv = k_new_row;
            const uint4 qv = *reinterpret_cast<const uint4*>(q_s + lane * 16);
            acc = __dp4a((int)kv.x, (int)qv.x, acc);
            acc = __dp4a((int)kv.y, (int)qv.y, acc);
            acc = __dp4a((int)kv.z, (int)qv.z, acc);
            acc = __dp4a((int)kv.w, (int)qv.w, acc);
            // and the key row goes into the cache for the steps to come
            *reinterpret_cast<uint4*>(p.kc + ((((size_t)b * p.H + h) * (size_t)p.lmax + (size_t)(len - 1)) * KV_D) + lane * 16) = kv;
        }
        acc = __reduce_add_sync(0xffffffffu, acc);
        if (lane == 0) scores[nc] = acc;
        vmax = max(vmax, acc);
    }
    vmax = __reduce_max_sync(0xffffffffu, vmax);
    if (lane == 0) wred[w] = (uint32_t)vmax;
    __syncthreads();
    if (tid == 0) {
        int m = (int)wred[0];
        for (int i = 1; i < KV_WARPS; ++i) m = max(m, (int)wred[i]);
        *x_max = m;
    }
    cluster_sync();
    int gmax = INT_MIN;
    for (int r = 0; r < C; ++r) gmax = max(gmax, (int)ld_cluster_u32(x_max, (uint32_t)r));

    // ---- softmax numerators and their sum ----
    const float m2 = p.c1 * __int2float_rn(gmax);
    float* ex = reinterpret_cast<float*>(scores);
    float part = 0.0f;
    for (int j = tid; j < n; j += KV_THREADS) {
        const float e = ex2_approx(fmaf(__int2float_rn(scores[j]), p.c1, -m2));
        ex[j] = e;
        part += e;
    }
    part = warp_sum(part);
    if (lane == 0) wred[w] = __float_as_uint(part);
    __syncthreads();
    if (tid == 0) {
        float s = __uint_as_float(wred[0]);
        for (int i = 1; i < KV_WARPS; ++i) s += __uint_as_float(wred[i]);
        *x_sum = s;
    }
    cluster_sync();
    float l = 0.0f;
    for (int r = 0; r < C; ++r) l += __uint_as_float(ld_cluster_u32(x_sum, (uint32_t)r));  // rank order
    const float k127 = __fdiv_rn(127.0f, l);  // P = round(127 * e / l)
    for (int g = tid; g < nt * (KV_TILE / 4); g += KV_THREADS) {  // four positions per word; zero beyond nc
        uint32_t c[4];
#pragma unroll
        for (int e = 0; e < 4; ++e) {
            const int j = 4 * g + e;
            c[e] = j < nc ? quant_code<false>(ex[j], k127) : 0u;  // e <= l: the code cannot exceed 127
        }
        pbar[g] = pack4(c[0], c[1], c[2], c[3]);
    }
    const int p_new = owns_new ? (int)(quant_code<false>(ex[nc], k127) & 0xffu) : 0;
    __syncthreads();

    // ---- phase 2: partial outputs; lane owns channels 4*lane .. 4*lane+3 ----
    int o[4] = {0, 0, 0, 0};
    for (int u = ntw; ok && u < total; ++u) {
        if (!(ok = wait_tile(u))) break;
        const int t = w + KV_WARPS * (u - ntw);
        const int ng = (min(KV_TILE, nc - KV_TILE * t) + 3) / 4;
        const uint8_t* tile = my_ring + (size_t)(u % KV_STAGES) * KV_TILE_BYTES + lane * 16;
        const uint32_t* pw = pbar + t * (KV_TILE / 4);
#pragma unroll 4
        for (int g = 0; g < ng; ++g) {
            const uint4 vv = *reinterpret_cast<const uint4*>(tile + g * 4 * KV_D);
            const int pg = (int)pw[g];
            o[0] = __dp4a((int)vv.x, pg, o[0]);
            o[1] = __dp4a((int)vv.y, pg, o[1]);
            o[2] = __dp4a((int)vv.z, pg, o[2]);
            o[3] = __dp4a((int)vv.w, pg, o[3]);
        }
        __syncwarp();
        if (lane == 0 && u + KV_STAGES < total) issue(u + KV_STAGES);
    }
    if (owns_new) {
        const int pos = len - 1;
        if (w == 0) {  // the newest position's share of the output, from its own value row
            const uint32_t vw = v_new_word;
#pragma unroll
            for (int k = 0; k < 4; ++k) o[k] += p_new * (int)(int8_t)((vw >> (8 * k)) & 0xffu);
        }
        // value row -> cache: channel tid, byte (pos % 4) of its 4-position word
        p.vc[(((size_t)b * p.H + h) * (size_t)p.lmax + (size_t)(pos & ~3)) * KV_D + (size_t)tid * 4 + (pos & 3)] =
            v_new_byte;
    }
    *reinterpret_cast<int4*>(wpart + w * KV_D + 4 * lane) = make_int4(o[0], o[1], o[2], o[3]);
    __syncthreads();
    {
        int s = wpart[tid];
#pragma unroll
        for (int i = 1; i < KV_WARPS; ++i) s += wpart[i * KV_D + tid];
        x_part[tid] = s;
    }
    cluster_sync();
    if (crank == 0) {
        int tot = 0;
        for (int r = 0; r < C; ++r) tot += (int)ld_cluster_u32(x_part + tid, (uint32_t)r);
        const float y = __fmul_rn(__int2float_rn(tot), p.alpha_pv);
        if (p.out_dt == SQ_I8)
            reinterpret_cast<int8_t*>(p.out)[out_off] = (int8_t)(quant_code(y, requant) & 0xffu);
        else if (p.out_dt == SQ_F16)
            reinterpret_cast<__half*>(p.out)[out_off] = __float2half_rn(y);
        else
            reinterpret_cast<__nv_bfloat16*>(p.out)[out_off] = __float2bfloat16_rn(y);
    }
    if (C > 1) cluster_sync();  // rank 0 has read every partial before any CTA of the cluster leaves
}

// Moves keys and values of T tokens per sequence from the fused QKV code buffer into the cache:
// a warp handles four consecutive cache positions of one (sequence, head); lane = four channels.
__global__ void __launch_bounds__(256)
kv_cache_write_kernel(const int8_t* __restrict__ qkv, int64_t ld, int B, int T, int H, const int32_t* __restrict__ pos0,
                      int8_t* __restrict__ kc, int8_t* __restrict__ vc, int64_t lmax, int groups, uint32_t* status) {
    pdl_wait();
    pdl_launch_dependents();
    const int lane = threadIdx.x & 31;
    const int64_t wid = (int64_t)blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
    if (wid >= (int64_t)B * H * groups) return;
    // heads vary fastest: the warps of a CTA read neighbouring 128-byte pieces of the same QKV rows
    const int h = (int)(wid % H);
    const int gi = (int)((wid / H) % groups);
    const int b = (int)(wid / ((int64_t)groups * H));
    const int p0 = pos0 ? __ldg(pos0 + b) : 0;
    if (p0 < 0 || (int64_t)p0 + T > lmax) {  // would run off the cache: write nothing for this sequence
        if (lane == 0 && gi == 0 && h == 0) atomicCAS(status, 0u, (uint32_t)SQ_ERR_SHAPE | (42u << 8));
        return;
    }
    const int pg = p0 / 4 + gi;  // 4-position group of the cache
    const int64_t hid = (int64_t)H * KV_D;
    const size_t head = ((size_t)b * H + h) * (size_t)lmax;
    uint32_t vw[4] = {0u, 0u, 0u, 0u};
    bool valid[4];
#pragma unroll
    for (int r = 0; r < 4; ++r) {
        const int pos = 4 * pg + r;
        valid[r] = pos >= p0 && pos < p0 + T;
        if (valid[r]) {
            const int8_t* src = qkv + ((int64_t)b * T + (pos - p0)) * ld + hid + (int64_t)h * KV_D + 4 * lane;
            const uint32_t kw = __ldg(reinterpret_cast<const uint32_t*>(src));
            vw[r] = __ldg(reinterpret_cast<const uint32_t*>(src + hid));
            *reinterpret_cast<uint32_t*>(kc + (head + pos) * KV_D + 4 * lane) = kw;
        }
    }
    int8_t* vdst = vc + (head + (size_t)4 * pg) * KV_D + 16 * lane;  // [channel 4*lane + k][position r]
    if (valid[0] && valid[1] && valid[2] && valid[3]) {
        const uint32_t t0 = __byte_perm(vw[0], vw[1], 0x5140), t1 = __byte_perm(vw[2], vw[3], 0x5140);
        const uint32_t t2 = __byte_perm(vw[0], vw[1], 0x7362), t3 = __byte_perm(vw[2], vw[3], 0x7362);
        *reinterpret_cast<uint4*>(vdst) = make_uint4(__byte_perm(t0, t1, 0x5410), __byte_perm(t0, t1, 0x7632),
                                                     __byte_perm(t2, t3, 0x5410), __byte_perm(t2, t3, 0x7632));
    } else {
#pragma unroll
        for (int r = 0; r < 4; ++r)
            if (valid[r])
#pragma unroll
                for (int k = 0; k < 4; ++k) vdst[4 * k + r] = (int8_t)((vw[r] >> (8 * k)) & 0xffu);
    }
}

}  // namespace

// Cluster width: enough CTAs to put two on every SM, each keeping a worthwhile number of keys, and a
// score buffer that fits in shared memory.  Splitting a sequence costs three cluster-wide meetings, so
// it is done only when (sequence, head) pairs alone leave SMs idle: measured on B200, 56 heads, context
// 2047, wanting 2 / 4 / 8 CTAs per SM: batch 2: 11.3 / 15.1 / 15.2 us, batch 4: 25.1 / 28.2 / 33.4,
// batch 8: 37.4 / 47.6 / 47.0 (batch 12: 63.8 / 64.0 / 58.9).
int kv_choose_cluster(int64_t B, int64_t H, int64_t max_len) {
    const int64_t want = 2LL * sm_count();
    int c = 1;
    while (c < KV_MAX_CLUSTER && B * H * c < want && max_len / (2 * c) >= 256) c *= 2;
    while (c < KV_MAX_CLUSTER && kv_smem_bytes((int)(((max_len + c - 1) / c + KV_TILE - 1) / KV_TILE * KV_TILE)) > 200 * 1024) c *= 2;
    return c;
}

sq_status kv_decode_attention(const int8_t* q, int64_t ldq, int8_t* kc, int8_t* vc, const int8_t* k_new,
                              const int8_t* v_new, int64_t ld_new, const int32_t* lens,
                              int64_t B, int64_t H, int64_t lmax, int64_t max_len, float alpha_qk, float alpha_pv,
                              const float* requant_mul, void* out, sq_dtype out_dt, int64_t ldo, uint32_t* status,
                              cudaStream_t st) {
    KvParams p;
    p.q = q; p.ldq = ldq; p.kc = kc; p.vc = vc; p.lens = lens; p.lmax = lmax;
    p.k_new = k_new; p.v_new = v_new; p.ld_new = ld_new;
    p.H = (int)H; p.max_len = (int)max_len;
    p.cluster = kv_choose_cluster(B, H, max_len);
    p.cap = (int)(((max_len + p.cluster - 1) / p.cluster + KV_TILE - 1) / KV_TILE * KV_TILE);
    p.c1 = alpha_qk * kLog2e;
    p.alpha_pv = alpha_pv;
    p.requant_mul = requant_mul; p.out = out; p.out_dt = (int)out_dt; p.ldo = ldo; p.status = status;
    const size_t smem = kv_smem_bytes(p.cap);
    if (smem > 227 * 1024) return SQ_ERR_UNSUPPORTED;
    static bool attr_set[64] = {false};  // per device
    int dev = 0;
    SQ_CUDA_OK(cudaGetDevice(&dev));
    if (dev < 0 || dev >= 64 || !attr_set[dev]) {
        SQ_CUDA_OK(cudaFuncSetAttribute(kv_decode_attention_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, 227 * 1024));
        if (dev >= 0 && dev < 64) attr_set[dev] = true;
    }
    return launch_pdl(kv_decode_attention_kernel, dim3((unsigned)p.cluster, (unsigned)H, (unsigned)B), dim3(KV_THREADS), smem, st,
                      p.cluster, p);
}

sq_status kv_cache_write(const int8_t* qkv, int64_t ld, int64_t B, int64_t T, int64_t H, const int32_t* pos0, int8_t* kc,
                         int8_t* vc, int64_t lmax, uint32_t* status, cudaStream_t st) {
    const int groups = (int)((T + 3) / 4 + 1);  // a run of T positions touches at most this many 4-groups
    const int64_t warps = B * H * groups;
    const int64_t blocks = (warps + 7) / 8;
    if (blocks >= ((int64_t)1 << 31)) return SQ_ERR_UNSUPPORTED;
    return launch_pdl(kv_cache_write_kernel, dim3((unsigned)blocks), dim3(256), 0, st, 1, qkv, ld, (int)B, (int)T, (int)H, pos0, kc,
                      vc, lmax, groups, status);
}

}  // namespace sq
