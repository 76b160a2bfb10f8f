// tcgen05 / TMA / mbarrier building blocks shared by the tensor-core kernels of libsq
// (inline PTX for sm_100a) and the host-side tensor-map encoder.
#pragma once
#include <cuda.h>

#include <algorithm>

#include "sq_common.cuh"

namespace sq {
namespace tc {

constexpr int BLOCK_M = 128;  // accumulator rows per CTA (TMEM lanes)
constexpr int BLOCK_K = 128;  // INT8 elements = bytes: exactly one 128-byte swizzle row
constexpr int UMMA_K = 32;    // K per tcgen05.mma for 8-bit operands
constexpr uint32_t kWaitCycles = 2000000000u;  // ~1 s at B200 clocks
constexpr uint32_t kPeerBitMask = 0xFEFFFFFFu; // clears the CTA-rank bit of a shared::cluster address:
                                               // the same offset in the EVEN CTA of the pair

// ------------------------------------------------------------------------------------
// PTX wrappers
// ------------------------------------------------------------------------------------
__device__ __forceinline__ uint32_t smem_u32(const void* p) {
    return (uint32_t)__cvta_generic_to_shared(p);
}
__device__ __forceinline__ uint32_t cluster_ctarank() {
    uint32_t r;
    asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
    return r;
}
__device__ __forceinline__ void cluster_sync_all() {
    asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory");
    asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");
}
__device__ __forceinline__ void mbar_init(uint64_t* bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count));
}
__device__ __forceinline__ void mbar_expect_tx(uint64_t* bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(bar)),
                 "r"(bytes)
                 : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint64_t* bar) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(bar)) : "memory");
}
// arrive on the barrier at the same shared-memory offset in the even CTA of the pair
__device__ __forceinline__ void mbar_arrive_even_cta(uint64_t* bar) {
    asm volatile("mbarrier.arrive.release.cluster.shared::cluster.b64 _, [%0];"
                 ::"r"(smem_u32(bar) & kPeerBitMask)
                 : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint64_t* bar, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok)
        : "r"(smem_u32(bar)), "r"(parity)
        : "memory");
    return ok != 0;
}
// One lane of a converged warp (the same one every time).
__device__ __forceinline__ bool elect_one() {
    uint32_t pred;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "elect.sync _|p, 0xffffffff;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(pred));
    return pred != 0;
}
__device__ __forceinline__ bool mbar_try_wait_u32(uint32_t bar_addr, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok)
        : "r"(bar_addr), "r"(parity)
        : "memory");
    return ok != 0;
}
// Bounded wait.  Returns false (and raises the CTA's abort flag + the global status word)
// if the phase does not complete within the cycle budget or another role already aborted.
__device__ __forceinline__ bool mbar_wait(uint64_t* bar, uint32_t parity, volatile uint32_t* abort_flag,
                                          uint32_t* status, uint32_t where, uint32_t budget = kWaitCycles) {
    if (mbar_try_wait(bar, parity)) return true;
    const long long t0 = clock64();
    uint32_t spins = 0;
    while (!mbar_try_wait(bar, parity)) {
        if ((++spins & 63u) == 0u) {
            if (*abort_flag) return false;
            if ((unsigned long long)(clock64() - t0) > (unsigned long long)budget) {
                *abort_flag = 1u;
                atomicCAS(status, 0u, ((uint32_t)SQ_ERR_TIMEOUT) | (where << 8));
                return false;
            }
        }
    }
    return true;
}

// The same bounded wait by a whole, converged warp: every lane polls, the outcome is put to a vote, so the
// warp leaves converged and with one answer (a lane that timed out next to one that did not would
// otherwise part ways with it for good).
__device__ __forceinline__ bool mbar_wait_warp(uint64_t* bar, uint32_t bar_addr, uint32_t parity,
                                               volatile uint32_t* abort_flag, uint32_t* status, uint32_t where) {
    if (__all_sync(0xffffffffu, mbar_try_wait_u32(bar_addr, parity))) return true;
    const bool w = mbar_wait(bar, parity, abort_flag, status, where);
    return __all_sync(0xffffffffu, w);
}

// Tiled TMA load of one box into this CTA's shared memory.  With CG = 2 the completion is
// signalled on the EVEN CTA's barrier (same offset), which gathers both CTAs' bytes.
template <int CG>
__device__ __forceinline__ void tma_load_4d(void* dst, const CUtensorMap* map, uint64_t* bar, int c0,
                                            int c1, int c2, int c3) {
    if (CG == 1) {
        asm volatile(
            "cp.async.bulk.tensor.4d.shared::cluster.global.mbarrier::complete_tx::bytes "
            "[%0], [%1, {%3, %4, %5, %6}], [%2];"
            ::"r"(smem_u32(dst)), "l"(map), "r"(smem_u32(bar)), "r"(c0), "r"(c1), "r"(c2), "r"(c3)
            : "memory");
    } else {
        asm volatile(
            "cp.async.bulk.tensor.4d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes "
            "[%0], [%1, {%3, %4, %5, %6}], [%2];"
            ::"r"(smem_u32(dst)), "l"(map), "r"(smem_u32(bar) & kPeerBitMask), "r"(c0), "r"(c1), "r"(c2),
            "r"(c3)
            : "memory");
    }
}

// L2 eviction policy for data that is read exactly once (a weight matrix streamed at the generation
// stage): its lines are the first to go, so activations and partial sums stay resident.
__device__ __forceinline__ uint64_t l2_policy_evict_first() {
    uint64_t pol;
    asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(pol));
    return pol;
}
// tma_load_4d<1> with an L2 cache policy
__device__ __forceinline__ void tma_load_4d_policy(void* dst, const CUtensorMap* map, uint64_t* bar, int c0, int c1,
                                                   int c2, int c3, uint64_t policy) {
    asm volatile(
        "cp.async.bulk.tensor.4d.shared::cluster.global.mbarrier::complete_tx::bytes.L2::cache_hint "
        "[%0], [%1, {%3, %4, %5, %6}], [%2], %7;"
        ::"r"(smem_u32(dst)), "l"(map), "r"(smem_u32(bar)), "r"(c0), "r"(c1), "r"(c2), "r"(c3), "l"(policy)
        : "memory");
}

__device__ __forceinline__ uint64_t l2_policy_evict_last() {
    uint64_t pol;
    asm volatile("createpolicy.fractional.L2::evict_last.b64 %0, 1.0;" : "=l"(pol));
    return pol;
}
// tma_load_4d<CG> with an L2 cache policy
template <int CG>
__device__ __forceinline__ void tma_load_4d_hint(void* dst, const CUtensorMap* map, uint64_t* bar, int c0, int c1,
                                                 int c2, int c3, uint64_t policy) {
    if (CG == 1) {
        tma_load_4d_policy(dst, map, bar, c0, c1, c2, c3, policy);
    } else {
        asm volatile(
            "cp.async.bulk.tensor.4d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes.L2::cache_hint "
            "[%0], [%1, {%3, %4, %5, %6}], [%2], %7;"
            ::"r"(smem_u32(dst)), "l"(map), "r"(smem_u32(bar) & kPeerBitMask), "r"(c0), "r"(c1), "r"(c2), "r"(c3), "l"(policy)
            : "memory");
    }
}

// Pulls one box of a tensor map into L2 without a shared-memory destination.
__device__ __forceinline__ void tma_prefetch_l2_4d(const CUtensorMap* map, int c0, int c1, int c2, int c3) {
    asm volatile("cp.async.bulk.prefetch.tensor.4d.L2.global [%0, {%1, %2, %3, %4}];"
                 ::"l"(map), "r"(c0), "r"(c1), "r"(c2), "r"(c3)
                 : "memory");
}

__device__ __forceinline__ void tcgen05_fence_before() {
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
}
__device__ __forceinline__ void tcgen05_fence_after() {
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
}
// D[tmem] (+)= A[smem] * B[smem], INT8 x INT8 -> INT32
template <int CG>
__device__ __forceinline__ void umma_i8(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc,
                                        uint32_t idesc, uint32_t accumulate) {
    if (CG == 1) {
        asm volatile(
            "{\n\t.reg .pred p;\n\t"
            "setp.ne.b32 p, %4, 0;\n\t"
            "tcgen05.mma.cta_group::1.kind::i8 [%0], %1, %2, %3, p;\n\t}"
            ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate)
            : "memory");
    } else {
        asm volatile(
            "{\n\t.reg .pred p;\n\t"
            "setp.ne.b32 p, %4, 0;\n\t"
            "tcgen05.mma.cta_group::2.kind::i8 [%0], %1, %2, %3, p;\n\t}"
            ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate)
            : "memory");
    }
}
// The barrier (in every CTA of the group, same offset) receives one arrival once every MMA
// issued so far by this thread has completed.
template <int CG>
__device__ __forceinline__ void umma_commit(uint64_t* bar) {
    if (CG == 1) {
        asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];"
                     ::"r"(smem_u32(bar))
                     : "memory");
    } else {
        const uint16_t mask = 3;  // both CTAs of the pair
        asm volatile(
            "tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.multicast::cluster.b64 [%0], %1;"
            ::"r"(smem_u32(bar)), "h"(mask)
            : "memory");
    }
}
template <int CG>
__device__ __forceinline__ void umma_commit_u32(uint32_t bar_addr) {
    if (CG == 1) {
        asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar_addr) : "memory");
    } else {
        const uint16_t mask = 3;  // both CTAs of the pair
        asm volatile(
            "tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.multicast::cluster.b64 [%0], %1;"
            ::"r"(bar_addr), "h"(mask)
            : "memory");
    }
}
__device__ __forceinline__ void tmem_ld32(uint32_t taddr, uint32_t (&r)[32]) {
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
        "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
        "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]),
          "=r"(r[7]), "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]),
          "=r"(r[14]), "=r"(r[15]), "=r"(r[16]), "=r"(r[17]), "=r"(r[18]), "=r"(r[19]),
          "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]), "=r"(r[24]), "=r"(r[25]),
          "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
        : "r"(taddr)
        : "memory");
}
__device__ __forceinline__ void tmem_ld_wait() {
    asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
}
template <int THREADS>
__device__ __forceinline__ void epi_bar_sync() {
    asm volatile("bar.sync 1, %0;" ::"n"(THREADS) : "memory");
}
template <int CG>
__device__ __forceinline__ void tmem_alloc(uint32_t* holder, uint32_t cols) {
    if (CG == 1) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;"
                     ::"r"(smem_u32(holder)), "r"(cols) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    } else {
        asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;"
                     ::"r"(smem_u32(holder)), "r"(cols) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
    }
}
template <int CG>
__device__ __forceinline__ void tmem_dealloc(uint32_t base, uint32_t cols) {
    if (CG == 1)
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(base), "r"(cols) : "memory");
    else
        asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(base), "r"(cols) : "memory");
}

// Shared-memory matrix descriptor (sm_100 format): 128-byte swizzle, 8-row groups 1024 B
// apart.  For a K-major tile the rows are M/N indices; for the [K, N]-stored B operand
// ("MN-major") the rows are K indices and the 128 contiguous bytes are N indices.
__device__ __forceinline__ uint64_t make_smem_desc(uint32_t saddr, uint32_t lbo_bytes) {
    uint64_t d = 0;
    d |= (uint64_t)((saddr & 0x3FFFFu) >> 4);        // start address, bits [0,14)
    d |= (uint64_t)((lbo_bytes >> 4) & 0x3FFFu) << 16;  // leading-dimension byte offset
    d |= (uint64_t)(1024u >> 4) << 32;               // stride-dimension byte offset: 8 rows
    d |= (uint64_t)1 << 46;                          // descriptor version of sm_100
    d |= (uint64_t)2 << 61;                          // SWIZZLE_128B
    return d;
}

// The same descriptor in halves, for the MMA lane's inner loop: only the start address (and the
// leading-dimension offset) live in the low word, so a stage's and a K slice's descriptors are the
// first one's low word plus a multiple of 16 bytes >> 4; the high word never changes.
__device__ __forceinline__ uint32_t smem_desc_lo(uint32_t saddr, uint32_t lbo_bytes) {
    return ((saddr & 0x3FFFFu) >> 4) | (((lbo_bytes >> 4) & 0x3FFFu) << 16);
}
constexpr uint32_t kSmemDescHi = (1024u >> 4) | (1u << 14) | (2u << 29);  // SBO 1024 B, sm_100 version, SWIZZLE_128B
static_assert(((uint64_t)kSmemDescHi << 32) == (((uint64_t)(1024u >> 4) << 32) | ((uint64_t)1 << 46) | ((uint64_t)2 << 61)),
              "high word of the shared-memory descriptor");

// The same MMA with the operand descriptors given as low words (high word: kSmemDescHi).
template <int CG>
__device__ __forceinline__ void umma_i8_lo(uint32_t d_tmem, uint32_t a_lo, uint32_t b_lo, uint32_t idesc,
                                           uint32_t accumulate) {
    if (CG == 1) {
        asm volatile(
            "{\n\t.reg .pred p;\n\t.reg .b64 da, db;\n\t"
            "setp.ne.b32 p, %4, 0;\n\t"
            "mov.b64 da, {%1, %5};\n\t"
            "mov.b64 db, {%2, %5};\n\t"
            "tcgen05.mma.cta_group::1.kind::i8 [%0], da, db, %3, p;\n\t}"
            ::"r"(d_tmem), "r"(a_lo), "r"(b_lo), "r"(idesc), "r"(accumulate), "r"(kSmemDescHi)
            : "memory");
    } else {
        asm volatile(
            "{\n\t.reg .pred p;\n\t.reg .b64 da, db;\n\t"
            "setp.ne.b32 p, %4, 0;\n\t"
            "mov.b64 da, {%1, %5};\n\t"
            "mov.b64 db, {%2, %5};\n\t"
            "tcgen05.mma.cta_group::2.kind::i8 [%0], da, db, %3, p;\n\t}"
            ::"r"(d_tmem), "r"(a_lo), "r"(b_lo), "r"(idesc), "r"(accumulate), "r"(kSmemDescHi)
            : "memory");
    }
}

// Instruction descriptor of tcgen05.mma kind::i8: signed 8-bit A and B, INT32 D.
__host__ __device__ constexpr inline uint32_t make_idesc(int mma_m, int mma_n, int b_is_kn) {
    return (2u << 4)                       // D format: S32
           | (1u << 7)                     // A format: signed 8-bit
           | (1u << 10)                    // B format: signed 8-bit
           | (0u << 15)                    // A is K-major
           | ((uint32_t)(b_is_kn ? 1 : 0) << 16)  // B major-ness
           | ((uint32_t)(mma_n >> 3) << 17)       // N / 8
           | ((uint32_t)(mma_m >> 4) << 24);      // M / 16
}

__device__ __forceinline__ void tma_store_4d(const CUtensorMap* map, const void* src, int c0, int c1, int c2,
                                             int c3) {
    asm volatile("cp.async.bulk.tensor.4d.global.shared::cta.bulk_group [%0, {%2, %3, %4, %5}], [%1];"
                 ::"l"(map), "r"(smem_u32(src)), "r"(c0), "r"(c1), "r"(c2), "r"(c3)
                 : "memory");
    asm volatile("cp.async.bulk.commit_group;" ::: "memory");
}
__device__ __forceinline__ void tma_store_wait_read() {  // staging tile may be overwritten again
    asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory");
}
__device__ __forceinline__ void tma_store_wait_all() {
    asm volatile("cp.async.bulk.wait_group 0;" ::: "memory");
}


// ------------------------------------------------------------------------------------
// Host side: tensor maps
// ------------------------------------------------------------------------------------
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*,
                                  CUtensorMapInterleave, CUtensorMapSwizzle, CUtensorMapL2promotion,
                                  CUtensorMapFloatOOBfill);

inline EncodeTiledFn encode_fn() {
    static EncodeTiledFn fn = nullptr;
    if (fn == nullptr) {
        void* ptr = nullptr;
        cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &ptr, cudaEnableDefault, &q) == cudaSuccess &&
            q == cudaDriverEntryPointSuccess)
            fn = reinterpret_cast<EncodeTiledFn>(ptr);
    }
    return fn;
}

// Rank-4 INT8 tensor map over {inner (contiguous), row, head, batch} with the three outer
// dimensions ordered by ascending stride; reports which coordinate slot each one got.
// box_inner x box_rows bytes are copied per request (128-byte swizzle).
inline bool make_map(CUtensorMap* map, const void* base, int esz, int64_t inner, int64_t rows, int64_t heads,
              int64_t batch, int64_t s_row, int64_t s_head, int64_t s_batch, int box_inner, int box_rows,
              int* slot_row, int* slot_head, int* slot_batch) {
    EncodeTiledFn fn = encode_fn();
    if (!fn) return false;
    struct Dim { int64_t extent, stride; int box; int* slot; };
    Dim d[3] = {{rows, s_row, box_rows, slot_row}, {heads, s_head, 1, slot_head}, {batch, s_batch, 1, slot_batch}};
    // extent-1 dimensions never move the address: give them a harmless large stride so that
    // the order below stays ascending
    // strides are given in elements of `esz` bytes
    s_row *= esz; s_head *= esz; s_batch *= esz;
    d[0].stride = s_row; d[1].stride = s_head; d[2].stride = s_batch;
    int64_t span = std::max<int64_t>(inner * esz, 16);
    for (auto& x : d) if (x.extent > 1) span = std::max(span, x.extent * x.stride);
    span = (span + 15) / 16 * 16;
    for (auto& x : d) if (x.extent <= 1) x.stride = span;
    std::stable_sort(d, d + 3, [](const Dim& a, const Dim& b) { return a.stride < b.stride; });
    cuuint64_t gdim[4] = {(cuuint64_t)inner, (cuuint64_t)d[0].extent, (cuuint64_t)d[1].extent, (cuuint64_t)d[2].extent};
    cuuint64_t gstr[3] = {(cuuint64_t)d[0].stride, (cuuint64_t)d[1].stride, (cuuint64_t)d[2].stride};
    cuuint32_t box[4] = {(cuuint32_t)box_inner, (cuuint32_t)d[0].box, (cuuint32_t)d[1].box, (cuuint32_t)d[2].box};
    cuuint32_t estr[4] = {1, 1, 1, 1};
    for (int i = 0; i < 3; ++i) *d[i].slot = i + 1;
    const CUtensorMapDataType ty = esz == 1 ? CU_TENSOR_MAP_DATA_TYPE_UINT8
                                   : esz == 2 ? CU_TENSOR_MAP_DATA_TYPE_UINT16 : CU_TENSOR_MAP_DATA_TYPE_INT32;
    CUresult r = fn(map, ty, 4, const_cast<void*>(base), gdim, gstr, box, estr,
                    CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                    CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    return r == CUDA_SUCCESS;
}


}  // namespace tc
}  // namespace sq
