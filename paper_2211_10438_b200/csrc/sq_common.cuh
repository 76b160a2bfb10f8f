// Shared device/host helpers of libsq (CUDA side only).
#pragma once
#include <cuda_bf16.h>
#include <cuda_fp16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include <utility>

#include "../../include/sq.h"

namespace sq {

constexpr float kAbsmaxFloor = 1e-5f;  // smallest absolute maximum used as a divisor
constexpr int kNumSMsB200 = 148;

#define SQ_CUDA_OK(expr)                              \
    do {                                              \
        cudaError_t e__ = (expr);                     \
        if (e__ != cudaSuccess) return SQ_ERR_CUDA;   \
    } while (0)

inline sq_status launch_status() {
    return cudaPeekAtLastError() == cudaSuccess ? SQ_OK : (cudaGetLastError(), SQ_ERR_CUDA);
}

inline bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15) == 0; }

int sm_count();  // SMs of the current device (cached)

// ---------------------------------------------------------------------------------------
// 16-bit activation types: unpack 8 values (one 16-byte vector) to fp32, exactly.
// ---------------------------------------------------------------------------------------
template <typename T>
struct Act;

template <>
struct Act<__half> {
    using T2 = __half2;
    static __device__ __forceinline__ float2 to_float2(uint32_t u) {
        return __half22float2(*reinterpret_cast<const __half2*>(&u));
    }
    static __device__ __forceinline__ float to_float(__half v) { return __half2float(v); }
    static __device__ __forceinline__ __half from_float(float v) { return __float2half_rn(v); }
    // |a| and max are exact in fp16, so packed forms may be used for absolute maxima
    static __device__ __forceinline__ uint32_t absmax2(uint32_t acc, uint32_t v) {
        __half2 r = __hmax2(*reinterpret_cast<const __half2*>(&acc),
                            __habs2(*reinterpret_cast<const __half2*>(&v)));
        return *reinterpret_cast<uint32_t*>(&r);
    }
    static __device__ __forceinline__ float hmax_of2(uint32_t u) {
        float2 f = to_float2(u);
        return fmaxf(f.x, f.y);
    }
};

template <>
struct Act<__nv_bfloat16> {
    using T2 = __nv_bfloat162;
    static __device__ __forceinline__ float2 to_float2(uint32_t u) {
        // bf16 -> fp32 is a 16-bit shift
        return make_float2(__uint_as_float(u << 16), __uint_as_float(u & 0xffff0000u));
    }
    static __device__ __forceinline__ float to_float(__nv_bfloat16 v) { return __bfloat162float(v); }
    static __device__ __forceinline__ __nv_bfloat16 from_float(float v) {
        return __float2bfloat16_rn(v);
    }
    static __device__ __forceinline__ uint32_t absmax2(uint32_t acc, uint32_t v) {
        __nv_bfloat162 r = __hmax2(*reinterpret_cast<const __nv_bfloat162*>(&acc),
                                   __habs2(*reinterpret_cast<const __nv_bfloat162*>(&v)));
        return *reinterpret_cast<uint32_t*>(&r);
    }
    static __device__ __forceinline__ float hmax_of2(uint32_t u) {
        float2 f = to_float2(u);
        return fmaxf(f.x, f.y);
    }
};

template <typename T>
__device__ __forceinline__ void unpack8(const uint4& v, float (&f)[8]) {
    float2 a = Act<T>::to_float2(v.x), b = Act<T>::to_float2(v.y), c = Act<T>::to_float2(v.z),
           d = Act<T>::to_float2(v.w);
    f[0] = a.x; f[1] = a.y; f[2] = b.x; f[3] = b.y;
    f[4] = c.x; f[5] = c.y; f[6] = d.x; f[7] = d.y;
}

// ---------------------------------------------------------------------------------------
// Eq. 1 pieces.  Every operation is an explicitly rounded fp32 intrinsic so that the
// compiler cannot contract or reassociate: the codes are a bit-exact contract.
// ---------------------------------------------------------------------------------------
__device__ __forceinline__ float step_size(float absmax) {
    return __fdiv_rn(fmaxf(absmax, kAbsmaxFloor), 127.0f);
}
__device__ __forceinline__ float recip_step(float delta) { return __fdiv_rn(1.0f, delta); }

// round(v * inv) with ONE rounding: the fused multiply-add adds 1.5 * 2^23 to the exact
// product, so the fp32 result is rounded (half to even) at integer granularity and the code
// sits in the low mantissa bits as a two's-complement byte.  CLAMP keeps it in [-127, 127];
// without it the caller guarantees |v * inv| < 127.5 (dynamic step sizes).
constexpr float kRoundMagic = 12582912.0f;
template <bool CLAMP = true>
__device__ __forceinline__ uint32_t quant_code(float v, float inv) {
    float r = __fmaf_rn(v, inv, kRoundMagic);
    if (CLAMP) r = fminf(fmaxf(r, kRoundMagic - 127.0f), kRoundMagic + 127.0f);
    return __float_as_uint(r);  // low byte = the INT8 code
}
// low bytes of four words -> one word
__device__ __forceinline__ uint32_t pack4(uint32_t a, uint32_t b, uint32_t c, uint32_t d) {
    return __byte_perm(__byte_perm(a, b, 0x0040), __byte_perm(c, d, 0x0040), 0x5410);
}
template <bool CLAMP = true>
__device__ __forceinline__ uint2 quant8(const float (&f)[8], float inv) {
    uint2 r;
    r.x = pack4(quant_code<CLAMP>(f[0], inv), quant_code<CLAMP>(f[1], inv), quant_code<CLAMP>(f[2], inv),
                quant_code<CLAMP>(f[3], inv));
    r.y = pack4(quant_code<CLAMP>(f[4], inv), quant_code<CLAMP>(f[5], inv), quant_code<CLAMP>(f[6], inv),
                quant_code<CLAMP>(f[7], inv));
    return r;
}

// The same codes from packed pairs: sm_100's two-wide fp32 multiply-add rounds each half exactly
// like the scalar instruction and takes one issue slot for two values.
template <typename T>
__device__ __forceinline__ void unpack8_pairs(const uint4& v, float2 (&f)[4]) {
    f[0] = Act<T>::to_float2(v.x); f[1] = Act<T>::to_float2(v.y);
    f[2] = Act<T>::to_float2(v.z); f[3] = Act<T>::to_float2(v.w);
}
template <bool CLAMP = true>
__device__ __forceinline__ uint2 quant8_pairs(const float2 (&f)[4], float inv) {
    const float2 inv2 = make_float2(inv, inv), magic2 = make_float2(kRoundMagic, kRoundMagic);
    uint32_t c[8];
#pragma unroll
    for (int j = 0; j < 4; ++j) {
        float2 r = __ffma2_rn(f[j], inv2, magic2);
        if (CLAMP) {
            r.x = fminf(fmaxf(r.x, kRoundMagic - 127.0f), kRoundMagic + 127.0f);
            r.y = fminf(fmaxf(r.y, kRoundMagic - 127.0f), kRoundMagic + 127.0f);
        }
        c[2 * j] = __float_as_uint(r.x);
        c[2 * j + 1] = __float_as_uint(r.y);
    }
    return make_uint2(pack4(c[0], c[1], c[2], c[3]), pack4(c[4], c[5], c[6], c[7]));
}

// 1/sqrt(v) for the LayerNorm statistic: the hardware approximation plus one Newton step (about
// one unit in the last place; the statistic is a tolerance quantity, the element-wise part that
// consumes it is the bit-exact one).
__device__ __forceinline__ float rsqrt_refined(float v) {
    const float r = rsqrtf(v), h = 0.5f * v;
    return fmaf(r, fmaf(-h * r, r, 0.5f), r);
}

// ---------------------------------------------------------------------------------------
// Reductions
// ---------------------------------------------------------------------------------------
__device__ __forceinline__ float warp_max(float v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, o));
    return v;
}
__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    return v;
}
// Block-wide reductions; `red` is shared scratch of >= 33 floats.  All threads get the result.
template <bool IS_MAX>
__device__ __forceinline__ float block_reduce(float v, float* red) {
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, nwarp = (blockDim.x + 31) >> 5;
    v = IS_MAX ? warp_max(v) : warp_sum(v);
    __syncthreads();  // protect `red` from the previous use
    if (lane == 0) red[warp] = v;
    __syncthreads();
    if (warp == 0) {
        float t = lane < nwarp ? red[lane] : (IS_MAX ? 0.0f : 0.0f);
        t = IS_MAX ? warp_max(t) : warp_sum(t);
        if (lane == 0) red[32] = t;
    }
    __syncthreads();
    return red[32];
}

// ---------------------------------------------------------------------------------------
// Programmatic dependent launch.  The runtime kernels of the path are launched with the
// programmatic-stream-serialisation attribute: a kernel may be scheduled while its predecessor
// in the stream is still draining, runs its set-up (barriers, tensor memory, descriptor and
// weight prefetch) and then blocks in pdl_wait() until the predecessor has completed and its
// writes are visible.  No global memory that an earlier kernel produces or still reads may be
// touched before pdl_wait().  Both instructions are no-ops for ordinary launches.
// ---------------------------------------------------------------------------------------
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void pdl_launch_dependents() {
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
}

template <typename... KArgs, typename... Args>
inline sq_status launch_pdl(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t st,
                            int cluster_x, Args&&... args) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid;
    cfg.blockDim = block;
    cfg.dynamicSmemBytes = smem;
    cfg.stream = st;
    cudaLaunchAttribute attr[2];
    int n = 0;
    attr[n].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[n].val.programmaticStreamSerializationAllowed = 1;
    ++n;
    if (cluster_x > 1) {
        attr[n].id = cudaLaunchAttributeClusterDimension;
        attr[n].val.clusterDim.x = (unsigned)cluster_x;
        attr[n].val.clusterDim.y = 1;
        attr[n].val.clusterDim.z = 1;
        ++n;
    }
    cfg.attrs = attr;
    cfg.numAttrs = n;
    if (cudaLaunchKernelEx(&cfg, kernel, std::forward<Args>(args)...) != cudaSuccess) {
        cudaGetLastError();
        return SQ_ERR_CUDA;
    }
    return launch_status();
}

// max for non-negative floats through their (order-preserving) bit patterns
__device__ __forceinline__ void atomic_max_nonneg(float* addr, float v) {
    atomicMax(reinterpret_cast<unsigned int*>(addr), __float_as_uint(v));
}

}  // namespace sq
