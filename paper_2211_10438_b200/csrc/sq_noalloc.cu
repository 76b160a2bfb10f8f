// sq_ln_quant_tensor_noalloc: the per-tensor-dynamic fused LayerNorm + quantise for callers
// that cannot hand the library a workspace because they cannot allocate device memory at all
// (e.g. code running inside an inference server's pre-sized arena, a plug-in that is only given
// its input and output buffers, or a real-time loop where cudaMalloc's implicit synchronisation
// is forbidden).  The scratch the two-pass scheme needs -- one absmax word and the per-row
// LayerNorm statistics -- lives in a fixed array that is part of the library image.
#include <mutex>

#include "sq_common.cuh"
#include "sq_kernels.h"

namespace {

// Scratch layout: [0, 256) header (absmax word at byte 16), then 2 floats per row.
constexpr size_t kScratchBytes = sq::kWsHeader + (size_t)SQ_NOALLOC_MAX_ROWS * 2 * sizeof(float);

// Every GPU that loads the library holds this array (about 128 KB) until the process exits.
static __device__ __align__(256) unsigned char g_noalloc_scratch[kScratchBytes];

// In host code the name g_noalloc_scratch is only a stand-in for the symbol, not a device
// address: the address is looked up once per device and cached here.
std::mutex g_mu;
void* g_scratch_addr[64] = {nullptr};

// Device address of the scratch array on the CURRENT device (looked up on first use).
sq_status scratch_address(void** out) {
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return SQ_ERR_CUDA;
    if (dev < 0 || dev >= 64) return SQ_ERR_UNSUPPORTED;
    std::lock_guard<std::mutex> lock(g_mu);
    if (g_scratch_addr[dev] == nullptr) {
        void* p = nullptr;
        if (cudaGetSymbolAddress(&p, g_noalloc_scratch) != cudaSuccess || p == nullptr) {
            cudaGetLastError();
            return SQ_ERR_CUDA;
        }
        g_scratch_addr[dev] = p;
    }
    *out = g_scratch_addr[dev];
    return SQ_OK;
}

}  // namespace

extern "C" sq_status sq_ln_quant_tensor_noalloc(const void* X, sq_dtype dt, int64_t M, int64_t C,
                                                const void* gamma_hat, const void* beta_hat, float eps,
                                                int8_t* Xq, float* x_scale, void* stream) {
    using namespace sq;
    if ((dt != SQ_F16 && dt != SQ_BF16) || !(eps >= 0.0f)) return SQ_ERR_INVALID_ARG;
    if (M < 0 || C < 0) return SQ_ERR_SHAPE;
    if (M > SQ_NOALLOC_MAX_ROWS) return SQ_ERR_UNSUPPORTED;  // beyond the built-in scratch
    if (M == 0 || C == 0) return SQ_OK;
    if (!X || !Xq || !x_scale || !gamma_hat) return SQ_ERR_INVALID_ARG;
    if (C % 8 != 0 || !aligned16(X) || (reinterpret_cast<uintptr_t>(Xq) & 7) != 0 || !aligned16(gamma_hat) ||
        (beta_hat && !aligned16(beta_hat)))
        return SQ_ERR_ALIGN;
    void* base = nullptr;
    sq_status s = scratch_address(&base);
    if (s != SQ_OK) return s;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    float* word = reinterpret_cast<float*>(static_cast<char*>(base) + kWsAbsmaxOff);
    float* stats = reinterpret_cast<float*>(static_cast<char*>(base) + kWsHeader);
    // The array keeps whatever the previous call left: the running maximum must start at zero.
    // (The statistics are fully overwritten by pass 1 before pass 2 reads them.)
    SQ_CUDA_OK(cudaMemsetAsync(word, 0, sizeof(float), st));
    s = row_quant(X, dt, M, C, nullptr, gamma_hat, beta_hat, eps, true, ROW_ABSMAX_ONLY, nullptr, nullptr, word,
                  stats, 0, nullptr, st);
    if (s != SQ_OK) return s;
    return row_quant(X, dt, M, C, nullptr, gamma_hat, beta_hat, eps, true, ROW_FROM_ABSMAX_WORD, Xq, x_scale,
                     word, stats, 1, nullptr, st);
}
