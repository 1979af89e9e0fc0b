// Fused quantize + NVFP4 linear for callers that cannot allocate device memory.
//
// Some callers of this library run where cudaMalloc is not an option: inside a serving loop whose
// memory pool is frozen after start-up, in a plugin that is handed input and output buffers and
// nothing else, or under a framework that forbids allocation once its CUDA graphs are built.  For
// them the scratch that nvfp4_quantize_linear takes from the caller (the quantized activations, their
// scale factors and the per-tensor scale) lives here, in a fixed array that is part of the
// library's device image.  Every GPU that loads the library holds the array until the process
// exits, so it is kept modest; problems whose scratch would not fit are rejected.
#include "sol_internal.h"

namespace sol {
namespace {

constexpr size_t kStaticScratchBytes = 64u << 20;  // 64 MiB: enough for M*K up to ~119M elements

// File-scope device array.  In host code this name is only a handle for the runtime's symbol
// calls, never an address a kernel may be given.
static __device__ __align__(256) uint8_t g_static_scratch[kStaticScratchBytes];

uint8_t *g_scratch_ptr[64] = {};

// Device address of the array on the current device, looked up once per device.
sol_status_t scratch_address(int device, uint8_t **out) {
    if (device < 0 || device >= 64) return SOL_ERR_CUDA;
    if (g_scratch_ptr[device] == nullptr) {
        void *ptr = nullptr;
        if (cudaGetSymbolAddress(&ptr, g_static_scratch) != cudaSuccess || ptr == nullptr) {
            cudaGetLastError();
            return SOL_ERR_CUDA;
        }
        g_scratch_ptr[device] = static_cast<uint8_t *>(ptr);
    }
    *out = g_scratch_ptr[device];
    return SOL_OK;
}

size_t align256(size_t v) { return (v + 255) & ~static_cast<size_t>(255); }

}  // namespace
}  // namespace sol

using namespace sol;

extern "C" {

size_t sol_nvfp4_static_scratch_bytes(void) { return kStaticScratchBytes; }

sol_status_t nvfp4_quantize_linear_static(const void *x_bf16, int64_t ldx, const void *wq, const void *wsf,
                                          const float *w_tscale, const void *bias_bf16, void *y_bf16,
                                          int64_t M, int64_t N, int64_t K, int64_t ldy, void *stream) {
    if (x_bf16 == nullptr || wq == nullptr || wsf == nullptr || w_tscale == nullptr || y_bf16 == nullptr)
        return SOL_ERR_NULL_POINTER;
    if (M <= 0 || N <= 0 || K <= 0 || K % 32 != 0 || N % 8 != 0 || M > (1LL << 30) || N > (1LL << 24) ||
        K > (1LL << 24) || ldx < K || ldy < N)
        return SOL_ERR_BAD_SHAPE;
    if (!aligned16(x_bf16) || !aligned16(wq) || !aligned16(wsf) || !aligned16(y_bf16) || ldx % 8 != 0 ||
        ldy % 8 != 0 || (bias_bf16 != nullptr && !aligned16(bias_bf16)) ||
        (reinterpret_cast<uintptr_t>(w_tscale) & 3u))
        return SOL_ERR_ALIGNMENT;
    const size_t data_bytes = align256(sol_nvfp4_data_bytes(M, K));
    const size_t scale_bytes = align256(sol_nvfp4_scale_bytes(M, K, SOL_SF_SWIZZLED_128x4));
    if (data_bytes + scale_bytes + 256 > kStaticScratchBytes) return SOL_ERR_WORKSPACE_TOO_SMALL;
    const DeviceInfo *dev = nullptr;
    sol_status_t st = check_arch(&dev);
    if (st != SOL_OK) return st;
    uint8_t *scratch = nullptr;
    st = scratch_address(dev->device, &scratch);
    if (st != SOL_OK) return st;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    uint8_t *xq = scratch;
    uint8_t *xsf = xq + data_bytes;
    float *xts = reinterpret_cast<float *>(xsf + scale_bytes);
    // The array keeps whatever the previous call left in it.  Nothing below relies on old contents:
    // the amax step zeroes the scale word it accumulates into, and the quantizer writes every byte of
    // the data and scale regions it hands to the GEMM, padding included.
    st = launch_amax_quantize(x_bf16, M, K, ldx, xts, xq, xsf, SOL_SF_SWIZZLED_128x4, s, dev);
    if (st != SOL_OK) return st;
    return launch_gemm_nvfp4(xq, xsf, xts, wq, wsf, w_tscale, bias_bf16, y_bf16, M, N, K, ldy, s, dev);
}

}  // extern "C"
