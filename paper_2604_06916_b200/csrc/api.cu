// C-ABI entry points: argument validation, size queries, device checks, TMA descriptor
// encoding.  Every compute step runs in the kernels of quantize.cu and gemm.cu.
#include "sol_internal.h"
#include "gemm_common.cuh"

#include <cstddef>
#include <mutex>

namespace sol {

__device__ DeviceStatusBlock g_status_block = {0u, 0u, kDefaultWaitLimitCycles};

namespace {

std::mutex g_mutex;
DeviceInfo g_devices[64];
uint32_t *g_status_ptr[64] = {};

using EncodeTiledFn = CUresult (*)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *,
                                   const cuuint64_t *, const cuuint32_t *, const cuuint32_t *,
                                   CUtensorMapInterleave, CUtensorMapSwizzle, CUtensorMapL2promotion,
                                   CUtensorMapFloatOOBfill);
EncodeTiledFn g_encode = nullptr;

EncodeTiledFn encode_fn() {
    std::lock_guard<std::mutex> lock(g_mutex);
    if (g_encode == nullptr) {
        void *fn = nullptr;
        cudaDriverEntryPointQueryResult qres;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &qres) == cudaSuccess &&
            qres == cudaDriverEntryPointSuccess)
            g_encode = reinterpret_cast<EncodeTiledFn>(fn);
    }
    return g_encode;
}

}  // namespace

const DeviceInfo *current_device_info() {
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return nullptr;
    std::lock_guard<std::mutex> lock(g_mutex);
    DeviceInfo &d = g_devices[dev];
    if (!d.ok) {
        cudaDeviceProp prop;
        if (cudaGetDeviceProperties(&prop, dev) != cudaSuccess) return nullptr;
        d.device = dev;
        d.sm_count = prop.multiProcessorCount;
        d.cc_major = prop.major;
        d.cc_minor = prop.minor;
        void *sym = nullptr;
        if (cudaGetSymbolAddress(&sym, g_status_block) != cudaSuccess) return nullptr;
        g_status_ptr[dev] = static_cast<uint32_t *>(sym);
        d.ok = true;
    }
    return &d;
}

sol_status_t check_arch(const DeviceInfo **info_out) {
    const DeviceInfo *d = current_device_info();
    if (d == nullptr) {
        cudaGetLastError();
        return SOL_ERR_CUDA;
    }
    if (d->cc_major != 10) return SOL_ERR_UNSUPPORTED_ARCH;
    *info_out = d;
    return SOL_OK;
}

uint32_t *device_status_word() {
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return nullptr;
    return g_status_ptr[dev];
}

bool make_tmap_2d(CUtensorMap *out, CUtensorMapDataType dtype, uint32_t elem_bytes, const void *base,
                  uint64_t inner, uint64_t outer, uint64_t pitch_bytes, uint32_t box_inner, uint32_t box_outer,
                  CUtensorMapSwizzle swizzle) {
    EncodeTiledFn fn = encode_fn();
    if (fn == nullptr) return false;
    (void)elem_bytes;
    cuuint64_t dims[2] = {inner, outer};
    cuuint64_t strides[1] = {pitch_bytes};
    cuuint32_t box[2] = {box_inner, box_outer};
    cuuint32_t estr[2] = {1, 1};
    return fn(out, dtype, 2, const_cast<void *>(base), dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
              swizzle, CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

bool make_tmap_3d_bf16(CUtensorMap *out, const void *base, uint64_t d0, uint64_t d1, uint64_t d2, uint64_t pitch1_bytes,
                       uint64_t pitch2_bytes, uint32_t box0, uint32_t box1) {
    EncodeTiledFn fn = encode_fn();
    if (fn == nullptr) return false;
    cuuint64_t dims[3] = {d0, d1, d2};
    cuuint64_t strides[2] = {pitch1_bytes, pitch2_bytes};
    cuuint32_t box[3] = {box0, box1, 1};
    cuuint32_t estr[3] = {1, 1, 1};
    return fn(out, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void *>(base), dims, strides, box, estr,
              CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
              CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

bool make_tmap_sf(CUtensorMap *out, const void *base, uint64_t chunks_k, uint64_t row_chunks,
                  uint32_t box_row_chunks, uint32_t box_k_chunks) {
    EncodeTiledFn fn = encode_fn();
    if (fn == nullptr) return false;
    cuuint64_t dims[3] = {128, chunks_k, row_chunks};
    cuuint64_t strides[2] = {512, 512 * chunks_k};
    cuuint32_t box[3] = {128, box_k_chunks, box_row_chunks};
    cuuint32_t estr[3] = {1, 1, 1};
    return fn(out, CU_TENSOR_MAP_DATA_TYPE_UINT32, 3, const_cast<void *>(base), dims, strides, box, estr,
              CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
              CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

namespace {

bool shape_ok(int64_t rows, int64_t K) {
    // the streaming kernels index their tiles (128 rows x 256 elements) and 32 KB pieces with a one-dimensional grid
    return rows > 0 && K > 0 && K % 32 == 0 && rows <= (1LL << 30) && K <= (1LL << 24) &&
           ceil_div(rows, 128) * ceil_div(K, 256) <= 0x7FFFFFFFLL && ceil_div(rows * (K / 8), 2048) <= 0x7FFFFFFFLL;
}

size_t align256(size_t v) { return (v + 255) & ~static_cast<size_t>(255); }

}  // namespace
}  // namespace sol

using namespace sol;

extern "C" {

const char *sol_status_string(sol_status_t status) {
    switch (status) {
        case SOL_OK: return "SOL_OK";
        case SOL_ERR_NULL_POINTER: return "SOL_ERR_NULL_POINTER";
        case SOL_ERR_BAD_SHAPE: return "SOL_ERR_BAD_SHAPE";
        case SOL_ERR_ALIGNMENT: return "SOL_ERR_ALIGNMENT";
        case SOL_ERR_WORKSPACE_TOO_SMALL: return "SOL_ERR_WORKSPACE_TOO_SMALL";
        case SOL_ERR_UNSUPPORTED_ARCH: return "SOL_ERR_UNSUPPORTED_ARCH";
        case SOL_ERR_CUDA: return "SOL_ERR_CUDA";
        case SOL_ERR_TIMEOUT: return "SOL_ERR_TIMEOUT";
        case SOL_ERR_BAD_LAYOUT: return "SOL_ERR_BAD_LAYOUT";
    }
    return "SOL_ERR_UNKNOWN";
}

size_t sol_nvfp4_data_bytes(int64_t rows, int64_t K) {
    if (!shape_ok(rows, K)) return 0;
    return static_cast<size_t>(rows) * static_cast<size_t>(K / 2);
}

size_t sol_nvfp4_scale_bytes(int64_t rows, int64_t K, sol_sf_layout_t layout) {
    if (!shape_ok(rows, K)) return 0;
    if (layout == SOL_SF_ROW_MAJOR) return static_cast<size_t>(rows) * static_cast<size_t>(K / 16);
    if (layout == SOL_SF_SWIZZLED_128x4)
        return static_cast<size_t>(ceil_div(rows, 128)) * static_cast<size_t>(ceil_div(K, 64)) * 512;
    return 0;
}

size_t sol_nvfp4_linear_workspace_bytes(int64_t M, int64_t N, int64_t K) {
    if (!shape_ok(M, K) || N <= 0) return 0;
    return align256(sol_nvfp4_data_bytes(M, K)) + align256(sol_nvfp4_scale_bytes(M, K, SOL_SF_SWIZZLED_128x4)) + 256;
}

sol_status_t sol_amax_bf16(const void *x, int64_t rows, int64_t K, int64_t ld, float *tensor_scale_out,
                           void *stream) {
    if (x == nullptr || tensor_scale_out == nullptr) return SOL_ERR_NULL_POINTER;
    if (!shape_ok(rows, K) || ld < K) return SOL_ERR_BAD_SHAPE;
    if (!aligned16(x) || ld % 8 != 0 || (reinterpret_cast<uintptr_t>(tensor_scale_out) & 3u)) return SOL_ERR_ALIGNMENT;
    const DeviceInfo *dev = nullptr;
    sol_status_t st = check_arch(&dev);
    if (st != SOL_OK) return st;
    return launch_amax(x, rows, K, ld, tensor_scale_out, static_cast<cudaStream_t>(stream), dev);
}

sol_status_t nvfp4_quantize(const void *x_bf16, int64_t M, int64_t K, int64_t ldx, const float *tensor_scale,
                            void *q_out, void *sf_out, sol_sf_layout_t layout, void *stream) {
    if (x_bf16 == nullptr || tensor_scale == nullptr || q_out == nullptr || sf_out == nullptr)
        return SOL_ERR_NULL_POINTER;
    if (!shape_ok(M, K) || ldx < K) return SOL_ERR_BAD_SHAPE;
    if (layout != SOL_SF_ROW_MAJOR && layout != SOL_SF_SWIZZLED_128x4) return SOL_ERR_BAD_LAYOUT;
    if (!aligned16(x_bf16) || !aligned16(q_out) || !aligned16(sf_out) || ldx % 8 != 0 ||
        (reinterpret_cast<uintptr_t>(tensor_scale) & 3u))
        return SOL_ERR_ALIGNMENT;
    const DeviceInfo *dev = nullptr;
    sol_status_t st = check_arch(&dev);
    if (st != SOL_OK) return st;
    return launch_quantize(x_bf16, M, K, ldx, tensor_scale, q_out, sf_out, layout, static_cast<cudaStream_t>(stream));
}

sol_status_t nvfp4_quantize_weight(const void *w_bf16, int64_t N, int64_t K, int64_t ldw, void *q_out,
                                   void *sf_out, float *tensor_scale_out, sol_sf_layout_t layout, void *stream) {
    if (w_bf16 == nullptr || tensor_scale_out == nullptr || q_out == nullptr || sf_out == nullptr)
        return SOL_ERR_NULL_POINTER;
    if (!shape_ok(N, K) || ldw < K) return SOL_ERR_BAD_SHAPE;
    if (layout != SOL_SF_ROW_MAJOR && layout != SOL_SF_SWIZZLED_128x4) return SOL_ERR_BAD_LAYOUT;
    if (!aligned16(w_bf16) || !aligned16(q_out) || !aligned16(sf_out) || ldw % 8 != 0 ||
        (reinterpret_cast<uintptr_t>(tensor_scale_out) & 3u))
        return SOL_ERR_ALIGNMENT;
    const DeviceInfo *dev = nullptr;
    sol_status_t st = check_arch(&dev);
    if (st != SOL_OK) return st;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    st = launch_amax(w_bf16, N, K, ldw, tensor_scale_out, s, dev);
    if (st != SOL_OK) return st;
    return launch_quantize(w_bf16, N, K, ldw, tensor_scale_out, q_out, sf_out, layout, s);
}

static sol_status_t check_requantize_lora(const void *w, const void *a, const void *b, const void *merged,
                                          const void *q, const void *sf, const float *ts, int64_t ldw, int64_t lda,
                                          int64_t ldb, int64_t N, int64_t K, int64_t r, sol_sf_layout_t layout) {
    if (w == nullptr || a == nullptr || b == nullptr || merged == nullptr || q == nullptr || sf == nullptr ||
        ts == nullptr)
        return SOL_ERR_NULL_POINTER;
    if (!shape_ok(N, K) || ldw < K || lda < K || r < 1 || r > lora_max_rank() || ldb < r || N > 65535LL * 64)
        return SOL_ERR_BAD_SHAPE;
    if (layout != SOL_SF_ROW_MAJOR && layout != SOL_SF_SWIZZLED_128x4) return SOL_ERR_BAD_LAYOUT;
    if (!aligned16(w) || !aligned16(a) || !aligned16(merged) || !aligned16(q) || !aligned16(sf) || ldw % 8 != 0 ||
        lda % 8 != 0 || (reinterpret_cast<uintptr_t>(b) & 1u) || (reinterpret_cast<uintptr_t>(ts) & 3u))
        return SOL_ERR_ALIGNMENT;
    return SOL_OK;
}

sol_status_t nvfp4_requantize_lora(const void *w_bf16, int64_t ldw, const void *lora_a, int64_t lda,
                                   const void *lora_b, int64_t ldb, int64_t N, int64_t K, int64_t r, float scaling,
                                   void *merged_bf16, void *q_out, void *sf_out, float *tensor_scale_out,
                                   sol_sf_layout_t layout, void *stream) {
    sol_status_t st = check_requantize_lora(w_bf16, lora_a, lora_b, merged_bf16, q_out, sf_out, tensor_scale_out, ldw,
                                            lda, ldb, N, K, r, layout);
    if (st != SOL_OK) return st;
    const DeviceInfo *dev = nullptr;
    st = check_arch(&dev);
    if (st != SOL_OK) return st;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    MergeGroup mg = {};
    mg.w[0] = static_cast<const uint16_t *>(w_bf16);
    mg.a[0] = static_cast<const uint16_t *>(lora_a);
    mg.b[0] = static_cast<const uint16_t *>(lora_b);
    mg.out[0] = static_cast<uint16_t *>(merged_bf16);
    mg.scale_words[0] = tensor_scale_out;
    st = launch_lora_merge(mg, 1, ldw, lda, ldb, N, K, r, scaling, s);
    if (st != SOL_OK) return st;
    return launch_quantize_from_amax(merged_bf16, N, K, K, tensor_scale_out, q_out, sf_out, layout, s);
}

sol_status_t nvfp4_requantize_lora_batch(int64_t count, const void *const *w_list, const void *const *a_list,
                                         const void *const *b_list, void *const *q_list, void *const *sf_list,
                                         float *const *ts_list, int64_t N, int64_t K, int64_t r, float scaling,
                                         void *merged_bf16, int64_t merged_matrices, sol_sf_layout_t layout,
                                         void *stream) {
    if (count < 0 || merged_matrices < 1) return SOL_ERR_BAD_SHAPE;
    if (count == 0) return SOL_OK;
    if (w_list == nullptr || a_list == nullptr || b_list == nullptr || q_list == nullptr || sf_list == nullptr ||
        ts_list == nullptr)
        return SOL_ERR_NULL_POINTER;
    // validate every matrix before the first launch: an error status means nothing was launched
    for (int64_t i = 0; i < count; ++i) {
        const sol_status_t st = check_requantize_lora(w_list[i], a_list[i], b_list[i], merged_bf16, q_list[i],
                                                      sf_list[i], ts_list[i], K, K, r, N, K, r, layout);
        if (st != SOL_OK) return st;
    }
    const DeviceInfo *dev = nullptr;
    sol_status_t st = check_arch(&dev);
    if (st != SOL_OK) return st;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    const int64_t group = merged_matrices < kMaxGroup ? merged_matrices : kMaxGroup;
    for (int64_t i0 = 0; i0 < count; i0 += group) {
        const int n = static_cast<int>(count - i0 < group ? count - i0 : group);
        MergeGroup mg = {};
        QuantGroup qg = {};
        for (int i = 0; i < n; ++i) {
            uint16_t *merged = static_cast<uint16_t *>(merged_bf16) + static_cast<int64_t>(i) * N * K;
            mg.w[i] = static_cast<const uint16_t *>(w_list[i0 + i]);
            mg.a[i] = static_cast<const uint16_t *>(a_list[i0 + i]);
            mg.b[i] = static_cast<const uint16_t *>(b_list[i0 + i]);
            mg.out[i] = merged;
            mg.scale_words[i] = ts_list[i0 + i];
            qg.x[i] = merged;
            qg.scale_words[i] = ts_list[i0 + i];
            qg.q[i] = static_cast<uint8_t *>(q_list[i0 + i]);
            qg.sf[i] = static_cast<uint8_t *>(sf_list[i0 + i]);
        }
        st = launch_lora_merge(mg, n, K, K, r, N, K, r, scaling, s);
        if (st != SOL_OK) return st;
        st = launch_quantize_group(qg, n, N, K, layout, s);
        if (st != SOL_OK) return st;
    }
    return SOL_OK;
}

static sol_status_t check_linear_common(const void *bias, const void *y, int64_t M, int64_t N, int64_t K,
                                        int64_t ldy) {
    if (!shape_ok(M, K) || N <= 0 || N % 8 != 0 || N > (1LL << 24) || ldy < N) return SOL_ERR_BAD_SHAPE;
    if (!aligned16(y) || ldy % 8 != 0 || (bias != nullptr && !aligned16(bias))) return SOL_ERR_ALIGNMENT;
    return SOL_OK;
}

sol_status_t nvfp4_linear(const void *xq, const void *xsf, const float *x_tscale, const void *wq, const void *wsf,
                          const float *w_tscale, const void *bias_bf16, void *y_bf16, int64_t M, int64_t N,
                          int64_t K, int64_t ldy, void *stream) {
    if (xq == nullptr || xsf == nullptr || x_tscale == nullptr || wq == nullptr || wsf == nullptr ||
        w_tscale == nullptr || y_bf16 == nullptr)
        return SOL_ERR_NULL_POINTER;
    sol_status_t st = check_linear_common(bias_bf16, y_bf16, M, N, K, ldy);
    if (st != SOL_OK) return st;
    if (!aligned16(xq) || !aligned16(xsf) || !aligned16(wq) || !aligned16(wsf) ||
        (reinterpret_cast<uintptr_t>(x_tscale) & 3u) || (reinterpret_cast<uintptr_t>(w_tscale) & 3u))
        return SOL_ERR_ALIGNMENT;
    const DeviceInfo *dev = nullptr;
    st = check_arch(&dev);
    if (st != SOL_OK) return st;
    return launch_gemm_nvfp4(xq, xsf, x_tscale, wq, wsf, w_tscale, bias_bf16, y_bf16, M, N, K, ldy,
                             static_cast<cudaStream_t>(stream), dev);
}

sol_status_t bf16_linear(const void *x_bf16, const void *w_bf16, const void *bias_bf16, void *y_bf16, int64_t M,
                         int64_t N, int64_t K, int64_t ldx, int64_t ldw, int64_t ldy, void *stream) {
    if (x_bf16 == nullptr || w_bf16 == nullptr || y_bf16 == nullptr) return SOL_ERR_NULL_POINTER;
    sol_status_t st = check_linear_common(bias_bf16, y_bf16, M, N, K, ldy);
    if (st != SOL_OK) return st;
    if (ldx < K || ldw < K) return SOL_ERR_BAD_SHAPE;
    if (!aligned16(x_bf16) || !aligned16(w_bf16) || ldx % 8 != 0 || ldw % 8 != 0) return SOL_ERR_ALIGNMENT;
    const DeviceInfo *dev = nullptr;
    st = check_arch(&dev);
    if (st != SOL_OK) return st;
    return launch_gemm_bf16(x_bf16, w_bf16, bias_bf16, y_bf16, M, N, K, ldx, ldw, ldy,
                            static_cast<cudaStream_t>(stream), dev);
}

sol_status_t nvfp4_linear_quantized_out(const void *xq, const void *xsf, const float *x_tscale, const void *wq,
                                        const void *wsf, const float *w_tscale, const void *bias_bf16,
                                        sol_activation_t activation, const float *out_tscale, void *hq_out,
                                        void *hsf_out, float *amax_out, int64_t M, int64_t N, int64_t K, void *stream) {
    if (xq == nullptr || xsf == nullptr || x_tscale == nullptr || wq == nullptr || wsf == nullptr ||
        w_tscale == nullptr || out_tscale == nullptr || hq_out == nullptr || hsf_out == nullptr)
        return SOL_ERR_NULL_POINTER;
    if (!shape_ok(M, K) || N <= 0 || N % 64 != 0 || N > (1LL << 24)) return SOL_ERR_BAD_SHAPE;
    if (activation != SOL_ACT_NONE && activation != SOL_ACT_GELU_TANH) return SOL_ERR_BAD_LAYOUT;
    if (!aligned16(xq) || !aligned16(xsf) || !aligned16(wq) || !aligned16(wsf) || !aligned16(hq_out) ||
        !aligned16(hsf_out) || (bias_bf16 != nullptr && !aligned16(bias_bf16)) ||
        (reinterpret_cast<uintptr_t>(x_tscale) & 3u) || (reinterpret_cast<uintptr_t>(w_tscale) & 3u) ||
        (reinterpret_cast<uintptr_t>(out_tscale) & 3u) || (reinterpret_cast<uintptr_t>(amax_out) & 3u))
        return SOL_ERR_ALIGNMENT;
    const DeviceInfo *dev = nullptr;
    sol_status_t st = check_arch(&dev);
    if (st != SOL_OK) return st;
    return gemm::launch_pair256_nvfp4_quant_out(xq, xsf, x_tscale, wq, wsf, w_tscale, bias_bf16,
                                                activation == SOL_ACT_GELU_TANH ? 1 : 0, out_tscale, hq_out, hsf_out,
                                                reinterpret_cast<uint32_t *>(amax_out), M, N, K,
                                                static_cast<cudaStream_t>(stream), dev);
}

size_t sol_mxfp4_scale_bytes(int64_t rows, int64_t K, sol_sf_layout_t layout) {
    if (!shape_ok(rows, K)) return 0;
    if (layout == SOL_SF_ROW_MAJOR) return static_cast<size_t>(rows) * static_cast<size_t>(K / 32);
    if (layout == SOL_SF_SWIZZLED_128x4)
        return static_cast<size_t>(ceil_div(rows, 128)) * static_cast<size_t>(ceil_div(K, 128)) * 512;
    return 0;
}

sol_status_t mxfp4_quantize(const void *x_bf16, int64_t rows, int64_t K, int64_t ldx, void *q_out, void *sf_out,
                            sol_sf_layout_t layout, void *stream) {
    if (x_bf16 == nullptr || q_out == nullptr || sf_out == nullptr) return SOL_ERR_NULL_POINTER;
    if (!shape_ok(rows, K) || ldx < K) return SOL_ERR_BAD_SHAPE;
    if (layout != SOL_SF_ROW_MAJOR && layout != SOL_SF_SWIZZLED_128x4) return SOL_ERR_BAD_LAYOUT;
    if (!aligned16(x_bf16) || !aligned16(q_out) || !aligned16(sf_out) || ldx % 8 != 0) return SOL_ERR_ALIGNMENT;
    const DeviceInfo *dev = nullptr;
    sol_status_t st = check_arch(&dev);
    if (st != SOL_OK) return st;
    return launch_mxfp4_quantize(x_bf16, rows, K, ldx, q_out, sf_out, layout, static_cast<cudaStream_t>(stream));
}

sol_status_t mxfp4_linear(const void *xq, const void *xsf, const void *wq, const void *wsf, const void *bias_bf16,
                          void *y_bf16, int64_t M, int64_t N, int64_t K, int64_t ldy, void *stream) {
    if (xq == nullptr || xsf == nullptr || wq == nullptr || wsf == nullptr || y_bf16 == nullptr)
        return SOL_ERR_NULL_POINTER;
    sol_status_t st = check_linear_common(bias_bf16, y_bf16, M, N, K, ldy);
    if (st != SOL_OK) return st;
    if (!aligned16(xq) || !aligned16(xsf) || !aligned16(wq) || !aligned16(wsf)) return SOL_ERR_ALIGNMENT;
    const DeviceInfo *dev = nullptr;
    st = check_arch(&dev);
    if (st != SOL_OK) return st;
    return gemm::launch_pair256_mxfp4(xq, xsf, wq, wsf, bias_bf16, y_bf16, M, N, K, ldy,
                                      static_cast<cudaStream_t>(stream), dev);
}

sol_status_t mxfp4_linear_quantized_out(const void *xq, const void *xsf, const void *wq, const void *wsf,
                                        const void *bias_bf16, sol_activation_t activation, void *hq_out, void *hsf_out,
                                        float *amax_out, int64_t M, int64_t N, int64_t K, void *stream) {
    if (xq == nullptr || xsf == nullptr || wq == nullptr || wsf == nullptr || hq_out == nullptr || hsf_out == nullptr)
        return SOL_ERR_NULL_POINTER;
    if (!shape_ok(M, K) || N <= 0 || N % 128 != 0 || N > (1LL << 24)) return SOL_ERR_BAD_SHAPE;
    if (activation != SOL_ACT_NONE && activation != SOL_ACT_GELU_TANH) return SOL_ERR_BAD_LAYOUT;
    if (!aligned16(xq) || !aligned16(xsf) || !aligned16(wq) || !aligned16(wsf) || !aligned16(hq_out) ||
        !aligned16(hsf_out) || (bias_bf16 != nullptr && !aligned16(bias_bf16)) ||
        (reinterpret_cast<uintptr_t>(amax_out) & 3u))
        return SOL_ERR_ALIGNMENT;
    const DeviceInfo *dev = nullptr;
    sol_status_t st = check_arch(&dev);
    if (st != SOL_OK) return st;
    return gemm::launch_pair256_mxfp4_quant_out(xq, xsf, wq, wsf, bias_bf16, activation == SOL_ACT_GELU_TANH ? 1 : 0,
                                                hq_out, hsf_out, reinterpret_cast<uint32_t *>(amax_out), M, N, K,
                                                static_cast<cudaStream_t>(stream), dev);
}

sol_status_t mxfp4_linear_split_out(const void *xq, const void *xsf, const void *wq, const void *wsf,
                                    const void *bias_bf16, void *y_bf16, int64_t ldy, int64_t n_split,
                                    sol_activation_t activation, void *hq_dest, void *hsf_dest, int64_t dest_K,
                                    int64_t dest_col0, float *amax_out, int64_t M, int64_t N, int64_t K, void *stream) {
    if (xq == nullptr || xsf == nullptr || wq == nullptr || wsf == nullptr || y_bf16 == nullptr || hq_dest == nullptr ||
        hsf_dest == nullptr)
        return SOL_ERR_NULL_POINTER;
    if (!shape_ok(M, K) || N <= 0 || N > (1LL << 24) || n_split <= 0 || n_split >= N || n_split % 256 != 0 ||
        (N - n_split) % 128 != 0 || ldy < n_split || dest_K <= 0 || dest_K % 128 != 0 || dest_col0 < 0 ||
        dest_col0 % 128 != 0 || dest_col0 + (N - n_split) > dest_K)
        return SOL_ERR_BAD_SHAPE;
    if (activation != SOL_ACT_NONE && activation != SOL_ACT_GELU_TANH) return SOL_ERR_BAD_LAYOUT;
    if (!aligned16(xq) || !aligned16(xsf) || !aligned16(wq) || !aligned16(wsf) || !aligned16(y_bf16) ||
        !aligned16(hq_dest) || !aligned16(hsf_dest) || ldy % 8 != 0 || (bias_bf16 != nullptr && !aligned16(bias_bf16)) ||
        (reinterpret_cast<uintptr_t>(amax_out) & 3u))
        return SOL_ERR_ALIGNMENT;
    const DeviceInfo *dev = nullptr;
    sol_status_t st = check_arch(&dev);
    if (st != SOL_OK) return st;
    return gemm::launch_pair256_mxfp4_split_out(xq, xsf, wq, wsf, bias_bf16, y_bf16, ldy, n_split,
                                                activation == SOL_ACT_GELU_TANH ? 1 : 0, hq_dest, hsf_dest, dest_K,
                                                dest_col0, reinterpret_cast<uint32_t *>(amax_out), M, N, K,
                                                static_cast<cudaStream_t>(stream), dev);
}

sol_status_t mxfp4_quantize_into(const void *x_bf16, int64_t M, int64_t K, int64_t ldx, void *q_dest, void *sf_dest,
                                 int64_t dest_K, int64_t dest_col0, void *stream) {
    if (x_bf16 == nullptr || q_dest == nullptr || sf_dest == nullptr) return SOL_ERR_NULL_POINTER;
    if (!shape_ok(M, K) || ldx < K || K % 128 != 0 || dest_K <= 0 || dest_K % 128 != 0 || dest_col0 < 0 ||
        dest_col0 % 128 != 0 || dest_col0 + K > dest_K)
        return SOL_ERR_BAD_SHAPE;
    if (!aligned16(x_bf16) || !aligned16(q_dest) || !aligned16(sf_dest) || ldx % 8 != 0) return SOL_ERR_ALIGNMENT;
    const DeviceInfo *dev = nullptr;
    sol_status_t st = check_arch(&dev);
    if (st != SOL_OK) return st;
    return launch_mxfp4_quantize_into(x_bf16, M, K, ldx, q_dest, sf_dest, dest_K, dest_col0,
                                      static_cast<cudaStream_t>(stream));
}

sol_status_t solrl_select_contrastive(const float *rewards, const uint64_t *seeds, int64_t P, int64_t N, int64_t K,
                                      int32_t *idx_out, uint64_t *seeds_out, float *advantages_out, void *stream) {
    if (rewards == nullptr || idx_out == nullptr || (seeds_out != nullptr && seeds == nullptr)) return SOL_ERR_NULL_POINTER;
    if (P <= 0 || P > 0x7FFFFFFF || N <= 0 || N > selection_max_candidates() || K <= 0 || K % 2 != 0 || K > N)
        return SOL_ERR_BAD_SHAPE;
    if ((reinterpret_cast<uintptr_t>(rewards) & 3u) || (reinterpret_cast<uintptr_t>(idx_out) & 3u) ||
        (reinterpret_cast<uintptr_t>(seeds) & 7u) || (reinterpret_cast<uintptr_t>(seeds_out) & 7u) ||
        (reinterpret_cast<uintptr_t>(advantages_out) & 3u))
        return SOL_ERR_ALIGNMENT;
    const DeviceInfo *dev = nullptr;
    sol_status_t st = check_arch(&dev);
    if (st != SOL_OK) return st;
    return launch_select_contrastive(rewards, seeds, P, N, K, idx_out, seeds_out, advantages_out,
                                     static_cast<cudaStream_t>(stream));
}

sol_status_t solrl_rank_consistency(const float *rewards_ref, const float *rewards_proxy, int64_t P, int64_t N,
                                    int64_t k, int64_t *counts_out, float *metrics_out, void *stream) {
    if (rewards_ref == nullptr || rewards_proxy == nullptr || counts_out == nullptr) return SOL_ERR_NULL_POINTER;
    if (P <= 0 || P > 0x7FFFFFFF || N < 2 || 2 * N > selection_max_candidates() || k <= 0 || k > N)
        return SOL_ERR_BAD_SHAPE;
    if ((reinterpret_cast<uintptr_t>(rewards_ref) & 3u) || (reinterpret_cast<uintptr_t>(rewards_proxy) & 3u) ||
        (reinterpret_cast<uintptr_t>(counts_out) & 7u) || (reinterpret_cast<uintptr_t>(metrics_out) & 3u))
        return SOL_ERR_ALIGNMENT;
    const DeviceInfo *dev = nullptr;
    sol_status_t st = check_arch(&dev);
    if (st != SOL_OK) return st;
    return launch_rank_consistency(rewards_ref, rewards_proxy, P, N, k, counts_out, metrics_out,
                                   static_cast<cudaStream_t>(stream));
}

sol_status_t nvfp4_linear_split_out(const void *xq, const void *xsf, const float *x_tscale, const void *wq,
                                    const void *wsf, const float *w_tscale, const void *bias_bf16, void *y_bf16,
                                    int64_t ldy, int64_t n_split, sol_activation_t activation, const float *out_tscale,
                                    void *hq_dest, void *hsf_dest, int64_t dest_K, int64_t dest_col0, float *amax_out,
                                    int64_t M, int64_t N, int64_t K, void *stream) {
    if (xq == nullptr || xsf == nullptr || x_tscale == nullptr || wq == nullptr || wsf == nullptr ||
        w_tscale == nullptr || y_bf16 == nullptr || out_tscale == nullptr || hq_dest == nullptr || hsf_dest == nullptr)
        return SOL_ERR_NULL_POINTER;
    if (!shape_ok(M, K) || N <= 0 || N > (1LL << 24) || n_split <= 0 || n_split >= N || n_split % 256 != 0 ||
        (N - n_split) % 64 != 0 || ldy < n_split || dest_K <= 0 || dest_K % 64 != 0 || dest_col0 < 0 ||
        dest_col0 % 64 != 0 || dest_col0 + (N - n_split) > dest_K)
        return SOL_ERR_BAD_SHAPE;
    if (activation != SOL_ACT_NONE && activation != SOL_ACT_GELU_TANH) return SOL_ERR_BAD_LAYOUT;
    if (!aligned16(xq) || !aligned16(xsf) || !aligned16(wq) || !aligned16(wsf) || !aligned16(y_bf16) ||
        !aligned16(hq_dest) || !aligned16(hsf_dest) || ldy % 8 != 0 || (bias_bf16 != nullptr && !aligned16(bias_bf16)) ||
        (reinterpret_cast<uintptr_t>(x_tscale) & 3u) || (reinterpret_cast<uintptr_t>(w_tscale) & 3u) ||
        (reinterpret_cast<uintptr_t>(out_tscale) & 3u) || (reinterpret_cast<uintptr_t>(amax_out) & 3u))
        return SOL_ERR_ALIGNMENT;
    const DeviceInfo *dev = nullptr;
    sol_status_t st = check_arch(&dev);
    if (st != SOL_OK) return st;
    return gemm::launch_pair256_nvfp4_split_out(xq, xsf, x_tscale, wq, wsf, w_tscale, bias_bf16, y_bf16, ldy, n_split,
                                                activation == SOL_ACT_GELU_TANH ? 1 : 0, out_tscale, hq_dest, hsf_dest,
                                                dest_K, dest_col0, reinterpret_cast<uint32_t *>(amax_out), M, N, K,
                                                static_cast<cudaStream_t>(stream), dev);
}

sol_status_t nvfp4_quantize_into(const void *x_bf16, int64_t M, int64_t K, int64_t ldx, const float *tensor_scale,
                                 void *q_dest, void *sf_dest, int64_t dest_K, int64_t dest_col0, void *stream) {
    if (x_bf16 == nullptr || tensor_scale == nullptr || q_dest == nullptr || sf_dest == nullptr)
        return SOL_ERR_NULL_POINTER;
    if (!shape_ok(M, K) || ldx < K || K % 64 != 0 || dest_K <= 0 || dest_K % 64 != 0 || dest_col0 < 0 ||
        dest_col0 % 64 != 0 || dest_col0 + K > dest_K)
        return SOL_ERR_BAD_SHAPE;
    if (!aligned16(x_bf16) || !aligned16(q_dest) || !aligned16(sf_dest) || ldx % 8 != 0 ||
        (reinterpret_cast<uintptr_t>(tensor_scale) & 3u))
        return SOL_ERR_ALIGNMENT;
    const DeviceInfo *dev = nullptr;
    sol_status_t st = check_arch(&dev);
    if (st != SOL_OK) return st;
    return launch_quantize_into(x_bf16, M, K, ldx, tensor_scale, q_dest, sf_dest, dest_K, dest_col0,
                                static_cast<cudaStream_t>(stream));
}

sol_status_t nvfp4_layernorm_quantize(const void *x_bf16, int64_t M, int64_t K, int64_t ldx, const void *scale_bf16,
                                      const void *shift_bf16, int64_t rows_per_sample, float eps,
                                      const float *tensor_scale, void *q_out, void *sf_out, float *amax_out,
                                      void *stream) {
    if (x_bf16 == nullptr || scale_bf16 == nullptr || shift_bf16 == nullptr || tensor_scale == nullptr ||
        q_out == nullptr || sf_out == nullptr)
        return SOL_ERR_NULL_POINTER;
    if (!shape_ok(M, K) || K % 64 != 0 || K > layernorm_max_k() || ldx < K || rows_per_sample <= 0 || !(eps >= 0.0f))
        return SOL_ERR_BAD_SHAPE;
    if (!aligned16(x_bf16) || !aligned16(scale_bf16) || !aligned16(shift_bf16) || !aligned16(q_out) ||
        !aligned16(sf_out) || ldx % 8 != 0 || (reinterpret_cast<uintptr_t>(tensor_scale) & 3u) ||
        (reinterpret_cast<uintptr_t>(amax_out) & 3u))
        return SOL_ERR_ALIGNMENT;
    const DeviceInfo *dev = nullptr;
    sol_status_t st = check_arch(&dev);
    if (st != SOL_OK) return st;
    return launch_layernorm_quantize(x_bf16, M, K, ldx, scale_bf16, shift_bf16, rows_per_sample, eps, tensor_scale,
                                     q_out, sf_out, reinterpret_cast<uint32_t *>(amax_out),
                                     static_cast<cudaStream_t>(stream));
}

sol_status_t sol_attention_bf16(const void *q, const void *k, const void *v, void *out, int64_t batch, int64_t seq_q,
                                int64_t seq_kv, int64_t heads, int64_t head_dim, int64_t ld_q, int64_t ld_k, int64_t ld_v,
                                int64_t ld_out, void *stream) {
    if (q == nullptr || k == nullptr || v == nullptr || out == nullptr) return SOL_ERR_NULL_POINTER;
    if (head_dim != 64 && head_dim != 128) return SOL_ERR_BAD_SHAPE;
    const int64_t cols = heads * head_dim;
    if (batch <= 0 || seq_q <= 0 || seq_kv <= 0 || heads <= 0 || batch > 65535 || heads > 65535 ||
        seq_q > (1LL << 24) || seq_kv > (1LL << 24) || ld_q < cols || ld_k < cols || ld_v < cols || ld_out < cols)
        return SOL_ERR_BAD_SHAPE;
    if (!aligned16(q) || !aligned16(k) || !aligned16(v) || !aligned16(out) || ld_q % 8 != 0 || ld_k % 8 != 0 ||
        ld_v % 8 != 0 || ld_out % 8 != 0)
        return SOL_ERR_ALIGNMENT;
    const DeviceInfo *dev = nullptr;
    sol_status_t st = check_arch(&dev);
    if (st != SOL_OK) return st;
    const attn::Stream b{q, k, v, out, seq_q, seq_kv, ld_q, ld_k, ld_v, ld_out};
    return attn::launch_attention(nullptr, b, batch, heads, head_dim, nullptr, static_cast<cudaStream_t>(stream));
}

sol_status_t sol_attention_nvfp4_out(const void *q, const void *k, const void *v, int64_t batch, int64_t seq_q,
                                     int64_t seq_kv, int64_t heads, int64_t head_dim, int64_t ld_q, int64_t ld_k, int64_t ld_v,
                                     const float *out_tscale, void *q_dest, void *sf_dest, int64_t dest_K,
                                     int64_t dest_col0, float *amax_out, void *stream) {
    if (q == nullptr || k == nullptr || v == nullptr || out_tscale == nullptr || q_dest == nullptr || sf_dest == nullptr)
        return SOL_ERR_NULL_POINTER;
    if (head_dim != 64 && head_dim != 128) return SOL_ERR_BAD_SHAPE;
    const int64_t cols = heads * head_dim;
    if (batch <= 0 || seq_q <= 0 || seq_kv <= 0 || heads <= 0 || batch > 65535 || heads > 65535 ||
        seq_q > (1LL << 24) || seq_kv > (1LL << 24) || ld_q < cols || ld_k < cols || ld_v < cols || dest_K <= 0 ||
        dest_K % 64 != 0 || dest_col0 < 0 || dest_col0 % 64 != 0 || dest_col0 + cols > dest_K || dest_K > (1LL << 24) ||
        batch * seq_q > (1LL << 30))
        return SOL_ERR_BAD_SHAPE;
    if (!aligned16(q) || !aligned16(k) || !aligned16(v) || !aligned16(q_dest) || !aligned16(sf_dest) || ld_q % 8 != 0 ||
        ld_k % 8 != 0 || ld_v % 8 != 0 || (reinterpret_cast<uintptr_t>(out_tscale) & 3u) ||
        (reinterpret_cast<uintptr_t>(amax_out) & 3u))
        return SOL_ERR_ALIGNMENT;
    const DeviceInfo *dev = nullptr;
    sol_status_t st = check_arch(&dev);
    if (st != SOL_OK) return st;
    const attn::Stream b{q, k, v, nullptr, seq_q, seq_kv, ld_q, ld_k, ld_v, cols};
    const attn::QuantDest qd{q_dest, sf_dest, out_tscale, reinterpret_cast<uint32_t *>(amax_out), dest_K, dest_col0};
    return attn::launch_attention(nullptr, b, batch, heads, head_dim, &qd, static_cast<cudaStream_t>(stream));
}

sol_status_t sol_attention_bf16_joint(const sol_attention_stream_t *first, const sol_attention_stream_t *second,
                                      int64_t batch, int64_t heads, int64_t head_dim, void *stream) {
    if (first == nullptr || second == nullptr) return SOL_ERR_NULL_POINTER;
    if (head_dim != 64 && head_dim != 128) return SOL_ERR_BAD_SHAPE;
    const sol_attention_stream_t *both[2] = {first, second};
    const int64_t cols = heads * head_dim;
    if (batch <= 0 || heads <= 0 || batch > 65535 || heads > 65535) return SOL_ERR_BAD_SHAPE;
    for (const sol_attention_stream_t *s : both) {
        if (s->q == nullptr || s->k == nullptr || s->v == nullptr || s->out == nullptr) return SOL_ERR_NULL_POINTER;
        if (s->seq <= 0 || s->seq > (1LL << 24) || s->ld_q < cols || s->ld_k < cols || s->ld_v < cols || s->ld_out < cols)
            return SOL_ERR_BAD_SHAPE;
        if (!aligned16(s->q) || !aligned16(s->k) || !aligned16(s->v) || !aligned16(s->out) || s->ld_q % 8 != 0 ||
            s->ld_k % 8 != 0 || s->ld_v % 8 != 0 || s->ld_out % 8 != 0)
            return SOL_ERR_ALIGNMENT;
    }
    if (first->seq % 256 != 0) return SOL_ERR_BAD_SHAPE;  // the first stream must fill whole query-tile pairs
    const DeviceInfo *dev = nullptr;
    sol_status_t st = check_arch(&dev);
    if (st != SOL_OK) return st;
    const attn::Stream a{first->q, first->k, first->v, first->out, first->seq, first->seq,
                         first->ld_q, first->ld_k, first->ld_v, first->ld_out};
    const attn::Stream b{second->q, second->k, second->v, second->out, second->seq, second->seq,
                         second->ld_q, second->ld_k, second->ld_v, second->ld_out};
    return attn::launch_attention(&a, b, batch, heads, head_dim, nullptr, static_cast<cudaStream_t>(stream));
}

sol_status_t nvfp4_quantize_linear(const void *x_bf16, int64_t ldx, const void *wq, const void *wsf,
                                   const float *w_tscale, const void *bias_bf16, void *y_bf16, int64_t M,
                                   int64_t N, int64_t K, int64_t ldy, void *workspace, size_t workspace_bytes,
                                   void *stream) {
    if (x_bf16 == nullptr || wq == nullptr || wsf == nullptr || w_tscale == nullptr || y_bf16 == nullptr ||
        workspace == nullptr)
        return SOL_ERR_NULL_POINTER;
    sol_status_t st = check_linear_common(bias_bf16, y_bf16, M, N, K, ldy);
    if (st != SOL_OK) return st;
    if (ldx < K) return SOL_ERR_BAD_SHAPE;
    if (!aligned16(x_bf16) || !aligned16(wq) || !aligned16(wsf) || ldx % 8 != 0 ||
        (reinterpret_cast<uintptr_t>(w_tscale) & 3u) || (reinterpret_cast<uintptr_t>(workspace) & 255u))
        return SOL_ERR_ALIGNMENT;
    if (workspace_bytes < sol_nvfp4_linear_workspace_bytes(M, N, K)) return SOL_ERR_WORKSPACE_TOO_SMALL;
    const DeviceInfo *dev = nullptr;
    st = check_arch(&dev);
    if (st != SOL_OK) return st;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    uint8_t *ws = static_cast<uint8_t *>(workspace);
    uint8_t *xq = ws;
    uint8_t *xsf = xq + align256(sol_nvfp4_data_bytes(M, K));
    float *xts = reinterpret_cast<float *>(xsf + align256(sol_nvfp4_scale_bytes(M, K, SOL_SF_SWIZZLED_128x4)));
    st = launch_amax_quantize(x_bf16, M, K, ldx, xts, xq, xsf, SOL_SF_SWIZZLED_128x4, s, dev);
    if (st != SOL_OK) return st;
    return launch_gemm_nvfp4(xq, xsf, xts, wq, wsf, w_tscale, bias_bf16, y_bf16, M, N, K, ldy, s, dev);
}

sol_status_t nvfp4_quantize_linear_delayed(const void *x_bf16, int64_t ldx, const void *wq, const void *wsf,
                                           const float *w_tscale, const void *bias_bf16, void *y_bf16, int64_t M,
                                           int64_t N, int64_t K, int64_t ldy, float *scale_state, void *workspace,
                                           size_t workspace_bytes, void *stream) {
    if (x_bf16 == nullptr || wq == nullptr || wsf == nullptr || w_tscale == nullptr || y_bf16 == nullptr ||
        workspace == nullptr || scale_state == nullptr)
        return SOL_ERR_NULL_POINTER;
    sol_status_t st = check_linear_common(bias_bf16, y_bf16, M, N, K, ldy);
    if (st != SOL_OK) return st;
    if (ldx < K) return SOL_ERR_BAD_SHAPE;
    if (!aligned16(x_bf16) || ldx % 8 != 0 || !aligned16(wq) || !aligned16(wsf) ||
        (reinterpret_cast<uintptr_t>(w_tscale) & 3u) || (reinterpret_cast<uintptr_t>(workspace) & 255u) ||
        (reinterpret_cast<uintptr_t>(scale_state) & 7u))
        return SOL_ERR_ALIGNMENT;
    if (workspace_bytes < sol_nvfp4_linear_workspace_bytes(M, N, K)) return SOL_ERR_WORKSPACE_TOO_SMALL;
    const DeviceInfo *dev = nullptr;
    st = check_arch(&dev);
    if (st != SOL_OK) return st;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    uint8_t *ws = static_cast<uint8_t *>(workspace);
    uint8_t *xq = ws;
    uint8_t *xsf = xq + align256(sol_nvfp4_data_bytes(M, K));
    st = launch_quantize_tracking(x_bf16, M, K, ldx, scale_state, xq, xsf, reinterpret_cast<uint32_t *>(scale_state + 1),
                                  s);
    if (st != SOL_OK) return st;
    return launch_gemm_nvfp4(xq, xsf, scale_state, wq, wsf, w_tscale, bias_bf16, y_bf16, M, N, K, ldy, s, dev);
}

sol_status_t sol_roll_tensor_scale(float *scale_state, void *stream) {
    if (scale_state == nullptr) return SOL_ERR_NULL_POINTER;
    if (reinterpret_cast<uintptr_t>(scale_state) & 7u) return SOL_ERR_ALIGNMENT;
    const DeviceInfo *dev = nullptr;
    sol_status_t st = check_arch(&dev);
    if (st != SOL_OK) return st;
    return launch_roll_scale(scale_state, static_cast<cudaStream_t>(stream));
}

sol_status_t nvfp4_quantize_linear_host(const void *x_host, int64_t ldx, const void *wq, const void *wsf,
                                        const float *w_tscale, const void *bias_bf16, void *y_host, int64_t M,
                                        int64_t N, int64_t K, int64_t ldy, void *x_dev, void *y_dev,
                                        void *workspace, size_t workspace_bytes, void *stream) {
    if (x_host == nullptr || y_host == nullptr || x_dev == nullptr || y_dev == nullptr) return SOL_ERR_NULL_POINTER;
    if (M <= 0 || N <= 0 || K <= 0 || ldx < K || ldy < N) return SOL_ERR_BAD_SHAPE;
    // validate everything else (and the device) before the first copy is queued
    if (wq == nullptr || wsf == nullptr || w_tscale == nullptr || workspace == nullptr) return SOL_ERR_NULL_POINTER;
    sol_status_t st = check_linear_common(bias_bf16, y_dev, M, N, K, N);
    if (st != SOL_OK) return st;
    if (!aligned16(x_dev) || !aligned16(wq) || !aligned16(wsf) || (reinterpret_cast<uintptr_t>(w_tscale) & 3u) ||
        (reinterpret_cast<uintptr_t>(workspace) & 255u))
        return SOL_ERR_ALIGNMENT;
    if (workspace_bytes < sol_nvfp4_linear_workspace_bytes(M, N, K)) return SOL_ERR_WORKSPACE_TOO_SMALL;
    const DeviceInfo *dev = nullptr;
    st = check_arch(&dev);
    if (st != SOL_OK) return st;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    if (cudaMemcpy2DAsync(x_dev, static_cast<size_t>(K) * 2, x_host, static_cast<size_t>(ldx) * 2,
                          static_cast<size_t>(K) * 2, static_cast<size_t>(M), cudaMemcpyHostToDevice, s) != cudaSuccess)
        return SOL_ERR_CUDA;
    st = nvfp4_quantize_linear(x_dev, K, wq, wsf, w_tscale, bias_bf16, y_dev, M, N, K, N, workspace, workspace_bytes,
                               stream);
    if (st != SOL_OK) return st;
    if (cudaMemcpy2DAsync(y_host, static_cast<size_t>(ldy) * 2, y_dev, static_cast<size_t>(N) * 2,
                          static_cast<size_t>(N) * 2, static_cast<size_t>(M), cudaMemcpyDeviceToHost, s) != cudaSuccess)
        return SOL_ERR_CUDA;
    return SOL_OK;
}

sol_status_t sol_set_wait_limit_cycles(int64_t cycles) {
    const DeviceInfo *dev = nullptr;
    sol_status_t st = check_arch(&dev);
    if (st != SOL_OK) return st;
    const long long limit = cycles > 0 ? static_cast<long long>(cycles) : kDefaultWaitLimitCycles;
    if (cudaMemcpyToSymbol(g_status_block, &limit, sizeof(limit), offsetof(DeviceStatusBlock, wait_limit_cycles)) !=
        cudaSuccess)
        return SOL_ERR_CUDA;
    return SOL_OK;
}

sol_status_t sol_test_hold_loads(int on) {
    const DeviceInfo *dev = nullptr;
    sol_status_t st = check_arch(&dev);
    if (st != SOL_OK) return st;
    const uint32_t flag = on ? 1u : 0u;
    if (cudaMemcpyToSymbol(g_status_block, &flag, sizeof(flag), offsetof(DeviceStatusBlock, hold_loads)) != cudaSuccess)
        return SOL_ERR_CUDA;
    return SOL_OK;
}

sol_status_t sol_last_device_status(void *stream, uint32_t *detail_out) {
    const DeviceInfo *dev = nullptr;
    sol_status_t st = check_arch(&dev);
    if (st != SOL_OK) return st;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    uint32_t word = 0;
    if (cudaStreamSynchronize(s) != cudaSuccess) return SOL_ERR_CUDA;
    if (cudaMemcpyFromSymbol(&word, g_status_block, sizeof(word)) != cudaSuccess) return SOL_ERR_CUDA;
    if (detail_out != nullptr) *detail_out = word;
    if (word != 0) {
        const uint32_t zero = 0;
        if (cudaMemcpyToSymbol(g_status_block, &zero, sizeof(zero)) != cudaSuccess) return SOL_ERR_CUDA;
        return SOL_ERR_TIMEOUT;
    }
    return SOL_OK;
}

}  // extern "C"
