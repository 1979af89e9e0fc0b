// Host-side helpers shared by the entry points: argument checks, device query, launch checks.
#pragma once
#include <cstdio>
#include <cstdlib>
#include <cuda.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "../../include/sol_nvfp4.h"

namespace sol {

inline bool aligned16(const void *p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }
inline int64_t ceil_div(int64_t a, int64_t b) { return (a + b - 1) / b; }

struct DeviceInfo {
    int device = -1;
    int sm_count = 0;
    int cc_major = 0;
    int cc_minor = 0;
    bool ok = false;
};

// Properties of the current device (queried once per device, cached on the host).
const DeviceInfo *current_device_info();

// SOL_OK when the current device is an sm_100 part, SOL_ERR_UNSUPPORTED_ARCH / SOL_ERR_CUDA otherwise.
sol_status_t check_arch(const DeviceInfo **info_out);

inline sol_status_t launch_status() {
    const cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess && getenv("SOL_NVFP4_VERBOSE") != nullptr)
        fprintf(stderr, "sol_nvfp4: launch failed: %s\n", cudaGetErrorString(e));
    return e == cudaSuccess ? SOL_OK : SOL_ERR_CUDA;
}

// Device status block, one per device.  `code` is written by a bounded wait that ran out (0 = none)
// and read and cleared by sol_last_device_status; `wait_limit_cycles` is the limit of every bounded
// wait in SM cycles (sol_set_wait_limit_cycles); `hold_loads` is the test hook of
// sol_test_hold_loads: while non-zero the load-issuing warps of the CTA-pair GEMM kernels issue
// nothing, so every consumer wait of those kernels runs into the limit.
struct DeviceStatusBlock {
    uint32_t code;
    uint32_t hold_loads;
    long long wait_limit_cycles;
};
constexpr long long kDefaultWaitLimitCycles = 4000000000LL;
// Pointer to the block's first word (kernels receive it as `status`; words 1.. follow the struct).
uint32_t *device_status_word();

// Internal launchers (arguments already validated).
sol_status_t launch_amax(const void *x, int64_t rows, int64_t K, int64_t ld, float *tscale_out,
                         cudaStream_t stream, const DeviceInfo *dev);
sol_status_t launch_quantize(const void *x, int64_t rows, int64_t K, int64_t ld, const float *tscale,
                             void *q, void *sf, sol_sf_layout_t layout, cudaStream_t stream);
// Per-tensor scale and quantizer in two kernels: scale_words[1] receives max|x| (as FP32 bits),
// the quantizer derives T from it and publishes T in scale_words[0].
sol_status_t launch_amax_quantize(const void *x, int64_t rows, int64_t K, int64_t ld, float *scale_words,
                                  void *q, void *sf, sol_sf_layout_t layout, cudaStream_t stream,
                                  const DeviceInfo *dev);
// Quantizer that derives T from max|x| left in scale_words[1] (FP32 bits) and publishes T in scale_words[0].
sol_status_t launch_quantize_from_amax(const void *x, int64_t rows, int64_t K, int64_t ld, float *scale_words,
                                       void *q, void *sf, sol_sf_layout_t layout, cudaStream_t stream,
                                       bool reverse = false);
// Groups of equally shaped matrices handled by one launch (blockIdx.z picks the matrix).
constexpr int kMaxGroup = 8;
struct MergeGroup {
    const uint16_t *w[kMaxGroup];   // base weights [N, K], pitch ldw
    const uint16_t *a[kMaxGroup];   // adapter down factors [r, K], pitch lda
    const uint16_t *b[kMaxGroup];   // adapter up factors [N, r], pitch ldb
    uint16_t *out[kMaxGroup];       // merged weights, dense [N, K]
    float *scale_words[kMaxGroup];  // [0]: T (written by the quantizer), [1]: max|W'| as FP32 bits
};
struct QuantGroup {
    const uint16_t *x[kMaxGroup];   // dense [rows, K]
    float *scale_words[kMaxGroup];
    uint8_t *q[kMaxGroup];
    uint8_t *sf[kMaxGroup];
};
// Adapter merge W' = bf16(W + s * B A) for `count` matrices: zeroes each scale_words[i][1], then
// accumulates max|W'| into it as FP32 bits.
sol_status_t launch_lora_merge(const MergeGroup &g, int count, int64_t ldw, int64_t lda, int64_t ldb, int64_t N,
                               int64_t K, int64_t r, float s, cudaStream_t stream);
sol_status_t launch_quantize_group(const QuantGroup &g, int count, int64_t rows, int64_t K, sol_sf_layout_t layout,
                                   cudaStream_t stream);
int lora_max_rank();
// Quantizes x [rows, K] into columns [dest_col0, dest_col0 + K) of a wider quantized tensor [rows, dest_K]
// (chunked scale layout; K, dest_K and dest_col0 multiples of 64).
sol_status_t launch_quantize_into(const void *x, int64_t rows, int64_t K, int64_t ld, const float *tscale, void *q,
                                  void *sf, int64_t dest_K, int64_t dest_col0, cudaStream_t stream);
// Quantizer with a caller-supplied T that also collects max|x| into *amax_track (atomicMax on FP32 bits).
sol_status_t launch_quantize_tracking(const void *x, int64_t rows, int64_t K, int64_t ld, const float *tscale, void *q,
                                      void *sf, uint32_t *amax_track, cudaStream_t stream);
// state[0] <- T(state[1]); state[1] <- 0.
sol_status_t launch_roll_scale(float *state, cudaStream_t stream);
// Layer norm + per-sample modulation + NVFP4 quantizer in one pass (K a multiple of 64, K <= layernorm_max_k()).
sol_status_t launch_layernorm_quantize(const void *x, int64_t rows, int64_t K, int64_t ld, const void *scale,
                                       const void *shift, int64_t rows_per_sample, float eps, const float *tscale,
                                       void *q, void *sf, uint32_t *amax_track, cudaStream_t stream);
int layernorm_max_k();
sol_status_t launch_mxfp4_quantize(const void *x, int64_t rows, int64_t K, int64_t ld, void *q, void *sf,
                                   sol_sf_layout_t layout, cudaStream_t stream);
// The same into columns [dest_col0, dest_col0 + K) of a wider MXFP4 tensor [rows, dest_K] (chunked scales;
// K, dest_K and dest_col0 multiples of 128).
sol_status_t launch_mxfp4_quantize_into(const void *x, int64_t rows, int64_t K, int64_t ld, void *q, void *sf,
                                        int64_t dest_K, int64_t dest_col0, cudaStream_t stream);
// Stage-1 selection and rank-consistency metrics (one block per prompt).
sol_status_t launch_select_contrastive(const float *rewards, const uint64_t *seeds, int64_t P, int64_t N, int64_t K,
                                       int32_t *idx_out, uint64_t *seeds_out, float *adv_out, cudaStream_t stream);
sol_status_t launch_rank_consistency(const float *ref, const float *proxy, int64_t P, int64_t N, int64_t k,
                                     int64_t *counts_out, float *metrics_out, cudaStream_t stream);
int selection_max_candidates();
sol_status_t launch_gemm_bf16(const void *x, const void *w, const void *bias, void *y, int64_t M,
                              int64_t N, int64_t K, int64_t ldx, int64_t ldw, int64_t ldy,
                              cudaStream_t stream, const DeviceInfo *dev);
sol_status_t launch_gemm_nvfp4(const void *xq, const void *xsf, const float *xts, const void *wq,
                               const void *wsf, const float *wts, const void *bias, void *y,
                               int64_t M, int64_t N, int64_t K, int64_t ldy, cudaStream_t stream,
                               const DeviceInfo *dev);

// 2-D row-major tensor map: `inner` contiguous elements per row, `outer` rows, row pitch in bytes.
// Returns false if the driver rejects it.
bool make_tmap_2d(CUtensorMap *out, CUtensorMapDataType dtype, uint32_t elem_bytes, const void *base,
                  uint64_t inner, uint64_t outer, uint64_t pitch_bytes, uint32_t box_inner,
                  uint32_t box_outer, CUtensorMapSwizzle swizzle);

// [d2][d1][d0] BF16 tensor with byte pitches between rows (d1) and slabs (d2); 128-byte swizzle, boxes of
// box0 x box1 x 1 elements.
bool make_tmap_3d_bf16(CUtensorMap *out, const void *base, uint64_t d0, uint64_t d1, uint64_t d2, uint64_t pitch1_bytes,
                       uint64_t pitch2_bytes, uint32_t box0, uint32_t box1);

namespace attn {
struct Stream {   // one token stream of an attention call: [batch, seq, heads, head_dim] views with token pitches
    const void *q, *k, *v;
    void *out;
    int64_t seq_q, seq_kv, ld_q, ld_k, ld_v, ld_out;
};
struct QuantDest {   // NVFP4 destination of the output: columns [dest_col0, dest_col0 + heads * head_dim) of a [rows, dest_K] tensor
    void *q, *sf;
    const float *tscale;
    uint32_t *amax_out;
    int64_t dest_K, dest_col0;
};
// Attention over the concatenation (a, then b) of two token streams, or over b alone when a is null;
// with `qd` (one stream only) the output is quantized into `qd` instead of written as BF16.
sol_status_t launch_attention(const Stream *a, const Stream &b, int64_t batch, int64_t heads, int64_t head_dim,
                              const QuantDest *qd, cudaStream_t stream);
}

// Scale-factor buffer in the chunked layout as a 3-D tensor [row chunk][k chunk][128 x u32]; the box
// covers `box_k_chunks` k-chunks of `box_row_chunks` row chunks (out-of-range chunks read as zero).
bool make_tmap_sf(CUtensorMap *out, const void *base, uint64_t chunks_k, uint64_t row_chunks,
                  uint32_t box_row_chunks, uint32_t box_k_chunks = 4);

}  // namespace sol
