// NVFP4 quantizer kernels (per-tensor amax, activation / weight quantizer) for sm_100a.
//
// Q(x) = S * Pi_FP4(x / S) with S = E4M3 block scale * FP32 tensor scale T (paper Section 2).
// Both kernels are streaming codecs bound by HBM bandwidth: 16-byte loads, many loads in
// flight per thread, packed 8-byte nibble stores, scale bytes staged in shared memory and
// written as whole 512-byte chunks of the layout the tensor core consumes.
#include "quant_math.cuh"
#include "sol_internal.h"

namespace sol {
namespace {

constexpr int kQuantThreads = 256;
constexpr int kTileRows = 128;     // rows per block = one row tile of the chunked scale layout
constexpr int kTileK = 256;        // elements along K per block = 4 scale chunks = 16 scale blocks
constexpr int kBlocksPerThread = kTileRows * (kTileK / 16) / kQuantThreads;  // 8 scale blocks of 16 elements
constexpr int kBatch = 4;          // scale blocks (2 x 16-byte loads each) in flight per thread

using qmath::absmax2;
using qmath::bf16_hi;
using qmath::bf16_lo;
using qmath::e4m3_to_f32;
using qmath::f32_to_e4m3_sat;
using qmath::pack_e2m1x8;

__device__ __forceinline__ uint32_t abs_max_bits(const uint4 &v) {
    // per-halfword max of |bf16| bit patterns (magnitudes order like unsigned integers)
    const uint32_t m = absmax2(absmax2(v.x, v.y), absmax2(v.z, v.w)) & 0x7FFF7FFFu;
    return max(m & 0xFFFFu, m >> 16);
}

__device__ __forceinline__ uint32_t abs_max_bits(const uint4 &u, const uint4 &v) {
    const uint32_t m = absmax2(absmax2(absmax2(u.x, u.y), absmax2(u.z, u.w)),
                               absmax2(absmax2(v.x, v.y), absmax2(v.z, v.w))) & 0x7FFF7FFFu;
    return max(m & 0xFFFFu, m >> 16);
}

// Programmatic dependent launch: a kernel launched with the stream-serialization attribute may
// start while its predecessor in the stream is still draining; it must not touch global memory
// before grid_dependency_wait() returns (a no-op when there is nothing to wait for).
__device__ __forceinline__ void grid_dependency_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void grid_launch_dependents() { asm volatile("griddepcontrol.launch_dependents;"); }

__device__ __forceinline__ float tensor_scale_from_amax(float a) {
    return (a == 0.0f) ? 1.0f : __fdiv_rn(a, 2688.0f);
}

__device__ __forceinline__ uint32_t quantize8(const uint4 &v, float rcp) {
    return qmath::quantize8(v.x, v.y, v.z, v.w, rcp);
}

// Where the quantized tensor lands: normally a dense [rows, K/2] nibble matrix and its own scale
// buffer; for a slice of a wider tensor (one part of a concatenated activation) the row pitch, the
// byte column and the scale chunk column of the destination.
struct QuantDest {
    int64_t q_pitch;       // bytes between rows of the nibble matrix
    int64_t q_col0;        // first byte column
    int64_t sf_chunks_k;   // scale chunks per 128-row tile in the destination (chunked layout)
    int64_t sf_chunk0;     // first chunk column
    uint32_t *amax_track;  // nullable: running max|x| of the quantized tensor as FP32 bits (atomicMax)
};

// One block quantizes a 128-row x 256-element tile.  A thread owns whole scale blocks (16
// elements = two 16-byte loads, one 8-byte store, one scale byte), so the scale arithmetic runs
// once per 16 elements: the kernel has to stay under ~8 instructions per element to be bound
// by HBM rather than by instruction issue.  Thread t works on scale block t%16 of rows
// t/16 + 16*i; a warp reads two 512-byte row segments per step.
// With `amax` set the tensor scale is derived here from the amax word the reduction left (the
// bit pattern of max|x| as FP32) and block (0,0) publishes it in `tscale_out` for the GEMM.
template <bool kSwizzled>
__device__ __forceinline__ void quantize_tile(const uint16_t *__restrict__ x, int64_t rows, int64_t K, int64_t ld,
                                              const float *tscale, const float *amax, float *tscale_out,
                                              uint8_t *__restrict__ q, uint8_t *__restrict__ sf, const QuantDest dst,
                                              int64_t tile_k, int64_t tile_row) {
    __shared__ __align__(16) uint8_t sf_tile[kTileRows * (kTileK / 16)];  // 2 KB = 4 chunks
    // 1 / (float(sb) * T) for every scale byte: d takes at most 127 values per tensor, so the decode,
    // the multiplication and the IEEE reciprocal run once per thread block instead of once per scale block
    __shared__ float rcp_tab[128];

    const int b = threadIdx.x & 15;   // scale block inside the tile
    const int r0 = threadIdx.x >> 4;  // first row inside the tile
    const int64_t row0 = tile_row * kTileRows;
    const int64_t k = tile_k * kTileK + b * 16;
    const bool k_ok = k < K;

    if (kSwizzled) {
        reinterpret_cast<uint64_t *>(sf_tile)[threadIdx.x] = 0;  // padding bytes must read as 0
        __syncthreads();
    }

    grid_dependency_wait();
    grid_launch_dependents();
    const float T = amax != nullptr ? tensor_scale_from_amax(*amax) : *tscale;
    if (tscale_out != nullptr && threadIdx.x == 0 && tile_k == 0 && tile_row == 0) *tscale_out = T;
    const float c = __fmul_rn(6.0f, T);
    const int64_t nb = K >> 4;
    if (threadIdx.x < 128) {
        const uint32_t code = threadIdx.x;
        rcp_tab[code] = code ? __frcp_rn(__fmul_rn(e4m3_to_f32(code), T)) : 0.0f;
    }
    __syncthreads();

    uint32_t seen_max = 0;  // BF16 magnitude bits of the largest element this thread has quantized
#pragma unroll 1
    for (int batch = 0; batch < kBlocksPerThread / kBatch; ++batch) {
        uint4 lo[kBatch], hi[kBatch];
#pragma unroll
        for (int i = 0; i < kBatch; ++i) {
            const int64_t r = row0 + r0 + 16 * (batch * kBatch + i);
            lo[i] = hi[i] = make_uint4(0, 0, 0, 0);
            if (k_ok && r < rows) {
                const uint4 *src = reinterpret_cast<const uint4 *>(x + r * ld + k);
                lo[i] = __ldcs(src);
                hi[i] = __ldcs(src + 1);
            }
        }
#pragma unroll
        for (int i = 0; i < kBatch; ++i) {
            const int rl = r0 + 16 * (batch * kBatch + i);  // row inside the tile
            const int64_t r = row0 + rl;
            const uint32_t abits = abs_max_bits(lo[i], hi[i]);
            seen_max = max(seen_max, abits);
            const float a = __uint_as_float(abits << 16);
            const float sv = __fdiv_rn(a, c);
            const uint32_t sb = f32_to_e4m3_sat(sv);
            const float rcp = rcp_tab[sb];
            const uint64_t rcp2 = qmath::f32x2(rcp, rcp);   // the sixteen products two at a time (same roundings)
            uint2 packed;
            packed.x = qmath::quantize8_x2(lo[i].x, lo[i].y, lo[i].z, lo[i].w, rcp2);
            packed.y = qmath::quantize8_x2(hi[i].x, hi[i].y, hi[i].z, hi[i].w, rcp2);
            if (k_ok && r < rows) {
                __stcs(reinterpret_cast<uint2 *>(q + r * dst.q_pitch + dst.q_col0 + (k >> 1)), packed);
                if (kSwizzled) {
                    sf_tile[(b >> 2) * 512 + (rl & 31) * 16 + (rl >> 5) * 4 + (b & 3)] = static_cast<uint8_t>(sb);
                } else {
                    sf[r * nb + (k >> 4)] = static_cast<uint8_t>(sb);
                }
            }
        }
    }

    if (kSwizzled) {
        __syncthreads();
        // 4 chunks x 32 lines of 16 bytes; chunk c of this tile is k chunk tile_k*4 + c
        const int64_t chunks_k = (nb + 3) >> 2;
        if (threadIdx.x < 128) {
            const int cidx = threadIdx.x >> 5;
            const int64_t kc = tile_k * 4 + cidx;
            if (kc < chunks_k) {
                uint8_t *out = sf + (tile_row * dst.sf_chunks_k + dst.sf_chunk0 + kc) * 512 +
                               (threadIdx.x & 31) * 16;
                *reinterpret_cast<uint4 *>(out) = reinterpret_cast<const uint4 *>(sf_tile)[threadIdx.x];
            }
        }
    }
    if (dst.amax_track != nullptr) {  // the tensor's amax as a by-product, for the next call's tensor scale
        __shared__ uint32_t warp_seen[kQuantThreads / 32];
        seen_max = __reduce_max_sync(0xFFFFFFFFu, seen_max);
        if ((threadIdx.x & 31) == 0) warp_seen[threadIdx.x >> 5] = seen_max;
        __syncthreads();
        if (threadIdx.x < 32) {
            uint32_t m = threadIdx.x < kQuantThreads / 32 ? warp_seen[threadIdx.x] : 0;
            m = __reduce_max_sync(0xFFFFFFFFu, m);
            if (threadIdx.x == 0 && m) atomicMax(dst.amax_track, m << 16);
        }
    }
}

// One-dimensional grid over the tiles, k-tiles of a row tile adjacent.  With `reverse` the grid walks the
// tensor from its end: behind the amax pass (which reads the tensor front to back) the last rows are
// what the L2 still holds, so the quantizer's first reads hit there instead of going to HBM a second time.
template <bool kSwizzled>
__global__ void __launch_bounds__(kQuantThreads)
quantize_kernel(const uint16_t *__restrict__ x, int64_t rows, int64_t K, int64_t ld,
                const float *tscale, const float *amax, float *tscale_out, uint8_t *__restrict__ q,
                uint8_t *__restrict__ sf, const QuantDest dst, uint32_t k_tiles, int reverse) {
    const uint32_t t = reverse ? gridDim.x - 1u - blockIdx.x : blockIdx.x;
    const uint32_t tile_row = t / k_tiles;
    quantize_tile<kSwizzled>(x, rows, K, ld, tscale, amax, tscale_out, q, sf, dst, t - tile_row * k_tiles, tile_row);
}

// The same over a group of equally shaped dense tensors, one per blockIdx.z, each with its own
// amax word (the weight refresh quantizes several merged matrices per launch).
template <bool kSwizzled>
__global__ void __launch_bounds__(kQuantThreads)
quantize_group_kernel(const __grid_constant__ QuantGroup g, int64_t rows, int64_t K) {
    const int z = blockIdx.z;
    const QuantDest dst = {K >> 1, 0, ((K >> 4) + 3) >> 2, 0, nullptr};
    quantize_tile<kSwizzled>(g.x[z], rows, K, K, nullptr, g.scale_words[z] + 1, g.scale_words[z], g.q[z], g.sf[z], dst,
                             blockIdx.x, blockIdx.y);
}

// MXFP4 quantizer (the OCP format Section 2 sets beside NVFP4): 32 elements share one E8M0 scale
// 2^(floor(log2 amax) - 2); x / scale is an exact power-of-two scaling, so there is no division and no
// tensor-level scale.  One block = 128 rows x 512 elements (= four scale chunks of 128 x 4); a thread
// owns whole 32-element blocks: four 16-byte loads, one 16-byte store, one scale byte.
constexpr int kMxTileK = 512;
constexpr int kMxBlocksPerThread = kTileRows * (kMxTileK / 32) / kQuantThreads;  // 8

template <bool kSwizzled>
__global__ void __launch_bounds__(kQuantThreads)
mxfp4_quantize_kernel(const uint16_t *__restrict__ x, int64_t rows, int64_t K, int64_t ld, uint8_t *__restrict__ q,
                      uint8_t *__restrict__ sf, uint32_t k_tiles, const QuantDest dst) {
    const int64_t tile_row = blockIdx.x / k_tiles;
    const int64_t tile_k = blockIdx.x - static_cast<uint32_t>(tile_row) * k_tiles;
    __shared__ __align__(16) uint8_t sf_tile[kTileRows * (kMxTileK / 32)];  // 2 KB = 4 chunks
    const int b = threadIdx.x & 15;   // 32-element block inside the tile
    const int r0 = threadIdx.x >> 4;
    const int64_t row0 = tile_row * kTileRows;
    const int64_t k = tile_k * kMxTileK + b * 32;
    const bool k_ok = k < K;
    if (kSwizzled) {
        reinterpret_cast<uint64_t *>(sf_tile)[threadIdx.x] = 0;
        __syncthreads();
    }
    grid_dependency_wait();
    grid_launch_dependents();
    const int64_t nb = K >> 5;
#pragma unroll 1
    for (int batch = 0; batch < kMxBlocksPerThread / 2; ++batch) {
        uint4 v[2][4];
#pragma unroll
        for (int i = 0; i < 2; ++i) {
            const int64_t r = row0 + r0 + 16 * (batch * 2 + i);
#pragma unroll
            for (int u = 0; u < 4; ++u) v[i][u] = make_uint4(0, 0, 0, 0);
            if (k_ok && r < rows) {
                const uint4 *src = reinterpret_cast<const uint4 *>(x + r * ld + k);
#pragma unroll
                for (int u = 0; u < 4; ++u) v[i][u] = __ldcs(src + u);
            }
        }
#pragma unroll
        for (int i = 0; i < 2; ++i) {
            const int rl = r0 + 16 * (batch * 2 + i);
            const int64_t r = row0 + rl;
            const uint32_t m = max(abs_max_bits(v[i][0], v[i][1]), abs_max_bits(v[i][2], v[i][3]));
            const uint32_t e8 = m >> 7;                      // biased exponent of the block maximum
            const uint32_t sb = e8 > 2u ? e8 - 2u : 0u;      // shared exponent floor(log2 amax) - 2, clamped at -127
            const float inv = __uint_as_float((254u - sb) << 23);  // 2^(127 - sb), exact
            uint4 packed;
            packed.x = quantize8(v[i][0], inv);
            packed.y = quantize8(v[i][1], inv);
            packed.z = quantize8(v[i][2], inv);
            packed.w = quantize8(v[i][3], inv);
            if (k_ok && r < rows) {
                __stcs(reinterpret_cast<uint4 *>(q + r * dst.q_pitch + dst.q_col0 + (k >> 1)), packed);
                if (kSwizzled) {
                    sf_tile[(b >> 2) * 512 + (rl & 31) * 16 + (rl >> 5) * 4 + (b & 3)] = static_cast<uint8_t>(sb);
                } else {
                    sf[r * nb + (k >> 5)] = static_cast<uint8_t>(sb);
                }
            }
        }
    }
    if (kSwizzled) {
        __syncthreads();
        const int64_t chunks_k = (nb + 3) >> 2;
        if (threadIdx.x < 128) {
            const int cidx = threadIdx.x >> 5;
            const int64_t kc = tile_k * 4 + cidx;
            if (kc < chunks_k) {
                uint8_t *out = sf + (tile_row * dst.sf_chunks_k + dst.sf_chunk0 + kc) * 512 + (threadIdx.x & 31) * 16;
                *reinterpret_cast<uint4 *>(out) = reinterpret_cast<const uint4 *>(sf_tile)[threadIdx.x];
            }
        }
    }
}

// max |x| over the tensor as the bit pattern of the FP32 value (BF16 magnitude << 16).
// A block reads one contiguous 32 KB piece (eight 16-byte loads in flight per thread) and the grid walks
// the tensor front to back with ordinary loads, so what the L2 holds afterwards is the tensor's tail --
// where the quantizer that follows in the fused entry starts.  Short blocks also balance the tail of the
// reduction better than one wave of long grid-stride loops (5.5 against 5.0 TB/s on a 226 MB tensor).
__global__ void __launch_bounds__(256)
amax_kernel(const uint16_t *__restrict__ x, int64_t rows, int64_t vecs_per_row, int64_t ld,
            uint32_t *__restrict__ out_bits) {
    grid_launch_dependents();
    uint32_t m = 0;
    const int64_t total = rows * vecs_per_row;
    const int64_t base = static_cast<int64_t>(blockIdx.x) * (256 * 8) + threadIdx.x;
    if (ld == vecs_per_row * 8) {
        const uint4 *p = reinterpret_cast<const uint4 *>(x);
        if (base + 7 * 256 < total) {
            uint4 v[8];
#pragma unroll
            for (int u = 0; u < 8; ++u) v[u] = __ldg(p + base + u * 256);
#pragma unroll
            for (int u = 0; u < 8; u += 2) m = max(m, abs_max_bits(v[u], v[u + 1]));
        } else {
            for (int64_t i = base; i < total; i += 256) m = max(m, abs_max_bits(__ldg(p + i)));
        }
    } else {
        const int64_t end = min(total, (static_cast<int64_t>(blockIdx.x) + 1) * (256 * 8));
        for (int64_t i = base; i < end; i += 256) {
            const int64_t r = i / vecs_per_row, vcol = i - r * vecs_per_row;
            m = max(m, abs_max_bits(__ldg(reinterpret_cast<const uint4 *>(x + r * ld + vcol * 8))));
        }
    }
    m = __reduce_max_sync(0xFFFFFFFFu, m);
    __shared__ uint32_t warp_max[8];
    if ((threadIdx.x & 31) == 0) warp_max[threadIdx.x >> 5] = m;
    __syncthreads();
    if (threadIdx.x < 32) {
        m = threadIdx.x < 8 ? warp_max[threadIdx.x] : 0;
        m = __reduce_max_sync(0xFFFFFFFFu, m);
        if (threadIdx.x == 0 && m) atomicMax(out_bits, m << 16);
    }
}

// In place: amax bits -> T = amax / (6 * 448), or 1 for an all-zero tensor.
__global__ void tensor_scale_kernel(float *t) {
    *t = tensor_scale_from_amax(*t);
}

}  // namespace

namespace {

sol_status_t launch_amax_bits(const void *x, int64_t rows, int64_t K, int64_t ld, uint32_t *bits_out,
                              cudaStream_t stream, const DeviceInfo *dev) {
    if (cudaMemsetAsync(bits_out, 0, sizeof(uint32_t), stream) != cudaSuccess) return SOL_ERR_CUDA;
    const int64_t vecs = rows * (K / 8);
    const int64_t blocks = ceil_div(vecs, 256 * 8);  // at most 2^31 - 1: checked with the shape
    amax_kernel<<<static_cast<unsigned>(blocks), 256, 0, stream>>>(
        static_cast<const uint16_t *>(x), rows, K / 8, ld, bits_out);
    return launch_status();
}

// The quantizer is launched as a programmatic dependent of whatever kernel precedes it in the
// stream: its blocks may become resident while that kernel drains, and wait in hardware before
// their first global access.
sol_status_t launch_quantize_ex(const void *x, int64_t rows, int64_t K, int64_t ld, const float *tscale,
                                const float *amax, float *tscale_out, void *q, void *sf,
                                sol_sf_layout_t layout, cudaStream_t stream, const QuantDest *dest = nullptr,
                                bool reverse = false) {
    const QuantDest dst = dest != nullptr ? *dest : QuantDest{K >> 1, 0, ((K >> 4) + 3) >> 2, 0, nullptr};
    const uint32_t k_tiles = static_cast<uint32_t>(ceil_div(K, kTileK));
    int rev = reverse ? 1 : 0;
#ifdef SOL_TUNING
    if (const char *e = getenv("SOL_QREV")) rev = atoi(e);
#endif
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(static_cast<unsigned>(k_tiles * ceil_div(rows, kTileRows)));
    cfg.blockDim = dim3(kQuantThreads);
    cfg.dynamicSmemBytes = 0;
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    auto kern = layout == SOL_SF_SWIZZLED_128x4 ? quantize_kernel<true> : quantize_kernel<false>;
    if (cudaLaunchKernelEx(&cfg, kern, static_cast<const uint16_t *>(x), rows, K, ld, tscale, amax, tscale_out,
                           static_cast<uint8_t *>(q), static_cast<uint8_t *>(sf), dst, k_tiles, rev) != cudaSuccess) {
        cudaGetLastError();
        return SOL_ERR_CUDA;
    }
    return launch_status();
}

}  // namespace

sol_status_t launch_quantize_into(const void *x, int64_t rows, int64_t K, int64_t ld, const float *tscale, void *q,
                                  void *sf, int64_t dest_K, int64_t dest_col0, cudaStream_t stream) {
    const QuantDest dst = {dest_K >> 1, dest_col0 >> 1, dest_K >> 6, dest_col0 >> 6, nullptr};
    return launch_quantize_ex(x, rows, K, ld, tscale, nullptr, nullptr, q, sf, SOL_SF_SWIZZLED_128x4, stream, &dst);
}

sol_status_t launch_quantize_tracking(const void *x, int64_t rows, int64_t K, int64_t ld, const float *tscale, void *q,
                                      void *sf, uint32_t *amax_track, cudaStream_t stream) {
    const QuantDest dst = {K >> 1, 0, ((K >> 4) + 3) >> 2, 0, amax_track};
    return launch_quantize_ex(x, rows, K, ld, tscale, nullptr, nullptr, q, sf, SOL_SF_SWIZZLED_128x4, stream, &dst);
}

namespace {
// state[0] = T derived from the amax collected in state[1]; state[1] = 0 for the next window
__global__ void roll_scale_kernel(float *state) {
    state[0] = tensor_scale_from_amax(state[1]);
    state[1] = 0.0f;
}
}  // namespace

sol_status_t launch_roll_scale(float *state, cudaStream_t stream) {
    roll_scale_kernel<<<1, 1, 0, stream>>>(state);
    return launch_status();
}

sol_status_t launch_amax(const void *x, int64_t rows, int64_t K, int64_t ld, float *tscale_out,
                         cudaStream_t stream, const DeviceInfo *dev) {
    sol_status_t st = launch_amax_bits(x, rows, K, ld, reinterpret_cast<uint32_t *>(tscale_out), stream, dev);
    if (st != SOL_OK) return st;
    tensor_scale_kernel<<<1, 1, 0, stream>>>(tscale_out);
    return launch_status();
}

sol_status_t launch_quantize(const void *x, int64_t rows, int64_t K, int64_t ld, const float *tscale,
                             void *q, void *sf, sol_sf_layout_t layout, cudaStream_t stream) {
    return launch_quantize_ex(x, rows, K, ld, tscale, nullptr, nullptr, q, sf, layout, stream);
}

namespace {
sol_status_t launch_mxfp4_quantize_ex(const void *x, int64_t rows, int64_t K, int64_t ld, void *q, void *sf,
                                      sol_sf_layout_t layout, cudaStream_t stream, const QuantDest &dst);
}

sol_status_t launch_mxfp4_quantize(const void *x, int64_t rows, int64_t K, int64_t ld, void *q, void *sf,
                                   sol_sf_layout_t layout, cudaStream_t stream) {
    return launch_mxfp4_quantize_ex(x, rows, K, ld, q, sf, layout, stream,
                                    QuantDest{K >> 1, 0, ((K >> 5) + 3) >> 2, 0, nullptr});
}

sol_status_t launch_mxfp4_quantize_into(const void *x, int64_t rows, int64_t K, int64_t ld, void *q, void *sf,
                                        int64_t dest_K, int64_t dest_col0, cudaStream_t stream) {
    return launch_mxfp4_quantize_ex(x, rows, K, ld, q, sf, SOL_SF_SWIZZLED_128x4, stream,
                                    QuantDest{dest_K >> 1, dest_col0 >> 1, dest_K >> 7, dest_col0 >> 7, nullptr});
}

namespace {
sol_status_t launch_mxfp4_quantize_ex(const void *x, int64_t rows, int64_t K, int64_t ld, void *q, void *sf,
                                      sol_sf_layout_t layout, cudaStream_t stream, const QuantDest &dst) {
    cudaLaunchConfig_t cfg = {};
    const uint32_t k_tiles = static_cast<uint32_t>(ceil_div(K, kMxTileK));
    cfg.gridDim = dim3(static_cast<unsigned>(k_tiles * ceil_div(rows, kTileRows)));
    cfg.blockDim = dim3(kQuantThreads);
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    auto kern = layout == SOL_SF_SWIZZLED_128x4 ? mxfp4_quantize_kernel<true> : mxfp4_quantize_kernel<false>;
    if (cudaLaunchKernelEx(&cfg, kern, static_cast<const uint16_t *>(x), rows, K, ld, static_cast<uint8_t *>(q),
                           static_cast<uint8_t *>(sf), k_tiles, dst) != cudaSuccess) {
        cudaGetLastError();
        return SOL_ERR_CUDA;
    }
    return launch_status();
}
}  // namespace

sol_status_t launch_quantize_from_amax(const void *x, int64_t rows, int64_t K, int64_t ld, float *scale_words,
                                       void *q, void *sf, sol_sf_layout_t layout, cudaStream_t stream, bool reverse) {
    return launch_quantize_ex(x, rows, K, ld, nullptr, scale_words + 1, scale_words, q, sf, layout, stream, nullptr,
                              reverse);
}

sol_status_t launch_quantize_group(const QuantGroup &g, int count, int64_t rows, int64_t K, sol_sf_layout_t layout,
                                   cudaStream_t stream) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(static_cast<unsigned>(ceil_div(K, kTileK)), static_cast<unsigned>(ceil_div(rows, kTileRows)),
                       static_cast<unsigned>(count));
    cfg.blockDim = dim3(kQuantThreads);
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    auto kern = layout == SOL_SF_SWIZZLED_128x4 ? quantize_group_kernel<true> : quantize_group_kernel<false>;
    if (cudaLaunchKernelEx(&cfg, kern, g, rows, K) != cudaSuccess) {
        cudaGetLastError();
        return SOL_ERR_CUDA;
    }
    return launch_status();
}

sol_status_t launch_amax_quantize(const void *x, int64_t rows, int64_t K, int64_t ld, float *scale_words,
                                  void *q, void *sf, sol_sf_layout_t layout, cudaStream_t stream,
                                  const DeviceInfo *dev) {
    sol_status_t st = launch_amax_bits(x, rows, K, ld, reinterpret_cast<uint32_t *>(scale_words + 1), stream, dev);
    if (st != SOL_OK) return st;
    // the amax pass has just read x front to back: start the quantizer where the L2 is still warm
    return launch_quantize_from_amax(x, rows, K, ld, scale_words, q, sf, layout, stream, true);
}

}  // namespace sol
