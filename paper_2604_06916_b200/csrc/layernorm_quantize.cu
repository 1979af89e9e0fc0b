// Adaptive layer norm fused with the NVFP4 activation quantizer, for sm_100a.
//
// Most quantized activations of a DiT block are produced by a layer norm (no learned affine)
// followed by a per-sample modulation, y = LN(x) (1 + scale[s]) + shift[s]; the linear that follows
// wants Q(y) (paper Section 2's Q with a caller-supplied tensor scale, Section 3.4's NVFP4 rollout).
// Unfused that is a norm pass (2 B read + 2 B written per element), an amax pass (2 B) and the
// quantizer (2.56 B); this kernel reads x once and writes 0.56 B per element.
//
// One warp owns one row at a time: its K values stay in registers between the mean, the centred
// variance and the normalise / modulate / quantize sweep, and there is no block-level
// synchronisation in the row loop.  Rows reach the warp through one row-sized slot in shared memory
// filled by a bulk asynchronous copy (cp.async.bulk + mbarrier): as soon as the row is in registers the
// warp requests the next one, which lands while this one is computed (a row takes several times the
// HBM latency), so the latency is not paid by a warp that holds 120 registers per thread, and a warp
// costs 6 KB of shared memory at K = 3072: sixteen warps fit an SM beside the modulation tables.  A lane owns whole 16-element
// scale blocks (blocks lane, lane + 32, ...), so K <= 4096.  A thread block works on rows of ONE
// sample and keeps that sample's modulation in shared memory as FP32 pairs (1 + scale, shift).  The
// block scale and the sixteen codes follow the quantizer's FP32 sequence on h = bf16(y); max|h| is
// collected for the next call's tensor scale.
#include "ptx.cuh"
#include "quant_math.cuh"
#include "sol_internal.h"

namespace sol {
namespace {

constexpr int kLnMaxWarps = 16;          // upper bound of warps per block (the launcher uses 4)
constexpr int kLnMaxBlocksPerLane = 8;   // 8 x 32 lanes x 16 elements = 4096

// One row (bytes, a multiple of 16, 16-byte aligned on both sides) global -> shared, completing on `bar`.
__device__ __forceinline__ void bulk_load_row(uint32_t dst, const void *src, uint32_t bytes, uint32_t bar) {
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                 ::"r"(dst), "l"(reinterpret_cast<uint64_t>(src)), "r"(bytes), "r"(bar)
                 : "memory");
}


// two FP32 -> packed BF16 (first argument in the low half), round to nearest even
__device__ __forceinline__ uint32_t pack_bf16x2(float lo, float hi) {
    uint32_t d;
    asm("cvt.rn.bf16x2.f32 %0, %1, %2;" : "=r"(d) : "f"(hi), "f"(lo));
    return d;
}

// grid = (blocks per sample, samples); block (j, s) takes rows s*rows_per_sample + j*kLnWarps + warp,
// striding by gridDim.x * kLnWarps inside the sample.
template <int kBlocksPerLane>
__global__ void __launch_bounds__(kLnMaxWarps * 32)
layernorm_quantize_kernel(const uint16_t *__restrict__ x, int64_t rows, int K, int64_t ld,
                          const uint16_t *__restrict__ scale, const uint16_t *__restrict__ shift,
                          int64_t rows_per_sample, float eps, const float *__restrict__ tscale,
                          uint8_t *__restrict__ q, uint8_t *__restrict__ sf, uint32_t *amax_track,
                          uint32_t *status) {
    // (1 + scale) x 2, shift x 2 of this block's sample for element pairs, laid out [pair within block][block] so
    // that the 32 lanes of a warp (consecutive blocks) read consecutive 16-byte words; behind it one row
    // slot of K BF16 per warp
    extern __shared__ __align__(16) float4 mod[];
    __shared__ __align__(8) uint64_t ring_bar[kLnMaxWarps];
    __shared__ float rcp_tab[128];
    __shared__ uint32_t warp_seen[kLnMaxWarps];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int kLnWarps = blockDim.x >> 5, kLnThreads = blockDim.x;
    const int64_t sample = blockIdx.y;
    const float T = *tscale;
    const float c6T = __fmul_rn(6.0f, T);
    for (uint32_t code = threadIdx.x; code < 128; code += kLnThreads)
        rcp_tab[code] = code ? __frcp_rn(__fmul_rn(qmath::e4m3_to_f32(code), T)) : 0.0f;
    const int nblocks = K >> 4;                 // scale blocks per row
    for (int k2 = threadIdx.x; k2 < (K >> 1); k2 += kLnThreads) {
        const uint32_t sc = __ldg(reinterpret_cast<const uint32_t *>(scale + sample * K) + k2);
        const uint32_t sh = __ldg(reinterpret_cast<const uint32_t *>(shift + sample * K) + k2);
        mod[(k2 & 7) * nblocks + (k2 >> 3)] =
            make_float4(1.0f + qmath::bf16_lo(sc), 1.0f + qmath::bf16_hi(sc), qmath::bf16_lo(sh), qmath::bf16_hi(sh));
    }
    __syncthreads();

    const int64_t chunks_k = nblocks >> 2;      // K is a multiple of 64: whole chunks only
    const int64_t first = sample * rows_per_sample;
    const int64_t last = min(rows, first + rows_per_sample);
    const float inv_k = 1.0f / static_cast<float>(K);
    uint32_t seen = 0;
    const uint32_t row_bytes = static_cast<uint32_t>(K) * 2u;
    const uint32_t ring = ptx::smem_u32(mod) + static_cast<uint32_t>(K) * 8u + warp * row_bytes;
    const uint32_t bar0 = ptx::smem_u32(&ring_bar[warp]);
    const int64_t stride = static_cast<int64_t>(gridDim.x) * kLnWarps;
    const int64_t r_first = first + static_cast<int64_t>(blockIdx.x) * kLnWarps + warp;
    if (lane == 0) {
        ptx::mbar_init(bar0, 1);
        ptx::fence_mbar_init();
    }
    __syncwarp();
    if (lane == 0 && r_first < last) {   // the warp's first row
        ptx::mbar_arrive_expect_tx(bar0, row_bytes);
        bulk_load_row(ring, x + r_first * ld, row_bytes, bar0);
    }
    uint32_t parity = 0;
    for (int64_t r = r_first; r < last; r += stride, parity ^= 1u) {
        // bounded, and every decision taken by a warp-wide vote: a copy that never lands ends the loop for the
        // whole warp (no other copy of this warp is in flight then)
        if (!__all_sync(0xFFFFFFFFu, ptx::mbar_try_wait(bar0, parity))) {
            const long long t0 = clock64();
            const long long limit = *reinterpret_cast<const volatile long long *>(status + 2);
            bool ok = true;
            while (!__all_sync(0xFFFFFFFFu, ptx::mbar_try_wait(bar0, parity))) {
                if (__any_sync(0xFFFFFFFFu, clock64() - t0 > limit)) {
                    ok = false;
                    break;
                }
            }
            if (!ok) {
                if (lane == 0) atomicExch(status, 0xA00u);
                break;
            }
        }
        // ---- the row from the ring into registers; block i of this lane = elements [(lane + 32 i) * 16, +16)
        uint32_t w[kBlocksPerLane][8];
        float s1 = 0.0f;
#pragma unroll
        for (int i = 0; i < kBlocksPerLane; ++i) {
            const int b = lane + 32 * i;
            uint4 v0 = make_uint4(0, 0, 0, 0), v1 = v0;
            if (b < nblocks) {
                const uint32_t src = ring + b * 32;
                asm volatile("ld.shared.v4.b32 {%0, %1, %2, %3}, [%4];" : "=r"(v0.x), "=r"(v0.y), "=r"(v0.z), "=r"(v0.w) : "r"(src));
                asm volatile("ld.shared.v4.b32 {%0, %1, %2, %3}, [%4];" : "=r"(v1.x), "=r"(v1.y), "=r"(v1.z), "=r"(v1.w) : "r"(src + 16));
            }
            w[i][0] = v0.x; w[i][1] = v0.y; w[i][2] = v0.z; w[i][3] = v0.w;
            w[i][4] = v1.x; w[i][5] = v1.y; w[i][6] = v1.z; w[i][7] = v1.w;
        }
        // every lane orders its reads of the slot before the bulk copy that refills it (the copy writes
        // through the async proxy, which an mbarrier or a warp barrier alone does not order behind generic reads)
        ptx::fence_proxy_async_smem();
        __syncwarp();
        if (lane == 0 && r + stride < last) {   // the slot is free again: fetch the next row
            ptx::mbar_arrive_expect_tx(bar0, row_bytes);
            bulk_load_row(ring, x + (r + stride) * ld, row_bytes, bar0);
        }
        // mean and variance in one sweep over data shifted by a pivot taken from the row (its first element):
        // sum (x - p) and sum (x - p)^2 lose no accuracy to cancellation as long as p lies within the data,
        // and the two warp reductions run side by side instead of one after the other
        const float pivot = __shfl_sync(0xFFFFFFFFu, qmath::bf16_lo(w[0][0]), 0);
        const uint64_t npivot2 = qmath::f32x2(-pivot, -pivot);
        // four independent accumulator pairs per sum: a single one is a chain of 48 dependent additions per lane
        uint64_t s1_2[4] = {0, 0, 0, 0}, s2_2[4] = {0, 0, 0, 0};   // lanes of 0.0f
#pragma unroll
        for (int i = 0; i < kBlocksPerLane; ++i) {
            if (lane + 32 * i < nblocks) {
#pragma unroll
                for (int e = 0; e < 8; ++e) {
                    const uint64_t d2 = qmath::add2(qmath::f32x2_of_bf16x2(w[i][e]), npivot2);
                    s1_2[e & 3] = qmath::add2(s1_2[e & 3], d2);
                    s2_2[e & 3] = qmath::fma2(d2, d2, s2_2[e & 3]);
                }
            }
        }
        float s2, s1b, s2b;
        qmath::f32x2_split(qmath::add2(qmath::add2(s1_2[0], s1_2[1]), qmath::add2(s1_2[2], s1_2[3])), s1, s1b);
        qmath::f32x2_split(qmath::add2(qmath::add2(s2_2[0], s2_2[1]), qmath::add2(s2_2[2], s2_2[3])), s2, s2b);
        s1 += s1b;
        s2 += s2b;
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) {
            s1 += __shfl_xor_sync(0xFFFFFFFFu, s1, o);
            s2 += __shfl_xor_sync(0xFFFFFFFFu, s2, o);
        }
        const float dm = s1 * inv_k;                       // mean - pivot
        const float mu = pivot + dm;
        const float var = fmaxf(fmaf(-dm, dm, s2 * inv_k), 0.0f);
        const float rstd = 1.0f / sqrtf(var + eps);
        const float nmr = -mu * rstd;   // xhat = fma(x, rstd, -mu * rstd)
        const uint64_t rstd2 = qmath::f32x2(rstd, rstd), nmr2 = qmath::f32x2(nmr, nmr);
        const int64_t row_tile = r >> 7;
        const int rr = static_cast<int>(r & 127);
        uint8_t *sf_row = sf + row_tile * chunks_k * 512 + (rr & 31) * 16 + (rr >> 5) * 4;
        // ---- normalise, modulate, round to BF16 (h takes the row's registers), then the block scales of all
        // the lane's blocks side by side (a division and a table look-up each), then the codes
        uint32_t bmax[kBlocksPerLane];
#pragma unroll
        for (int i = 0; i < kBlocksPerLane; ++i) {
            const int b = lane + 32 * i;
            uint32_t bm0 = 0, bm1 = 0;
            if (b < nblocks) {
                const float4 *mp = mod + b;
#pragma unroll
                for (int e = 0; e < 8; ++e) {
                    const float4 m = mp[e * nblocks];   // (1 + scale) and shift of two neighbouring elements
                    const uint64_t xh2 = qmath::fma2(qmath::f32x2_of_bf16x2(w[i][e]), rstd2, nmr2);
                    float y0, y1;
                    qmath::f32x2_split(qmath::fma2(xh2, qmath::f32x2(m.x, m.y), qmath::f32x2(m.z, m.w)), y0, y1);
                    w[i][e] = pack_bf16x2(y0, y1);
                    if (e & 1) bm1 = qmath::absmax2(bm1, w[i][e]);
                    else bm0 = qmath::absmax2(bm0, w[i][e]);
                }
            }
            const uint32_t bm = qmath::absmax2(bm0, bm1) & 0x7FFF7FFFu;
            bmax[i] = max(bm & 0xFFFFu, bm >> 16);
        }
        uint32_t sbv[kBlocksPerLane];
        float rcpv[kBlocksPerLane];
#pragma unroll
        for (int i = 0; i < kBlocksPerLane; ++i) {
            seen = max(seen, bmax[i]);
            sbv[i] = qmath::f32_to_e4m3_sat(__fdiv_rn(__uint_as_float(bmax[i] << 16), c6T));
            rcpv[i] = rcp_tab[sbv[i]];
        }
#pragma unroll
        for (int i = 0; i < kBlocksPerLane; ++i) {
            const int b = lane + 32 * i;
            if (b < nblocks) {
                const uint64_t rcp2 = qmath::f32x2(rcpv[i], rcpv[i]);
                uint2 packed;
                packed.x = qmath::quantize8_x2(w[i][0], w[i][1], w[i][2], w[i][3], rcp2);
                packed.y = qmath::quantize8_x2(w[i][4], w[i][5], w[i][6], w[i][7], rcp2);
                __stcs(reinterpret_cast<uint2 *>(q + r * (K >> 1) + b * 8), packed);
                // the lane's scale byte of its (row, chunk) slot (four neighbouring lanes fill one 4-byte slot)
                sf_row[(b >> 2) * 512 + (b & 3)] = static_cast<uint8_t>(sbv[i]);
            }
        }
    }
    // rows past M inside the last 128-row scale chunk are padding and read as 0 (first block only)
    if (blockIdx.x == 0 && blockIdx.y == 0) {
        const int64_t padded_rows = (rows + 127) / 128 * 128;
        for (int64_t r = rows + warp; r < padded_rows; r += kLnWarps) {
            const int rr = static_cast<int>(r & 127);
            uint8_t *sf_row = sf + (r >> 7) * chunks_k * 512 + (rr & 31) * 16 + (rr >> 5) * 4;
            for (int64_t c = lane; c < chunks_k; c += 32) *reinterpret_cast<uint32_t *>(sf_row + c * 512) = 0u;
        }
    }
    if (amax_track != nullptr) {
        seen = __reduce_max_sync(0xFFFFFFFFu, seen);
        if (lane == 0) warp_seen[warp] = seen;
        __syncthreads();
        if (threadIdx.x < 32) {
            uint32_t m = threadIdx.x < kLnWarps ? warp_seen[threadIdx.x] : 0;
            m = __reduce_max_sync(0xFFFFFFFFu, m);
            if (threadIdx.x == 0 && m) atomicMax(amax_track, m << 16);
        }
    }
}

}  // namespace

int layernorm_max_k() { return kLnMaxBlocksPerLane * 32 * 16; }

sol_status_t launch_layernorm_quantize(const void *x, int64_t rows, int64_t K, int64_t ld, const void *scale,
                                       const void *shift, int64_t rows_per_sample, float eps, const float *tscale,
                                       void *q, void *sf, uint32_t *amax_track, cudaStream_t stream) {
    const int64_t samples = ceil_div(rows, rows_per_sample);
    if (samples > 65535) return SOL_ERR_BAD_SHAPE;
    const DeviceInfo *dev = current_device_info();
    const int sms = dev != nullptr && dev->ok ? dev->sm_count : 148;
    // modulation table (8 bytes per element) + per warp one row slot of 2 bytes per element: four warps per
    // block, four blocks per SM at K = 3072 (registers allow no more)
    const int kLnWarps = 4;
    const int kLnThreads = kLnWarps * 32;
    const size_t smem = static_cast<size_t>(K) * 8 + static_cast<size_t>(kLnWarps) * K * 2;
    const int per_lane = static_cast<int>(ceil_div(K / 16, 32));
    auto launch = [&](auto kern) {
        // one wave of resident blocks, split evenly over the samples, never more blocks per sample
        // than it has groups of rows
        // (the static tables count against the 48 KB default too)
        if (smem + 1024 > 48 * 1024) cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, 208 * 1024);
        int per_sm = 0;
        if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, kern, kLnThreads, smem) != cudaSuccess || per_sm < 1)
            per_sm = 1;
        int64_t per_sample = (static_cast<int64_t>(sms) * per_sm) / samples;
        const int64_t row_groups = ceil_div(rows_per_sample < rows ? rows_per_sample : rows, kLnWarps);
        if (per_sample > row_groups) per_sample = row_groups;
        if (per_sample < 1) per_sample = 1;
        const dim3 grid(static_cast<unsigned>(per_sample), static_cast<unsigned>(samples));
        kern<<<grid, kLnThreads, smem, stream>>>(static_cast<const uint16_t *>(x), rows, static_cast<int>(K), ld,
                                                 static_cast<const uint16_t *>(scale), static_cast<const uint16_t *>(shift),
                                                 rows_per_sample, eps, tscale, static_cast<uint8_t *>(q),
                                                 static_cast<uint8_t *>(sf), amax_track, device_status_word());
    };
    if (per_lane <= 2) launch(layernorm_quantize_kernel<2>);
    else if (per_lane <= 4) launch(layernorm_quantize_kernel<4>);
    else if (per_lane <= 6) launch(layernorm_quantize_kernel<6>);
    else launch(layernorm_quantize_kernel<8>);
    return launch_status();
}

}  // namespace sol
