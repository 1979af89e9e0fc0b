// Pieces shared by the single-CTA and the CTA-pair tcgen05 GEMM kernels.
#pragma once
#include "ptx.cuh"
#include "sol_internal.h"

#include <cuda_bf16.h>
#include <cstdlib>

namespace sol {
namespace gemm {

enum class Kind { kBf16, kNvfp4 };

constexpr int kBM = 128;
constexpr int kRowBytes = 128;        // bytes of K per row per stage (one swizzle atom wide)
constexpr int kMmasPerStage = 4;      // 32 bytes of K per MMA
constexpr int kEpiWarps = 4;
constexpr int kEpiBufBytes = 32 * 128;  // 32 rows x 64 BF16
constexpr int kTmemCols = 512;
constexpr int kGroupM = 8;            // tile raster: groups of 8 row tiles sweep all column tiles

// Diagnostic switches, compiled in only with -DSOL_TUNING (never in the product build): they
// drop one part of the pipeline so its share of the time can be read off a timing run.
#ifdef SOL_TUNING
constexpr bool kTuning = true;
#else
constexpr bool kTuning = false;
#endif
enum : uint32_t { kDbgNoSfCopy = 1, kDbgNoMma = 2, kDbgNoEpilogue = 4, kDbgNoSfLoad = 8, kDbgNoStore = 16, kDbgTrace = 64, kDbgNoBLoad = 128 };

#ifdef SOL_TUNING
// timeline of the first pair: [event type][k-tile index] = clock64 of the even CTA's SM (rank 1: types 4,5)
__device__ long long g_trace[12][512];
#define SOL_TRACE(type, idx) do { if (blockIdx.x < 2 && (idx) < 512 && (threadIdx.x & 31) == 0) g_trace[type][idx] = clock64(); } while (0)
#else
#define SOL_TRACE(type, idx) do { } while (0)
#endif

struct Params {
    const uint8_t *sfa;    // scales of A, chunked layout (NVFP4 only)
    const uint8_t *sfb;
    const float *ts_a;     // per-tensor scales (NVFP4 only)
    const float *ts_b;
    const uint16_t *bias;  // BF16 [N] or null
    uint32_t *status;
    uint32_t dbg;
    int M, N, K;
    int m_tiles, n_tiles;
    // quantized-output epilogue (NVFP4 pair kernel only): Y leaves as the next linear's Q(X)
    uint8_t *sf_out;        // scales of the output, chunked layout for an [M, N] tensor
    const float *ts_out;    // tensor scale T of the output (caller supplied)
    uint32_t *amax_out;     // running max |h| as FP32 bits (atomicMax), or null
    int act;                // 0 = identity, 1 = GELU (tanh form) before the output quantizer
    int n_split;            // split mode: columns below it leave as BF16, the rest quantized
    int dest_col0;          // first column of the quantized part inside the destination tensor
    int dest_chunks_k;      // scale chunks per 128-row tile of the destination tensor
};

#ifndef SOL_WAIT_HINT
#define SOL_WAIT_HINT 200000u
#endif
__device__ __forceinline__ bool wait_bounded(uint32_t bar, uint32_t parity, volatile uint32_t *abort_flag,
                                             uint32_t *status, uint32_t code) {
    if (ptx::mbar_try_wait(bar, parity)) return true;
    const long long t0 = clock64();
    // long hardware suspends: a CTA has ~20 warps that mostly wait, and warps that poll in a tight loop
    // take issue slots from the few that have work (the epilogue at a tile boundary, above all)
    while (!ptx::mbar_try_wait_suspend(bar, parity, SOL_WAIT_HINT)) {
        if (*abort_flag) return false;
        // the limit lives in the device status block (words 2..3); it is read on this slow path only
        if (clock64() - t0 > *reinterpret_cast<const volatile long long *>(status + 2)) {
            *abort_flag = 1;
            atomicExch(status, code);
            return false;
        }
    }
    return true;
}

// Test hook (device status block, word 1): the load-issuing warps issue nothing while it is set.
__device__ __forceinline__ bool loads_held(const uint32_t *status) {
    return *reinterpret_cast<const volatile uint32_t *>(status + 1) != 0;
}

__device__ __forceinline__ void tile_coords(int t, int m_tiles, int n_tiles, int &mt, int &nt) {
    const int per_group = kGroupM * n_tiles;
    const int g = t / per_group;
    const int first = g * kGroupM;
    const int gsize = min(kGroupM, m_tiles - first);
    const int r = t - g * per_group;
    mt = first + r % gsize;
    nt = r / gsize;
}


// Drains one accumulator tile (32 TMEM lanes x kBN columns of this warp's quadrant) to Y:
// tcgen05.ld -> y = fma(acc, alpha, bias) -> BF16 -> 128-byte-swizzled staging buffer -> TMA store
// of 32 x 64 boxes (clipped at the matrix edge).  `release()` is called once the last TMEM load has
// completed, so the MMA warp can reuse the accumulator while the tail is converted and stored.
template <int kBN, class Release>
__device__ __forceinline__ void epilogue_tile(const CUtensorMap *tm_y, const Params &p, uint32_t t_acc, int m0, int n0,
                                              float alpha, uint32_t epi_warp, uint32_t &buf, int lane,
                                              Release release) {
#pragma unroll 1
    for (int c = 0; c < kBN / 64; ++c) {
        const uint32_t sbuf = epi_warp + buf * kEpiBufBytes;
        if (lane == 0) ptx::tma_store_wait_read<1>();  // the store issued two chunks ago has left sbuf
        __syncwarp();
#pragma unroll
        for (int h = 0; h < 2; ++h) {
            uint32_t acc[32];
            ptx::tmem_ld_32x32(t_acc + c * 64 + h * 32, acc);
            ptx::tmem_ld_wait();
            if (c == kBN / 64 - 1 && h == 1) {
                ptx::tc_fence_before_sync();
                __syncwarp();
                if (lane == 0) release();
            }
            const int nb = n0 + c * 64 + h * 32;
#pragma unroll
            for (int g = 0; g < 4; ++g) {  // 8 columns -> one 16-byte shared store
                uint4 bb = make_uint4(0, 0, 0, 0);
                if (p.bias != nullptr && nb + g * 8 < p.N)
                    bb = __ldg(reinterpret_cast<const uint4 *>(p.bias + nb + g * 8));
                const uint32_t bw[4] = {bb.x, bb.y, bb.z, bb.w};
                uint32_t o[4];
#pragma unroll
                for (int e = 0; e < 4; ++e) {
                    const float b0 = __uint_as_float(bw[e] << 16);
                    const float b1 = __uint_as_float(bw[e] & 0xFFFF0000u);
                    const float y0 = fmaf(__uint_as_float(acc[g * 8 + 2 * e]), alpha, b0);
                    const float y1 = fmaf(__uint_as_float(acc[g * 8 + 2 * e + 1]), alpha, b1);
                    __nv_bfloat162 pk = __floats2bfloat162_rn(y0, y1);
                    o[e] = *reinterpret_cast<uint32_t *>(&pk);
                }
                const uint32_t chunk16 = static_cast<uint32_t>(h * 4 + g) ^ (lane & 7u);  // 128-byte swizzle
                const uint32_t dst = sbuf + lane * 128 + chunk16 * 16;
                asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(dst), "r"(o[0]), "r"(o[1]), "r"(o[2]),
                             "r"(o[3])
                             : "memory");
            }
        }
        ptx::fence_proxy_async_smem();
        __syncwarp();
        if (lane == 0) {
            if (n0 + c * 64 < p.N && m0 < p.M && !(kTuning && (p.dbg & kDbgNoStore)))
                ptx::tma_store_2d(tm_y, n0 + c * 64, m0, sbuf);
            ptx::tma_store_commit();
        }
        buf ^= 1u;
    }
}

// Launchers of the two kernel families (arguments already validated).
sol_status_t launch_single_bf16(const void *x, const void *w, const void *bias, void *y, int64_t M, int64_t N,
                                int64_t K, int64_t ldx, int64_t ldw, int64_t ldy, cudaStream_t stream,
                                const DeviceInfo *dev);
sol_status_t launch_single_nvfp4(const void *xq, const void *xsf, const float *xts, const void *wq,
                                 const void *wsf, const float *wts, const void *bias, void *y, int64_t M,
                                 int64_t N, int64_t K, int64_t ldy, cudaStream_t stream, const DeviceInfo *dev);
sol_status_t launch_pair_bf16(const void *x, const void *w, const void *bias, void *y, int64_t M, int64_t N,
                              int64_t K, int64_t ldx, int64_t ldw, int64_t ldy, cudaStream_t stream,
                              const DeviceInfo *dev);
sol_status_t launch_pair_nvfp4(const void *xq, const void *xsf, const float *xts, const void *wq,
                               const void *wsf, const float *wts, const void *bias, void *y, int64_t M,
                               int64_t N, int64_t K, int64_t ldy, cudaStream_t stream, const DeviceInfo *dev);
sol_status_t launch_pair256_nvfp4_quant_out(const void *xq, const void *xsf, const float *xts, const void *wq,
                                            const void *wsf, const float *wts, const void *bias, int act,
                                            const float *ts_out, void *hq, void *hsf, uint32_t *amax_out,
                                            int64_t M, int64_t N, int64_t K, cudaStream_t stream,
                                            const DeviceInfo *dev);
sol_status_t launch_pair256_nvfp4_split_out(const void *xq, const void *xsf, const float *xts, const void *wq,
                                            const void *wsf, const float *wts, const void *bias, void *y_bf16,
                                            int64_t ldy, int64_t n_split, int act, const float *ts_out, void *hq,
                                            void *hsf, int64_t dest_K, int64_t dest_col0, uint32_t *amax_out,
                                            int64_t M, int64_t N, int64_t K, cudaStream_t stream,
                                            const DeviceInfo *dev);
sol_status_t launch_pair256_mxfp4(const void *xq, const void *xsf, const void *wq, const void *wsf, const void *bias,
                                  void *y, int64_t M, int64_t N, int64_t K, int64_t ldy, cudaStream_t stream,
                                  const DeviceInfo *dev);
sol_status_t launch_pair256_mxfp4_quant_out(const void *xq, const void *xsf, const void *wq, const void *wsf,
                                            const void *bias, int act, void *hq, void *hsf, uint32_t *amax_out, int64_t M,
                                            int64_t N, int64_t K, cudaStream_t stream, const DeviceInfo *dev);
sol_status_t launch_pair256_mxfp4_split_out(const void *xq, const void *xsf, const void *wq, const void *wsf,
                                            const void *bias, void *y_bf16, int64_t ldy, int64_t n_split, int act,
                                            void *hq, void *hsf, int64_t dest_K, int64_t dest_col0, uint32_t *amax_out,
                                            int64_t M, int64_t N, int64_t K, cudaStream_t stream, const DeviceInfo *dev);
sol_status_t launch_pair256_nvfp4(const void *xq, const void *xsf, const float *xts, const void *wq,
                                  const void *wsf, const float *wts, const void *bias, void *y, int64_t M,
                                  int64_t N, int64_t K, int64_t ldy, cudaStream_t stream, const DeviceInfo *dev);

}  // namespace gemm
}  // namespace sol
