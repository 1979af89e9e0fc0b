// Weight refresh, first half: merge rank-r adapters into the base weights and take the merged
// tensor's amax, for sm_100a.
//
//     W'[n][k] = bf16_rne( fma(s, sum_j B[n][j] * A[j][k], W[n][k]) )
//
// (paper Section 3.4 / Appendix B.2: the updated policy is re-quantized into the NVFP4 engine
// after every step; Section 4.1: adapters of rank 32, alpha 64).  W' decides quantized codes, so
// the sum is the fixed binary32 chain acc = fma(B[n][j], A[j][k], acc), j ascending from acc = 0,
// which rules the tensor cores out (their accumulation order is not this one).  With r = 32 that
// is 32 FMAs per 4 bytes moved: the kernel is bound by FP32 issue (128 FMA per clock per SM),
// not by HBM.  Each thread owns an 8 x 8 register tile, so one step of the chain costs six
// 16-byte shared-memory loads per 64 FMAs.  (The packed two-lane FMA was measured slower here:
// it issues on one of the two FP32 pipes only.)  W' goes to a BF16 buffer that the weight
// quantizer reads next (from L2 for layer-sized matrices); max|W'| is accumulated into the word
// the quantizer's tensor scale is derived from.
#include "sol_internal.h"

namespace sol {
namespace {

constexpr int kThreads = 128;
constexpr int kTileN = 64;    // rows of W per block: 8 thread rows x 8
constexpr int kTileK = 128;   // columns of W per block: 16 thread columns x (4 + 4)
constexpr int kBlocksPerSm = 4;  // small blocks in different phases (fill, FMA chain, store) overlap
constexpr int kMaxRank = 64;
constexpr int kBStride = kTileN + 4;  // floats per rank row of the B tile (16-byte aligned rows)
constexpr size_t kSmemPerRank = (kTileK + kBStride) * sizeof(float);

__device__ __forceinline__ float bf16_lo(uint32_t w) { return __uint_as_float(w << 16); }
__device__ __forceinline__ float bf16_hi(uint32_t w) { return __uint_as_float(w & 0xFFFF0000u); }

// two FP32 -> packed BF16 (first argument in the low half), round to nearest even
__device__ __forceinline__ uint32_t pack_bf16x2(float lo, float hi) {
    uint32_t d;
    asm("cvt.rn.bf16x2.f32 %0, %1, %2;" : "=r"(d) : "f"(hi), "f"(lo));
    return d;
}

// max(|a|, |b|) per BF16 half (sign bits of the result are garbage and masked off at the end)
__device__ __forceinline__ uint32_t absmax2(uint32_t a, uint32_t b) {
    uint32_t d;
    asm("max.xorsign.abs.bf16x2 %0, %1, %2;" : "=r"(d) : "r"(a), "r"(b));
    return d;
}

// Shared memory: A tile as FP32 [r][128]; B tile as FP32, transposed to [r][kBStride].
// kFull: the block's 64 x 128 tile lies inside the matrix (no bounds checks).
template <bool kFull>
__global__ void __launch_bounds__(kThreads, kBlocksPerSm)
lora_merge_kernel(const __grid_constant__ MergeGroup grp, int64_t ldw, int64_t lda, int64_t ldb, int64_t N,
                  int64_t K, int r, float s, int full_x, int b_vec) {
    const uint16_t *__restrict__ w = grp.w[blockIdx.z];
    const uint16_t *__restrict__ a = grp.a[blockIdx.z];
    const uint16_t *__restrict__ b = grp.b[blockIdx.z];
    uint16_t *__restrict__ out = grp.out[blockIdx.z];
    uint32_t *amax_bits = reinterpret_cast<uint32_t *>(grp.scale_words[blockIdx.z] + 1);
    extern __shared__ __align__(16) uint8_t smem[];
    float *As = reinterpret_cast<float *>(smem);   // [r][kTileK]
    float *Bs = As + r * kTileK;                   // [r][kBStride]

    // the launch covers either the interior tiles (kFull) or the ragged right and bottom edges
    int bx = blockIdx.x, by = blockIdx.y;
    if (!kFull) {
        // edge blocks: first the right column of tiles (all tile rows), then the rest of the bottom row
        const int tiles_x = static_cast<int>((K + kTileK - 1) / kTileK), tiles_y = static_cast<int>((N + kTileN - 1) / kTileN);
        int e = blockIdx.x;
        const int right = full_x < tiles_x ? tiles_y : 0;  // a ragged right column exists
        if (e < right) {
            bx = tiles_x - 1;
            by = e;
        } else {
            bx = e - right;
            by = tiles_y - 1;
        }
    }
    const int tx = threadIdx.x & 15, ty = threadIdx.x >> 4;
    const int64_t n0 = static_cast<int64_t>(by) * kTileN;
    const int64_t k0 = static_cast<int64_t>(bx) * kTileK;

    // Base weights of this thread's 8 x 8 tile: rows ty*8 + i, columns tx*4 + {0..3} and
    // 64 + tx*4 + {0..3}.  They are loaded after the FMA chain (its 64 accumulators leave no
    // registers to park them in); a prefetch into L2 now takes the HBM latency off that load.  A
    // half-warp's 8 rows x 2 runs of 128 bytes are 16 lines, one per lane.
    const int64_t c0 = k0 + tx * 4, c1 = c0 + 64;
    const uint16_t *wrow = w + (n0 + ty * 8) * ldw + c0;
    {
        const int prow = tx >> 1, pcol = (tx & 1) * 64;
        if (kFull || (n0 + ty * 8 + prow < N && k0 + pcol < K))
            asm volatile("prefetch.global.L2 [%0];" ::"l"(w + (n0 + ty * 8 + prow) * ldw + k0 + pcol));
    }

    // A tile: r x 128 BF16 -> FP32, four elements (8 bytes) per load
    for (int i = threadIdx.x; i < r * (kTileK / 4); i += kThreads) {
        const int j = i / (kTileK / 4), c = (i % (kTileK / 4)) * 4;
        uint2 v = make_uint2(0, 0);
        if (kFull || k0 + c < K) v = __ldg(reinterpret_cast<const uint2 *>(a + j * lda + k0 + c));
        *reinterpret_cast<float4 *>(As + j * kTileK + c) =
            make_float4(bf16_lo(v.x), bf16_hi(v.x), bf16_lo(v.y), bf16_hi(v.y));
    }
    // B tile: 64 rows x r BF16 -> FP32 [j][row]; consecutive threads take consecutive rows
    if (b_vec) {  // r and the pitch are multiples of 8 and the base is 16-byte aligned: 8 ranks per load
        for (int i = threadIdx.x; i < (r >> 3) * kTileN; i += kThreads) {
            const int row = i % kTileN, j = (i / kTileN) * 8;
            uint4 v = make_uint4(0, 0, 0, 0);
            if (kFull || n0 + row < N) v = __ldg(reinterpret_cast<const uint4 *>(b + (n0 + row) * ldb + j));
            float *dst = Bs + j * kBStride + row;
            dst[0 * kBStride] = bf16_lo(v.x);
            dst[1 * kBStride] = bf16_hi(v.x);
            dst[2 * kBStride] = bf16_lo(v.y);
            dst[3 * kBStride] = bf16_hi(v.y);
            dst[4 * kBStride] = bf16_lo(v.z);
            dst[5 * kBStride] = bf16_hi(v.z);
            dst[6 * kBStride] = bf16_lo(v.w);
            dst[7 * kBStride] = bf16_hi(v.w);
        }
    } else {
        for (int i = threadIdx.x; i < r * kTileN; i += kThreads) {
            const int row = i % kTileN, j = i / kTileN;
            uint32_t v = 0;
            if (kFull || n0 + row < N) v = static_cast<uint32_t>(__ldg(b + (n0 + row) * ldb + j)) << 16;
            Bs[j * kBStride + row] = __uint_as_float(v);
        }
    }
    __syncthreads();

    float acc[8][8];
#pragma unroll
    for (int i = 0; i < 8; ++i)
#pragma unroll
        for (int c = 0; c < 8; ++c) acc[i][c] = 0.0f;

    const float4 *ap = reinterpret_cast<const float4 *>(As) + tx;
    const float4 *bp = reinterpret_cast<const float4 *>(Bs) + ty * 2;
#pragma unroll 4
    for (int j = 0; j < r; ++j) {
        const float4 a0 = ap[j * (kTileK / 4)], a1 = ap[j * (kTileK / 4) + 16];
        const float4 b0 = bp[j * (kBStride / 4)], b1 = bp[j * (kBStride / 4) + 1];
        const float av[8] = {a0.x, a0.y, a0.z, a0.w, a1.x, a1.y, a1.z, a1.w};
        const float bv[8] = {b0.x, b0.y, b0.z, b0.w, b1.x, b1.y, b1.z, b1.w};
#pragma unroll
        for (int i = 0; i < 8; ++i)
#pragma unroll
            for (int c = 0; c < 8; ++c) acc[i][c] = __fmaf_rn(bv[i], av[c], acc[i][c]);
    }

    uint2 wv[8][2];
#pragma unroll
    for (int i = 0; i < 8; ++i) {
        if (kFull) {
            wv[i][0] = __ldcs(reinterpret_cast<const uint2 *>(wrow + i * ldw));
            wv[i][1] = __ldcs(reinterpret_cast<const uint2 *>(wrow + i * ldw + 64));
        } else {
            wv[i][0] = wv[i][1] = make_uint2(0, 0);
            if (n0 + ty * 8 + i < N) {
                if (c0 < K) wv[i][0] = __ldcs(reinterpret_cast<const uint2 *>(wrow + i * ldw));
                if (c1 < K) wv[i][1] = __ldcs(reinterpret_cast<const uint2 *>(wrow + i * ldw + 64));
            }
        }
    }

    uint32_t m2 = 0;
    uint16_t *orow = out + (n0 + ty * 8) * K + c0;
#pragma unroll
    for (int i = 0; i < 8; ++i) {
#pragma unroll
        for (int g = 0; g < 2; ++g) {
            const uint2 wq = wv[i][g];
            uint2 o;
            o.x = pack_bf16x2(__fmaf_rn(s, acc[i][4 * g + 0], bf16_lo(wq.x)), __fmaf_rn(s, acc[i][4 * g + 1], bf16_hi(wq.x)));
            o.y = pack_bf16x2(__fmaf_rn(s, acc[i][4 * g + 2], bf16_lo(wq.y)), __fmaf_rn(s, acc[i][4 * g + 3], bf16_hi(wq.y)));
            if (kFull || (n0 + ty * 8 + i < N && (g ? c1 : c0) < K)) {
                *reinterpret_cast<uint2 *>(orow + i * K + g * 64) = o;
                m2 = absmax2(m2, absmax2(o.x, o.y));
            }
        }
    }
    m2 &= 0x7FFF7FFFu;
    uint32_t m = max(m2 & 0xFFFFu, m2 >> 16);  // BF16 magnitudes order like unsigned integers
    m = __reduce_max_sync(0xFFFFFFFFu, m);
    __shared__ uint32_t warp_max[kThreads / 32];
    if ((threadIdx.x & 31) == 0) warp_max[threadIdx.x >> 5] = m;
    __syncthreads();
    if (threadIdx.x < 32) {
        m = threadIdx.x < kThreads / 32 ? warp_max[threadIdx.x] : 0;
        m = __reduce_max_sync(0xFFFFFFFFu, m);
        if (threadIdx.x == 0 && m) atomicMax(amax_bits, m << 16);
    }
}

__global__ void zero_amax_kernel(const __grid_constant__ MergeGroup grp, int count) {
    if (threadIdx.x < count) grp.scale_words[threadIdx.x][1] = 0.0f;
}

}  // namespace

int lora_max_rank() { return kMaxRank; }

sol_status_t launch_lora_merge(const MergeGroup &g, int count, int64_t ldw, int64_t lda, int64_t ldb, int64_t N,
                               int64_t K, int64_t r, float s, cudaStream_t stream) {
    static bool attr_set[64] = {};
    const size_t smem = static_cast<size_t>(r) * kSmemPerRank;
    int device = 0;
    if (cudaGetDevice(&device) != cudaSuccess) return SOL_ERR_CUDA;
    if (device >= 0 && device < 64 && !attr_set[device]) {
        if (cudaFuncSetAttribute(lora_merge_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                 kMaxRank * kSmemPerRank) != cudaSuccess ||
            cudaFuncSetAttribute(lora_merge_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                 kMaxRank * kSmemPerRank) != cudaSuccess)
            return SOL_ERR_CUDA;
        attr_set[device] = true;
    }
    zero_amax_kernel<<<1, 32, 0, stream>>>(g, count);
    const int tiles_x = static_cast<int>(ceil_div(K, kTileK)), tiles_y = static_cast<int>(ceil_div(N, kTileN));
    const int full_x = static_cast<int>(K / kTileK), full_y = static_cast<int>(N / kTileN);
    int b_vec = (r % 8 == 0 && ldb % 8 == 0) ? 1 : 0;
    for (int i = 0; i < count; ++i)
        if (!aligned16(g.b[i])) b_vec = 0;
    if (full_x > 0 && full_y > 0) {
        lora_merge_kernel<true><<<dim3(full_x, full_y, count), kThreads, smem, stream>>>(
            g, ldw, lda, ldb, N, K, static_cast<int>(r), s, full_x, b_vec);
    }
    // ragged edges: the right column of tiles (if K is not a multiple of 128), then what is left
    // of the bottom row (if N is not a multiple of 64)
    const int right = full_x < tiles_x ? tiles_y : 0;
    const int bottom = full_y < tiles_y ? (full_x < tiles_x ? tiles_x - 1 : tiles_x) : 0;
    if (right + bottom > 0) {
        lora_merge_kernel<false><<<dim3(right + bottom, 1, count), kThreads, smem, stream>>>(
            g, ldw, lda, ldb, N, K, static_cast<int>(r), s, full_x, b_vec);
    }
    return launch_status();
}

}  // namespace sol
