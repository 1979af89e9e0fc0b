// NVFP4 / MXFP4 CTA-pair GEMM with 256 x 256 pair tiles (tcgen05.mma.cta_group::2, kind::mxf4nvf4 / kind::mxf4).
//
// Why this shape: one MMA instruction costs its issuing thread ~50 cycles and a k-tile needs ~250 more
// for the commit, the look at the next stage's barriers and the loop, so the single MMA-issuing thread
// spends ~450-520 cycles per k-tile of four MMAs.  Only at N = 256 does the tensor core need that long
// (4 x 128 cycles); narrower tiles leave it idle.  N = 256 also has the lowest L2 -> SM traffic per flop.
//
// TMEM does not hold two 256-column accumulators plus the scale factors, so the two accumulators
// overlap: A = columns [0,256), B = [96,352), scale-factor buffers 3 x 48 columns at [352,496).
// Tiles alternate between A and B.  The epilogue drains the shared columns [96,256) first and
// signals `ovl_free`; the MMAs of the next tile start then, while the rest of the tile is still
// being converted and stored.  Eight epilogue warps (two per TMEM lane quadrant) shorten that wait.
//
// Warps per CTA: 0 = TMA producer (A, B: five stages of 32 KB); 1 = TMEM owner, MMA issuer in the even
// CTA; 2..9 = epilogue; 10..13 = scale-factor copy warps, one per TMEM lane quadrant, in both CTAs
// (shared memory -> registers -> tcgen05.st); 14 = TMA producer of the scale tiles, which travel in a
// ring of their own (five slots of 6 KB) that runs ahead of the A / B ring.
// No multicast loads; every mbarrier wait is bounded.
#include "gemm_common.cuh"
#include "quant_math.cuh"

namespace sol {
namespace gemm {
namespace {

constexpr int kBN = 256;
constexpr int kStages = 5;
constexpr int kBK = 256;                       // FP4 elements of K per stage = 128 bytes per row
constexpr int kMmaK = 64;
constexpr int kABytes = kBM * kRowBytes;       // 16 KB: this CTA's 128 rows of A
constexpr int kBBytes = (kBN / 2) * kRowBytes; // 16 KB: this CTA's half of the B tile
constexpr int kSfaBytes = 2048;                // 4 k-chunks x 512 bytes
constexpr int kSfbBytes = 4096;                // 2 row chunks x 4 k-chunks x 512 bytes
constexpr int kStageBytes = kABytes + kBBytes;  // 32 KB: one k-tile of A and B
constexpr int kSfSlotBytes = kSfaBytes + kSfbBytes;  // 6 KB: one k-tile of scale tiles
constexpr int kSfSlots = 5;                    // scale-tile ring in shared memory, released as soon as a tile is in registers
constexpr int kSfBufCols = 48;                 // per k-tile: 4 MMAs x (4 columns of A + 8 of B)
#ifdef SOL_SPAN
// Diagnostic build only (-DSOL_SPAN, otherwise identical to the product kernel): SM cycles and nanoseconds
// CTA 0 spent between the dependency wait and the final cluster barrier of the last launch.  Their ratio
// is the SM clock the kernel really ran at, which under the board's power cap is far from the maximum.
__device__ long long g_span[2];
#endif
constexpr int kAccStride = 96;                 // accumulator B starts here; [96,256) is shared
constexpr int kSfBufs = 3;
constexpr int kSfCol = kAccStride + kBN;       // 352
constexpr int kEpiWarpsFp4 = 8;
constexpr int kSfCopyWarps = 4;                // one per TMEM lane quadrant
constexpr int kWarps = 2 + kEpiWarpsFp4 + kSfCopyWarps + 1;
constexpr int kThreadsFp4 = 32 * (kWarps + (kTuning ? 1 : 0));  // 480 (+ a probe warp in the diagnostic build)
constexpr int kEpiBytes = kEpiWarpsFp4 * kEpiBufBytes;
constexpr int kBiasBytes = kEpiWarpsFp4 * 256;  // per epilogue warp: BF16 bias of its two 64-column chunks
constexpr int kNumBars = 2 * kStages + 6 + kSfBufs + 2 * kSfSlots;
constexpr int kBarBytes = 512;
constexpr int kSmemBytes = kStages * kStageBytes + kSfSlots * kSfSlotBytes + kEpiBytes + kBiasBytes + kBarBytes + 1024;
static_assert(8 * kNumBars + 8 <= kBarBytes, "barrier area");
static_assert(kSfCol + kSfBufs * kSfBufCols <= kTmemCols, "TMEM budget");
static_assert(kSmemBytes <= 232448, "shared memory budget");

// Converts one 64-column chunk held in registers: fma(acc, alpha, bias) -> BF16 -> swizzled staging
// buffer -> TMA store (32 rows x 64 columns, clipped at the matrix edge).
__device__ __forceinline__ void epilogue_store(const CUtensorMap *tm_y, const Params &p, const uint32_t (&lo)[32],
                                               const uint32_t (&hi)[32], int m0, int nc, float alpha, uint32_t sbuf,
                                               uint32_t sbias, int lane) {
    if (lane == 0) ptx::tma_store_wait_read<0>();  // the previous store of this warp has left the staging buffer
    __syncwarp();
#pragma unroll
    for (int g = 0; g < 8; ++g) {
        uint32_t bw[4];  // 8 bias values of columns nc + 8g .. (same address in every lane: a broadcast read)
        asm volatile("ld.shared.v4.b32 {%0, %1, %2, %3}, [%4];"
                     : "=r"(bw[0]), "=r"(bw[1]), "=r"(bw[2]), "=r"(bw[3])
                     : "r"(sbias + g * 16));
        uint32_t o[4];
#pragma unroll
        for (int e = 0; e < 4; ++e) {
            const uint32_t a0 = g < 4 ? lo[g * 8 + 2 * e] : hi[(g - 4) * 8 + 2 * e];
            const uint32_t a1 = g < 4 ? lo[g * 8 + 2 * e + 1] : hi[(g - 4) * 8 + 2 * e + 1];
            const float y0 = fmaf(__uint_as_float(a0), alpha, __uint_as_float(bw[e] << 16));
            const float y1 = fmaf(__uint_as_float(a1), alpha, __uint_as_float(bw[e] & 0xFFFF0000u));
            __nv_bfloat162 pk = __floats2bfloat162_rn(y0, y1);
            o[e] = *reinterpret_cast<uint32_t *>(&pk);
        }
        const uint32_t chunk16 = static_cast<uint32_t>(g) ^ (lane & 7u);  // 128-byte swizzle
        const uint32_t dst = sbuf + lane * 128 + chunk16 * 16;
        asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(dst), "r"(o[0]), "r"(o[1]), "r"(o[2]), "r"(o[3])
                     : "memory");
    }
    ptx::fence_proxy_async_smem();
    __syncwarp();
    if (lane == 0) {
        if (nc < p.N && m0 < p.M && !(kTuning && (p.dbg & kDbgNoStore))) ptx::tma_store_2d(tm_y, nc, m0, sbuf);
        ptx::tma_store_commit();
    }
}

// Output modes of the kernel: BF16 Y, or Y passed through an activation and quantized for the next
// linear (packed E2M1 + E4M3 block scales along N, with a caller-supplied tensor scale).
// kOutSplit: tiles left of column n_split leave as BF16, tiles right of it quantized into a column
// range of a wider destination tensor (the concatenated input of the next linear).
enum : int { kOutBf16 = 0, kOutQuant = 1, kOutSplit = 2 };

// tanh-form GELU, 0.5 y (1 + tanh(u)), u = sqrt(2/pi) y (1 + 0.044715 y^2), with the hardware tanh
// (one special-function op per element; the epilogue is bound by that unit, and the exact form
// y / (1 + exp(-2u)) needs two).  tanh.approx is good to ~2^-11, far inside the BF16 rounding and
// the FP4 grid that follow.
__device__ __forceinline__ float gelu_tanh(float y) {
    const float u = y * fmaf(0.79788456080286536f * 0.044715f, y * y, 0.79788456080286536f);
    float t;
    asm("tanh.approx.f32 %0, %1;" : "=f"(t) : "f"(u));
    const float hy = 0.5f * y;
    return fmaf(hy, t, hy);
}

// The same 64-column chunk, but leaving as the next linear's quantized activations: h = bf16(act(
// fma(acc, alpha, bias))), then per 16 columns the block scale and sixteen nibbles in the
// quantizer's FP32 sequence.  A row's 64 columns are 32 bytes of nibbles (staged, one TMA store
// of 32 rows x 32 bytes per chunk) and the four scale bytes of one (row, k-chunk) slot of the
// chunked scale layout (one 4-byte store).  `amax2` collects max|h| per BF16 half.
__device__ __forceinline__ void epilogue_quant_store(const CUtensorMap *tm_q, const Params &p, const uint32_t (&lo)[32],
                                                     const uint32_t (&hi)[32], int m0, int quad_in_tile, int row_tile,
                                                     int nc, int nc_dst, float alpha, float Tq, float c6T, uint32_t sbuf,
                                                     uint32_t sbias, int lane, uint32_t &amax2) {
    const bool gelu = p.act != 0;
    if (lane == 0) ptx::tma_store_wait_read<0>();
    __syncwarp();
    uint32_t sfw = 0;
#pragma unroll
    for (int blk = 0; blk < 4; ++blk) {
        uint32_t hw[8];  // sixteen BF16 values of h
        uint32_t bm = 0;
#pragma unroll
        for (int g2 = 0; g2 < 2; ++g2) {
            const int g = blk * 2 + g2;
            uint32_t bw[4];
            asm volatile("ld.shared.v4.b32 {%0, %1, %2, %3}, [%4];"
                         : "=r"(bw[0]), "=r"(bw[1]), "=r"(bw[2]), "=r"(bw[3])
                         : "r"(sbias + g * 16));
#pragma unroll
            for (int e = 0; e < 4; ++e) {
                const uint32_t a0 = g < 4 ? lo[g * 8 + 2 * e] : hi[(g - 4) * 8 + 2 * e];
                const uint32_t a1 = g < 4 ? lo[g * 8 + 2 * e + 1] : hi[(g - 4) * 8 + 2 * e + 1];
                float y0 = fmaf(__uint_as_float(a0), alpha, __uint_as_float(bw[e] << 16));
                float y1 = fmaf(__uint_as_float(a1), alpha, __uint_as_float(bw[e] & 0xFFFF0000u));
                if (gelu) {
                    y0 = gelu_tanh(y0);
                    y1 = gelu_tanh(y1);
                }
                __nv_bfloat162 pk = __floats2bfloat162_rn(y0, y1);
                const uint32_t w = *reinterpret_cast<uint32_t *>(&pk);
                hw[g2 * 4 + e] = w;
                bm = qmath::absmax2(bm, w);
            }
        }
        amax2 = qmath::absmax2(amax2, bm);
        bm &= 0x7FFF7FFFu;
        const float a = __uint_as_float(max(bm & 0xFFFFu, bm >> 16) << 16);
        float rcp;
        const uint32_t sb = qmath::block_scale(a, c6T, Tq, rcp);
        sfw |= sb << (8 * blk);
        const uint32_t q0 = qmath::quantize8(hw[0], hw[1], hw[2], hw[3], rcp);
        const uint32_t q1 = qmath::quantize8(hw[4], hw[5], hw[6], hw[7], rcp);
        asm volatile("st.shared.v2.b32 [%0], {%1, %2};" ::"r"(sbuf + lane * 32 + blk * 8), "r"(q0), "r"(q1) : "memory");
    }
    const bool unit_ok = nc < p.N && !(kTuning && (p.dbg & kDbgNoStore));
    if (unit_ok && row_tile * 128 < p.M) {
        // rows past M inside the last 128-row chunk are padding and read as 0
        if (m0 + lane >= p.M) sfw = 0;
        const int64_t chunk = static_cast<int64_t>(row_tile) * p.dest_chunks_k + (nc_dst >> 6);
        *reinterpret_cast<uint32_t *>(p.sf_out + chunk * 512 + lane * 16 + quad_in_tile * 4) = sfw;
    }
    ptx::fence_proxy_async_smem();
    __syncwarp();
    if (lane == 0) {
        if (unit_ok && m0 < p.M) ptx::tma_store_2d(tm_q, nc_dst >> 1, m0, sbuf);
        ptx::tma_store_commit();
    }
}

// The MXFP4 form of the same: two 32-element blocks per 64-column chunk, each with the E8M0 scale
// 2^(floor(log2 amax) - 2) taken from the exponent field of the block maximum, codes by an exact
// power-of-two scaling; no tensor scale.  A scale chunk of the destination spans 128 columns, so the
// chunk's two scale bytes are one 2-byte store into the lower or upper half of a (row, chunk) slot.
__device__ __forceinline__ void epilogue_quant_store_mx(const CUtensorMap *tm_q, const Params &p, const uint32_t (&lo)[32],
                                                        const uint32_t (&hi)[32], int m0, int quad_in_tile, int row_tile,
                                                        int nc, int nc_dst, float alpha, uint32_t sbuf, uint32_t sbias,
                                                        int lane, uint32_t &amax2) {
    const bool gelu = p.act != 0;
    if (lane == 0) ptx::tma_store_wait_read<0>();
    __syncwarp();
    uint32_t sfw = 0;
#pragma unroll
    for (int blk = 0; blk < 2; ++blk) {
        uint32_t hw[16];  // thirty-two BF16 values of h
        uint32_t bm = 0;
#pragma unroll
        for (int g4 = 0; g4 < 4; ++g4) {
            const int g = blk * 4 + g4;
            uint32_t bw[4];
            asm volatile("ld.shared.v4.b32 {%0, %1, %2, %3}, [%4];"
                         : "=r"(bw[0]), "=r"(bw[1]), "=r"(bw[2]), "=r"(bw[3])
                         : "r"(sbias + g * 16));
#pragma unroll
            for (int e = 0; e < 4; ++e) {
                const uint32_t a0 = g < 4 ? lo[g * 8 + 2 * e] : hi[(g - 4) * 8 + 2 * e];
                const uint32_t a1 = g < 4 ? lo[g * 8 + 2 * e + 1] : hi[(g - 4) * 8 + 2 * e + 1];
                float y0 = fmaf(__uint_as_float(a0), alpha, __uint_as_float(bw[e] << 16));
                float y1 = fmaf(__uint_as_float(a1), alpha, __uint_as_float(bw[e] & 0xFFFF0000u));
                if (gelu) {
                    y0 = gelu_tanh(y0);
                    y1 = gelu_tanh(y1);
                }
                __nv_bfloat162 pk = __floats2bfloat162_rn(y0, y1);
                const uint32_t w = *reinterpret_cast<uint32_t *>(&pk);
                hw[g4 * 4 + e] = w;
                bm = qmath::absmax2(bm, w);
            }
        }
        amax2 = qmath::absmax2(amax2, bm);
        bm &= 0x7FFF7FFFu;
        const uint32_t e8 = max(bm & 0xFFFFu, bm >> 16) >> 7;   // biased exponent of the block maximum
        const uint32_t sb = e8 > 2u ? e8 - 2u : 0u;             // shared exponent floor(log2 amax) - 2, clamped at -127
        const float inv = __uint_as_float((254u - sb) << 23);   // 2^(127 - sb), exact
        sfw |= sb << (8 * blk);
#pragma unroll
        for (int h8 = 0; h8 < 2; ++h8) {
            const uint32_t q0 = qmath::quantize8(hw[8 * h8], hw[8 * h8 + 1], hw[8 * h8 + 2], hw[8 * h8 + 3], inv);
            const uint32_t q1 = qmath::quantize8(hw[8 * h8 + 4], hw[8 * h8 + 5], hw[8 * h8 + 6], hw[8 * h8 + 7], inv);
            asm volatile("st.shared.v2.b32 [%0], {%1, %2};" ::"r"(sbuf + lane * 32 + blk * 16 + h8 * 8), "r"(q0), "r"(q1)
                         : "memory");
        }
    }
    const bool unit_ok = nc < p.N && !(kTuning && (p.dbg & kDbgNoStore));
    if (unit_ok && row_tile * 128 < p.M) {
        if (m0 + lane >= p.M) sfw = 0;  // rows past M inside the last 128-row chunk are padding and read as 0
        const int64_t chunk = static_cast<int64_t>(row_tile) * p.dest_chunks_k + (nc_dst >> 7);
        *reinterpret_cast<uint16_t *>(p.sf_out + chunk * 512 + lane * 16 + quad_in_tile * 4 + ((nc_dst >> 6) & 1) * 2) =
            static_cast<uint16_t>(sfw);
    }
    ptx::fence_proxy_async_smem();
    __syncwarp();
    if (lane == 0) {
        if (unit_ok && m0 < p.M) ptx::tma_store_2d(tm_q, nc_dst >> 1, m0, sbuf);
        ptx::tma_store_commit();
    }
}

// kMx: MXFP4 operands (32-element blocks, E8M0 scales: a 512-byte scale chunk spans 128 elements of K,
// so a k-tile has two chunks per 128 rows instead of four, and no tensor scales) -- BF16 output, or
// (kOutQuant) the next linear's MXFP4 activations.
template <int kOut, bool kMx>
__global__ void __launch_bounds__(kThreadsFp4, 1)
gemm_pair_fp4_kernel(const __grid_constant__ CUtensorMap tm_a, const __grid_constant__ CUtensorMap tm_b,
                     const __grid_constant__ CUtensorMap tm_y, const __grid_constant__ CUtensorMap tm_q,
                     const __grid_constant__ CUtensorMap tm_sfa, const __grid_constant__ CUtensorMap tm_sfb,
                     const Params p) {
    extern __shared__ uint8_t smem_raw[];
    const uint32_t smem_base = (ptx::smem_u32(smem_raw) + 1023u) & ~1023u;
    uint8_t *smem_gen = smem_raw + (smem_base - ptx::smem_u32(smem_raw));

    const uint32_t sf_base = smem_base + kStages * kStageBytes;
    const uint32_t epi_base = sf_base + kSfSlots * kSfSlotBytes;
    const uint32_t bias_base = epi_base + kEpiBytes;
    const uint32_t bar_base = bias_base + kBiasBytes;
    uint8_t *bar_gen = smem_gen + kStages * kStageBytes + kSfSlots * kSfSlotBytes + kEpiBytes + kBiasBytes;
    auto full_bar = [&](int s) { return bar_base + 8u * s; };
    auto empty_bar = [&](int s) { return bar_base + 8u * (kStages + s); };
    auto acc_full_bar = [&](int s) { return bar_base + 8u * (2 * kStages + s); };
    auto acc_empty_bar = [&](int s) { return bar_base + 8u * (2 * kStages + 2 + s); };
    auto ovl_free_bar = [&](int s) { return bar_base + 8u * (2 * kStages + 4 + s); };
    auto sf_ready_bar = [&](int s) { return bar_base + 8u * (2 * kStages + 6 + s); };
    // The scale tiles travel in a ring of their own, a sixth of a k-tile's bytes each.  A slot is handed
    // back as soon as the copy warps hold its contents in registers, not when the k-tile's MMAs are
    // done, so the scale loads run several k-tiles ahead of the A and B loads and the copy into tensor
    // memory (load -> registers -> tcgen05.st -> arrive, ~800 cycles end to end) is off the critical path.
    auto sf_full_bar = [&](int s) { return bar_base + 8u * (2 * kStages + 6 + kSfBufs + s); };
    auto sf_empty_bar = [&](int s) { return bar_base + 8u * (2 * kStages + 6 + kSfBufs + kSfSlots + s); };
    uint32_t *tmem_ptr_smem = reinterpret_cast<uint32_t *>(bar_gen + 8 * kNumBars);
    volatile uint32_t *abort_flag = reinterpret_cast<volatile uint32_t *>(bar_gen + 8 * kNumBars + 4);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const uint32_t rank = ptx::cluster_ctarank();
    const bool leader = rank == 0;
    const int pair = blockIdx.x >> 1, num_pairs = gridDim.x >> 1;
    const int total_tiles = p.m_tiles * p.n_tiles;
    const int k_tiles = (p.K + kBK - 1) / kBK;
    const int tail_mmas = (p.K - (k_tiles - 1) * kBK + kMmaK - 1) / kMmaK;  // MMAs of the last k-tile (1..4)
    constexpr int kSfChunksK = kMx ? 2 : 4;                  // scale chunks along K per stage and 128 rows
    constexpr int kSfRowChunkBytes = kSfChunksK * 512;       // one 128-row chunk's scales of a stage
    constexpr int kSfLoadBytes = 3 * kSfRowChunkBytes;       // A (one row chunk) + B (two)

    if (threadIdx.x == 0) {
        for (int s = 0; s < kStages; ++s) {
            ptx::mbar_init(full_bar(s), 1);
            ptx::mbar_init(empty_bar(s), 1);
        }
        for (int s = 0; s < kSfSlots; ++s) {
            ptx::mbar_init(sf_full_bar(s), 1);
            ptx::mbar_init(sf_empty_bar(s), kSfCopyWarps);
        }
        for (int s = 0; s < 2; ++s) {
            ptx::mbar_init(acc_full_bar(s), 1);
            ptx::mbar_init(acc_empty_bar(s), 2 * kEpiWarpsFp4);
            ptx::mbar_init(ovl_free_bar(s), 2 * kEpiWarpsFp4);
        }
        for (int s = 0; s < kSfBufs; ++s) ptx::mbar_init(sf_ready_bar(s), 2 * kSfCopyWarps);
        *abort_flag = 0;
        ptx::fence_mbar_init();
        ptx::prefetch_tmap(&tm_a);
        ptx::prefetch_tmap(&tm_b);
        ptx::prefetch_tmap(&tm_y);
        ptx::prefetch_tmap(&tm_q);
        ptx::prefetch_tmap(&tm_sfa);
        ptx::prefetch_tmap(&tm_sfb);
    }
    if (warp == 1) {
        ptx::tmem_alloc_pair(ptx::smem_u32(tmem_ptr_smem), kTmemCols);
        ptx::tmem_relinquish_pair();
    }
    ptx::tc_fence_before_sync();
    __syncthreads();
    ptx::cluster_sync();
    ptx::tc_fence_after_sync();
    const uint32_t tmem_base = *tmem_ptr_smem;
    ptx::grid_dependency_wait();  // set-up above overlaps the previous kernel; its results are read below
#ifdef SOL_SPAN
    long long span_c0 = 0, span_g0 = 0;
    if (threadIdx.x == 0 && blockIdx.x == 0) {
        span_c0 = clock64();
        asm volatile("mov.u64 %0, %globaltimer;" : "=l"(span_g0));
    }
#endif

    if (kTuning && warp == kWarps) {
        // diagnostic build: polls each stage's `full` barrier without suspending and records when it completes
        if ((p.dbg & kDbgTrace) && leader && lane < 2) {
            int stage = 0;
            uint32_t phase = 0;
            const int n = ((total_tiles - pair + num_pairs - 1) / num_pairs) * k_tiles;
            for (int gi = 0; gi < n && gi < 512; ++gi) {
                const long long t0 = clock64();
                const uint32_t bar = lane == 0 ? full_bar(stage) : empty_bar(stage);
                while (!ptx::mbar_test_wait(bar, phase) && clock64() - t0 < 4000000) {}
#ifdef SOL_TUNING
                if (blockIdx.x < 2) g_trace[lane == 0 ? 11 : 1][gi] = clock64();
#endif
                if (++stage == kStages) { stage = 0; phase ^= 1u; }
            }
        }
    } else if (warp == 0) {
        // ------------------------------------------------------------ TMA producer: A and B tiles (both CTAs)
        const bool elected = ptx::elect_one();
        const uint32_t full0 = ptx::map_to_cta(full_bar(0), 0);  // the even CTA's barriers
        const bool no_b = kTuning && (p.dbg & kDbgNoBLoad);
        const uint32_t tx = 2u * (kABytes + (no_b ? 0 : kBBytes));
        [[maybe_unused]] int gi_trace = 0;
        int stage = 0;
        uint32_t phase = 0;
        bool ok = !loads_held(p.status);
        for (int t = pair; ok && t < total_tiles; t += num_pairs) {
            int mt, nt;
            tile_coords(t, p.m_tiles, p.n_tiles, mt, nt);
            const int m0 = mt * 2 * kBM + static_cast<int>(rank) * kBM;
            const int nb0 = nt * kBN + static_cast<int>(rank) * (kBN / 2);
            int kx = 0;
            for (int kt = 0; kt < k_tiles; ++kt, kx += kRowBytes) {
                if (!wait_bounded(empty_bar(stage), phase ^ 1u, abort_flag, p.status, 0x100u | stage)) {
                    ok = false;
                    break;
                }
                const uint32_t sa = smem_base + stage * kStageBytes;
                if (kTuning && (p.dbg & kDbgTrace) && leader) { SOL_TRACE(0, gi_trace); ++gi_trace; }
                if (elected) {
                    if (leader) ptx::mbar_arrive_expect_tx(full_bar(stage), tx);
                    ptx::tma_load_2d_pair(sa, &tm_a, kx, m0, full0 + 8u * stage);
                    if (!no_b) ptx::tma_load_2d_pair(sa + kABytes, &tm_b, kx, nb0, full0 + 8u * stage);
                }
                if (++stage == kStages) {
                    stage = 0;
                    phase ^= 1u;
                }
            }
        }
        __syncwarp();
    } else if (warp == kWarps - 1) {
        // ------------------------------------------------------------ TMA producer: scale-factor tiles (both CTAs)
        // Each CTA's tiles complete on a barrier of its own, where its own copy warps wait.
        const bool elected = ptx::elect_one();
        const uint32_t full0 = ptx::map_to_cta(sf_full_bar(0), rank);
        [[maybe_unused]] int sf_gi_trace = 0;
        int slot = 0;
        uint32_t phase = 0;
        bool ok = !loads_held(p.status);
        for (int t = pair; ok && t < total_tiles; t += num_pairs) {
            int mt, nt;
            tile_coords(t, p.m_tiles, p.n_tiles, mt, nt);
            const int rca = mt * 2 + static_cast<int>(rank);  // 128-row chunk of A owned by this CTA
            const int rcb = nt * 2;                            // first of the tile's two 128-row chunks of B
            for (int kt = 0; kt < k_tiles; ++kt) {
                if (!wait_bounded(sf_empty_bar(slot), phase ^ 1u, abort_flag, p.status, 0x800u | slot)) {
                    ok = false;
                    break;
                }
                const uint32_t ssfa = sf_base + slot * kSfSlotBytes;
                if (kTuning && (p.dbg & kDbgTrace) && leader) { SOL_TRACE(2, sf_gi_trace); ++sf_gi_trace; }
                if (elected) {
                    ptx::mbar_arrive_expect_tx(sf_full_bar(slot), kSfLoadBytes);
                    ptx::tma_load_3d_pair(ssfa, &tm_sfa, 0, kt * kSfChunksK, rca, full0 + 8u * slot);
                    ptx::tma_load_3d_pair(ssfa + kSfaBytes, &tm_sfb, 0, kt * kSfChunksK, rcb, full0 + 8u * slot);
                }
                if (++slot == kSfSlots) {
                    slot = 0;
                    phase ^= 1u;
                }
            }
        }
        __syncwarp();
    } else if (warp == 1) {
        // ------------------------------------------------------------ MMA issuer (even CTA)
        // The loop is warp-uniform so every operand lives in uniform registers; one elected lane issues.
        if (leader) {
            const bool elected = ptx::elect_one();
            // E2M1 x E2M1, M = 256; scale format UE4M3 (0) or UE8M0 (1) in bit 23
            const uint32_t idesc = (1u << 7) | (1u << 10) | (static_cast<uint32_t>(kBN >> 3) << 17) |
                                   (kMx ? (1u << 23) : 0u) | (static_cast<uint32_t>((2 * kBM) >> 4) << 24);
            // MXFP4: the odd instruction of a scale chunk takes bytes 2..3 of the scale columns (scale ids of
            // A in bits 29..30, of B in bits 4..5)
            constexpr uint32_t kSfIdHi = (2u << 29) | (2u << 4);
            const uint64_t desc_hi = ptx::smem_desc_sw128(0);
            const uint32_t a_lo0 = (smem_base & 0x3FFFFu) >> 4;
            const uint32_t b_lo0 = ((smem_base + kABytes) & 0x3FFFFu) >> 4;
            constexpr uint32_t kStageLo = kStageBytes >> 4;
            const bool no_mma = kTuning && (p.dbg & kDbgNoMma);
            const bool trace = kTuning && (p.dbg & kDbgTrace);
            int stage = 0;
            uint32_t phase = 0;
            uint32_t gi = 0;
            uint32_t sf_buf = 0, sf_phase = 0;  // scale-factor buffer ring
            bool sf_seen = false;
            bool ok = true;
            for (int t = pair, it = 0; ok && t < total_tiles; t += num_pairs, ++it) {
                const int x = it & 1;
                const uint32_t use = static_cast<uint32_t>(it >> 1);
                // this accumulator's previous tile is fully drained ...
                if (!wait_bounded(acc_empty_bar(x), (use & 1u) ^ 1u, abort_flag, p.status, 0x200u | x)) break;
                // ... and the previous tile (other accumulator) has given back the shared columns
                if (it > 0 && !wait_bounded(ovl_free_bar(x ^ 1), (static_cast<uint32_t>(it - 1) >> 1) & 1u, abort_flag,
                                            p.status, 0x900u | x))
                    break;
                ptx::tc_fence_after_sync();
                if (trace) SOL_TRACE(8, it);
                const uint32_t d_tmem = tmem_base + x * kAccStride;
                for (int kt = 0; kt < k_tiles; ++kt) {
                    // two conditions per k-tile: the scales are in TMEM (`sf_ready`, signalled by the copy warps,
                    // normally long before) and A and B are in shared memory (`full`); `sf_seen`: the previous
                    // k-tile already saw both complete (peek below)
                    if (!sf_seen) {
                        if (!wait_bounded(sf_ready_bar(sf_buf), sf_phase, abort_flag, p.status, 0x500u | sf_buf)) {
                            ok = false;
                            break;
                        }
                        if (!wait_bounded(full_bar(stage), phase, abort_flag, p.status, 0x300u | stage)) {
                            ok = false;
                            break;
                        }
                    }
                    ptx::tc_fence_after_sync();
                    if (trace) SOL_TRACE(6, gi);
                    const uint64_t a_desc = desc_hi | (a_lo0 + static_cast<uint32_t>(stage) * kStageLo);
                    const uint64_t b_desc = desc_hi | (b_lo0 + static_cast<uint32_t>(stage) * kStageLo);
                    const uint32_t sfa_t = tmem_base + kSfCol + sf_buf * kSfBufCols;
                    const uint32_t sfb_t = sfa_t + 16;
                    if (elected && !no_mma) {
                        if (kMx) {
                            const int nm = (kt + 1 < k_tiles) ? kMmasPerStage : tail_mmas;
#pragma unroll
                            for (int j = 0; j < kMmasPerStage; ++j)
                                if (j < nm)
                                    ptx::mma_mxfp4_pair(d_tmem, a_desc + 2u * j, b_desc + 2u * j,
                                                        idesc | ((j & 1) ? kSfIdHi : 0u), sfa_t + 4 * (j >> 1),
                                                        sfb_t + 8 * (j >> 1), (kt | j) != 0);
                        } else if (kt + 1 < k_tiles || tail_mmas == kMmasPerStage) {
                            ptx::mma_nvfp4_pair(d_tmem, a_desc, b_desc, idesc, sfa_t, sfb_t, kt != 0);
                            ptx::mma_nvfp4_pair(d_tmem, a_desc + 2, b_desc + 2, idesc, sfa_t + 4, sfb_t + 8, 1);
                            ptx::mma_nvfp4_pair(d_tmem, a_desc + 4, b_desc + 4, idesc, sfa_t + 8, sfb_t + 16, 1);
                            ptx::mma_nvfp4_pair(d_tmem, a_desc + 6, b_desc + 6, idesc, sfa_t + 12, sfb_t + 24, 1);
                        } else {
                            for (int j = 0; j < tail_mmas; ++j)  // ragged K: fewer than four 32-byte slices are valid
                                ptx::mma_nvfp4_pair(d_tmem, a_desc + 2u * j, b_desc + 2u * j, idesc, sfa_t + 4 * j,
                                                    sfb_t + 8 * j, (kt | j) != 0);
                        }
                    }
                    // next k-tile's scale-factor buffer (it may belong to the next tile)
                    const uint32_t nb = sf_buf + 1 == kSfBufs ? 0u : sf_buf + 1;
                    const uint32_t np = sf_buf + 1 == kSfBufs ? sf_phase ^ 1u : sf_phase;
                    // commit frees the stage in both CTAs; the peek tells whether the next buffer is ready
                    const int ns = stage + 1 == kStages ? 0 : stage + 1;
                    const uint32_t nph = stage + 1 == kStages ? phase ^ 1u : phase;
                    bool seen = false;
                    if (elected)
                        seen = ptx::tc_commit_pair_mcast_and_peek2(empty_bar(stage), 3, sf_ready_bar(nb), np, full_bar(ns), nph);
                    sf_seen = __any_sync(0xFFFFFFFFu, seen) != 0;  // keeps the loop warp-uniform
                    if (trace) SOL_TRACE(3, gi);
                    ++gi;
                    sf_buf = nb;
                    sf_phase = np;
                    if (++stage == kStages) {
                        stage = 0;
                        phase ^= 1u;
                    }
                }
                if (ok && elected) ptx::tc_commit_pair_mcast(acc_full_bar(x), 3);
                if (trace) SOL_TRACE(7, it);
            }
        }
        __syncwarp();
    } else if (warp >= 2 + kEpiWarpsFp4) {
        // ------------------------------------------------------------ scale-factor copy warps (both CTAs)
        // One warp per TMEM lane quadrant: lane t takes line t (16 bytes) of each 512-byte chunk into
        // registers, the slot goes back to the producer at once, and when the k-tile's buffer in tensor
        // memory is free (the MMAs of three k-tiles ago are done) the lines are written to the warp's own
        // quadrant with tcgen05.st -- the four warps together give the four-fold replication that the
        // scaled MMA reads.  Nothing of this passes through the tensor pipe or the MMA thread.
        {
            const bool elected = ptx::elect_one();
            const int w = warp - (2 + kEpiWarpsFp4);
            const uint32_t ready0 = ptx::map_to_cta(sf_ready_bar(0), 0);  // the even CTA's barriers
            int slot = 0;
            uint32_t phase = 0;
            uint32_t gi = 0;
            uint32_t sf_buf = 0;
            int old_stage = kStages - kSfBufs;  // smem stage of k-tile gi - kSfBufs, the last reader of this buffer
            uint32_t old_phase = 1;             // parity its `empty` barrier shows once those MMAs are done
            bool ok = true;
            for (int t = pair; ok && t < total_tiles; t += num_pairs) {
                for (int kt = 0; kt < k_tiles; ++kt) {
                    if (!wait_bounded(sf_full_bar(slot), phase, abort_flag, p.status, 0x600u | slot)) {
                        ok = false;
                        break;
                    }
                    const uint32_t ssf = sf_base + slot * kSfSlotBytes + lane * 16;
                    uint4 v[3 * kSfChunksK];
#pragma unroll
                    for (int c = 0; c < kSfChunksK; ++c) {
                        v[c] = ptx::lds128(ssf + c * 512);
                        v[kSfChunksK + c] = ptx::lds128(ssf + kSfaBytes + c * 512);
                        v[2 * kSfChunksK + c] = ptx::lds128(ssf + kSfaBytes + kSfRowChunkBytes + c * 512);
                    }
                    // the slot's next contents arrive through the async proxy: order these generic-proxy reads
                    // before it (the release chain to the producer starts at the arrive)
                    ptx::fence_proxy_async_smem();
                    __syncwarp();
                    if (elected) ptx::mbar_arrive(sf_empty_bar(slot));
                    if (gi >= kSfBufs && !(kTuning && (p.dbg & kDbgNoSfCopy)) &&
                        !wait_bounded(empty_bar(old_stage), old_phase, abort_flag, p.status, 0x700u | old_stage)) {
                        ok = false;
                        break;
                    }
                    ptx::tc_fence_after_sync();
                    if (kTuning && (p.dbg & kDbgTrace) && w == 0 && leader) SOL_TRACE(4, gi);
                    const uint32_t sf_t = tmem_base + kSfCol + sf_buf * kSfBufCols + (static_cast<uint32_t>(warp & 3) << 21);
#pragma unroll
                    for (int c = 0; c < kSfChunksK; ++c) {
                        ptx::tc_store_32x32b_x4(sf_t + 4 * c, v[c]);
                        ptx::tc_store_32x32b_x4(sf_t + 16 + 8 * c, v[kSfChunksK + c]);
                        ptx::tc_store_32x32b_x4(sf_t + 20 + 8 * c, v[2 * kSfChunksK + c]);
                    }
                    ptx::tc_wait_st();
                    ptx::tc_fence_before_sync();
                    __syncwarp();
                    if (elected) ptx::mbar_arrive_cluster(ready0 + 8u * sf_buf);
                    if (kTuning && (p.dbg & kDbgTrace) && w == 0 && leader) SOL_TRACE(5, gi);
                    ++gi;
                    if (++sf_buf == kSfBufs) sf_buf = 0;
                    if (++old_stage == kStages) {
                        old_stage = 0;
                        old_phase ^= 1u;
                    }
                    if (++slot == kSfSlots) {
                        slot = 0;
                        phase ^= 1u;
                    }
                }
            }
        }
        __syncwarp();
    } else {
        // ------------------------------------------------------------ epilogue (warps 2..9, both CTAs)
        const int e = warp - 2;
        const int quad = warp & 3;   // TMEM lanes [32*quad, 32*quad+32)
        const int half = e >> 2;     // which of the quadrant's two warps
        const uint32_t sbuf = epi_base + e * kEpiBufBytes;
        const uint32_t sbias = bias_base + e * 256;
        const float alpha = kMx ? 1.0f : __fmul_rn(__ldcg(p.ts_a), __ldcg(p.ts_b));
        const float Tq = (kOut != kOutBf16 && !kMx) ? __ldcg(p.ts_out) : 1.0f;
        const float c6T = __fmul_rn(6.0f, Tq);
        uint32_t amax2 = 0;
        for (int t = pair, it = 0; t < total_tiles; t += num_pairs, ++it) {
            int mt, nt;
            tile_coords(t, p.m_tiles, p.n_tiles, mt, nt);
            const int m0 = mt * 2 * kBM + static_cast<int>(rank) * kBM + quad * 32, n0 = nt * kBN;
            const int row_tile = mt * 2 + static_cast<int>(rank);
            const int x = it & 1;
            // 64-column units of the accumulator.  A (base 0) shares its columns [96,256) with the next
            // tile: units 2, 3 and the upper half of unit 1; B (base 96) its columns [0,160): units 0, 1 and
            // the lower half of unit 2.  Each warp takes one fully shared unit first and one other unit.
            const int first = x == 0 ? 2 + half : half;
            const int second = x == 0 ? half : 2 + half;
            {   // stage this warp's 2 x 64 bias values in shared memory while the main loop is still running
                const int unit = lane < 16 ? first : second;
                const int col = n0 + unit * 64 + (lane & 15) * 4;
                uint2 bv = make_uint2(0, 0);
                if (p.bias != nullptr && col < p.N) bv = __ldg(reinterpret_cast<const uint2 *>(p.bias + col));
                __syncwarp();  // the previous tile's reads of the staging area are done
                asm volatile("st.shared.v2.b32 [%0], {%1, %2};" ::"r"(sbias + lane * 8), "r"(bv.x), "r"(bv.y) : "memory");
                __syncwarp();
            }
            if (!wait_bounded(acc_full_bar(x), (static_cast<uint32_t>(it) >> 1) & 1u, abort_flag, p.status, 0x400u | x)) break;
            ptx::tc_fence_after_sync();
            if (kTuning && (p.dbg & kDbgTrace) && warp == 2) SOL_TRACE(9, it);
            const uint32_t t_acc = tmem_base + (static_cast<uint32_t>(quad * 32) << 16) + x * kAccStride;
            const uint32_t ovl_bar = ptx::map_to_cta(ovl_free_bar(x), 0);
            const uint32_t done_bar = ptx::map_to_cta(acc_empty_bar(x), 0);
            if (kTuning && (p.dbg & kDbgNoEpilogue)) {
                ptx::tc_fence_before_sync();
                __syncwarp();
                if (lane == 0) {
                    ptx::mbar_arrive_cluster(ovl_bar);
                    ptx::mbar_arrive_cluster(done_bar);
                }
                continue;
            }
            // The shared columns leave TMEM first and go straight back to the MMA warp; the arithmetic
            // runs from registers afterwards.  A warp whose second unit is partly shared also fetches
            // that half before it releases.
            const bool early = half == x;                 // second unit holds no shared columns
            const uint32_t t1 = t_acc + first * 64, t2 = t_acc + second * 64;
            const uint32_t shared_half = x == 0 ? 32u : 0u;  // A: upper half of unit 1, B: lower half of unit 2
            uint32_t a_lo[32], a_hi[32], b_sh[32], b_ot[32];
            ptx::tmem_ld_32x32(t1, a_lo);
            ptx::tmem_ld_32x32(t1 + 32, a_hi);
            if (!early) ptx::tmem_ld_32x32(t2 + shared_half, b_sh);
            ptx::tmem_ld_wait();
            ptx::tc_fence_before_sync();
            __syncwarp();
            if (lane == 0) ptx::mbar_arrive_cluster(ovl_bar);
            if (kTuning && (p.dbg & kDbgTrace) && warp == 2) SOL_TRACE(10, it);
            // split mode decides per tile; the quantized part lands at a column offset of the destination
            const bool as_bf16 = kOut == kOutBf16 || (kOut == kOutSplit && n0 < p.n_split);
            const int dst_shift = kOut == kOutSplit ? p.dest_col0 - p.n_split : 0;
            if (as_bf16)
                epilogue_store(&tm_y, p, a_lo, a_hi, m0, n0 + first * 64, alpha, sbuf, sbias, lane);
            else if constexpr (kMx)
                epilogue_quant_store_mx(&tm_q, p, a_lo, a_hi, m0, quad, row_tile, n0 + first * 64,
                                        n0 + first * 64 + dst_shift, alpha, sbuf, sbias, lane, amax2);
            else
                epilogue_quant_store(&tm_q, p, a_lo, a_hi, m0, quad, row_tile, n0 + first * 64,
                                     n0 + first * 64 + dst_shift, alpha, Tq, c6T, sbuf, sbias, lane, amax2);
            if (early) ptx::tmem_ld_32x32(t2 + shared_half, b_sh);
            ptx::tmem_ld_32x32(t2 + (shared_half ^ 32u), b_ot);
            ptx::tmem_ld_wait();
            ptx::tc_fence_before_sync();
            __syncwarp();
            if (lane == 0) ptx::mbar_arrive_cluster(done_bar);
            if (as_bf16) {
                if (x == 0)  // b_sh is the upper half
                    epilogue_store(&tm_y, p, b_ot, b_sh, m0, n0 + second * 64, alpha, sbuf, sbias + 128, lane);
                else
                    epilogue_store(&tm_y, p, b_sh, b_ot, m0, n0 + second * 64, alpha, sbuf, sbias + 128, lane);
            } else if constexpr (kMx) {
                if (x == 0)
                    epilogue_quant_store_mx(&tm_q, p, b_ot, b_sh, m0, quad, row_tile, n0 + second * 64,
                                            n0 + second * 64 + dst_shift, alpha, sbuf, sbias + 128, lane, amax2);
                else
                    epilogue_quant_store_mx(&tm_q, p, b_sh, b_ot, m0, quad, row_tile, n0 + second * 64,
                                            n0 + second * 64 + dst_shift, alpha, sbuf, sbias + 128, lane, amax2);
            } else {
                if (x == 0)
                    epilogue_quant_store(&tm_q, p, b_ot, b_sh, m0, quad, row_tile, n0 + second * 64,
                                         n0 + second * 64 + dst_shift, alpha, Tq, c6T, sbuf, sbias + 128, lane, amax2);
                else
                    epilogue_quant_store(&tm_q, p, b_sh, b_ot, m0, quad, row_tile, n0 + second * 64,
                                         n0 + second * 64 + dst_shift, alpha, Tq, c6T, sbuf, sbias + 128, lane, amax2);
            }
        }
        if (lane == 0) ptx::tma_store_wait_all<0>();
        if (kOut != kOutBf16 && p.amax_out != nullptr) {
            amax2 &= 0x7FFF7FFFu;
            uint32_t m = max(amax2 & 0xFFFFu, amax2 >> 16);
            m = __reduce_max_sync(0xFFFFFFFFu, m);
            if (lane == 0 && m) atomicMax(p.amax_out, m << 16);
        }
    }

    // ---------------------------------------------------------------- teardown
    if (*abort_flag) __nanosleep(2000000);
    ptx::tc_fence_before_sync();
    __syncthreads();
    ptx::cluster_sync();  // neither CTA frees TMEM or exits while its partner may still touch it
#ifdef SOL_SPAN
    if (threadIdx.x == 0 && blockIdx.x == 0) {
        long long g1;
        asm volatile("mov.u64 %0, %globaltimer;" : "=l"(g1));
        g_span[0] = clock64() - span_c0;
        g_span[1] = g1 - span_g0;
    }
#endif
    if (warp == 1) {
        ptx::tc_fence_after_sync();
        ptx::tmem_dealloc_pair(tmem_base, kTmemCols);
    }
}

}  // namespace

namespace {

struct QuantOut {          // where a quantized output goes (kOutQuant, kOutSplit)
    int act = 0;
    const float *ts_out = nullptr;
    void *hq = nullptr;
    void *hsf = nullptr;
    uint32_t *amax_out = nullptr;
    int64_t n_split = 0;   // kOutSplit: columns [0, n_split) leave as BF16 through y / ldy
    int64_t dest_K = 0;    // width of the destination tensor (its own N when not split)
    int64_t dest_col0 = 0;
};

sol_status_t launch_pair256(int out_mode, bool mx, const void *xq, const void *xsf, const float *xts, const void *wq,
                            const void *wsf, const float *wts, const void *bias, void *y, int64_t ldy,
                            const QuantOut &qo, int64_t M, int64_t N, int64_t K, cudaStream_t stream,
                            const DeviceInfo *dev) {
    const uint64_t chunks_k = static_cast<uint64_t>(ceil_div(K, mx ? 128 : 64));
    const uint32_t box_k = mx ? 2 : 4;
    CUtensorMap tm_a, tm_b, tm_y, tm_q, tm_sfa, tm_sfb;
    bool ok = make_tmap_2d(&tm_a, CU_TENSOR_MAP_DATA_TYPE_UINT8, 1, xq, K / 2, M, K / 2, 128, kBM,
                           CU_TENSOR_MAP_SWIZZLE_128B) &&
              make_tmap_2d(&tm_b, CU_TENSOR_MAP_DATA_TYPE_UINT8, 1, wq, K / 2, N, K / 2, 128, kBN / 2,
                           CU_TENSOR_MAP_SWIZZLE_128B) &&
              make_tmap_sf(&tm_sfa, xsf, chunks_k, static_cast<uint64_t>(ceil_div(M, 128)), 1, box_k) &&
              make_tmap_sf(&tm_sfb, wsf, chunks_k, static_cast<uint64_t>(ceil_div(N, 128)), 2, box_k);
    if (out_mode != kOutQuant)  // BF16 output: all N columns, or the first n_split of them
        ok = ok && make_tmap_2d(&tm_y, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, y, out_mode == kOutSplit ? qo.n_split : N, M,
                                ldy * 2, 64, 32, CU_TENSOR_MAP_SWIZZLE_128B);
    if (out_mode != kOutBf16)   // packed nibbles [M, dest_K/2]: boxes of 32 rows x 32 bytes (64 columns)
        ok = ok && make_tmap_2d(&tm_q, CU_TENSOR_MAP_DATA_TYPE_UINT8, 1, qo.hq, qo.dest_K / 2, M, qo.dest_K / 2, 32, 32,
                                CU_TENSOR_MAP_SWIZZLE_NONE);
    if (!ok) return SOL_ERR_CUDA;
    if (out_mode == kOutQuant) tm_y = tm_q;  // unused, but a valid descriptor for the prefetch
    if (out_mode == kOutBf16) tm_q = tm_y;
    Params p{};
    p.sfa = static_cast<const uint8_t *>(xsf);
    p.sfb = static_cast<const uint8_t *>(wsf);
    p.ts_a = xts;
    p.ts_b = wts;
    p.bias = static_cast<const uint16_t *>(bias);
    p.status = device_status_word();
    p.M = static_cast<int>(M);
    p.N = static_cast<int>(N);
    p.K = static_cast<int>(K);
    p.sf_out = static_cast<uint8_t *>(qo.hsf);
    p.ts_out = qo.ts_out;
    p.amax_out = qo.amax_out;
    p.act = qo.act;
    p.n_split = static_cast<int>(qo.n_split);
    p.dest_col0 = static_cast<int>(qo.dest_col0);
    p.dest_chunks_k = static_cast<int>(mx ? qo.dest_K >> 7 : qo.dest_K >> 6);  // a scale chunk spans 64 (NVFP4) or 128 columns
#ifdef SOL_TUNING
    if (const char *e = getenv("SOL_DBG")) p.dbg = static_cast<uint32_t>(atoi(e));
#endif
    auto kern = mx ? (out_mode == kOutBf16    ? gemm_pair_fp4_kernel<kOutBf16, true>
                      : out_mode == kOutQuant ? gemm_pair_fp4_kernel<kOutQuant, true>
                                              : gemm_pair_fp4_kernel<kOutSplit, true>)
                : out_mode == kOutBf16 ? gemm_pair_fp4_kernel<kOutBf16, false>
                : out_mode == kOutQuant ? gemm_pair_fp4_kernel<kOutQuant, false>
                                        : gemm_pair_fp4_kernel<kOutSplit, false>;
    static bool configured[6][64] = {};
    const int slot = (mx ? 3 : 0) + out_mode;
    if (dev->device < 64 && !configured[slot][dev->device]) {
        if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBytes) != cudaSuccess)
            return SOL_ERR_CUDA;
        configured[slot][dev->device] = true;
    }
    p.m_tiles = static_cast<int>(ceil_div(p.M, 2 * kBM));
    p.n_tiles = static_cast<int>(ceil_div(p.N, kBN));
    const int64_t tiles = static_cast<int64_t>(p.m_tiles) * p.n_tiles;
    int max_pairs = dev->sm_count / 2;
#ifdef SOL_TUNING
    if (const char *e = getenv("SOL_PAIRS")) max_pairs = atoi(e);
#endif
    const int pairs = static_cast<int>(tiles < max_pairs ? tiles : max_pairs);
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(static_cast<unsigned>(2 * pairs), 1, 1);
    cfg.blockDim = dim3(kThreadsFp4, 1, 1);
    cfg.dynamicSmemBytes = kSmemBytes;
    cfg.stream = stream;
    cudaLaunchAttribute attr[2];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = 2;
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[1].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 2;
    if (cudaLaunchKernelEx(&cfg, kern, tm_a, tm_b, tm_y, tm_q, tm_sfa, tm_sfb, p) != cudaSuccess) {
        cudaGetLastError();
        return SOL_ERR_CUDA;
    }
    return SOL_OK;
}

}  // namespace

sol_status_t launch_pair256_nvfp4(const void *xq, const void *xsf, const float *xts, const void *wq,
                                  const void *wsf, const float *wts, const void *bias, void *y, int64_t M,
                                  int64_t N, int64_t K, int64_t ldy, cudaStream_t stream, const DeviceInfo *dev) {
    return launch_pair256(kOutBf16, false, xq, xsf, xts, wq, wsf, wts, bias, y, ldy, QuantOut{}, M, N, K, stream, dev);
}

sol_status_t launch_pair256_mxfp4(const void *xq, const void *xsf, const void *wq, const void *wsf, const void *bias,
                                  void *y, int64_t M, int64_t N, int64_t K, int64_t ldy, cudaStream_t stream,
                                  const DeviceInfo *dev) {
    return launch_pair256(kOutBf16, true, xq, xsf, nullptr, wq, wsf, nullptr, bias, y, ldy, QuantOut{}, M, N, K, stream,
                          dev);
}

sol_status_t launch_pair256_mxfp4_quant_out(const void *xq, const void *xsf, const void *wq, const void *wsf,
                                            const void *bias, int act, void *hq, void *hsf, uint32_t *amax_out, int64_t M,
                                            int64_t N, int64_t K, cudaStream_t stream, const DeviceInfo *dev) {
    QuantOut qo;
    qo.act = act;
    qo.hq = hq;
    qo.hsf = hsf;
    qo.amax_out = amax_out;
    qo.dest_K = N;
    return launch_pair256(kOutQuant, true, xq, xsf, nullptr, wq, wsf, nullptr, bias, nullptr, 0, qo, M, N, K, stream, dev);
}

sol_status_t launch_pair256_mxfp4_split_out(const void *xq, const void *xsf, const void *wq, const void *wsf,
                                            const void *bias, void *y_bf16, int64_t ldy, int64_t n_split, int act,
                                            void *hq, void *hsf, int64_t dest_K, int64_t dest_col0, uint32_t *amax_out,
                                            int64_t M, int64_t N, int64_t K, cudaStream_t stream, const DeviceInfo *dev) {
    QuantOut qo;
    qo.act = act;
    qo.hq = hq;
    qo.hsf = hsf;
    qo.amax_out = amax_out;
    qo.n_split = n_split;
    qo.dest_K = dest_K;
    qo.dest_col0 = dest_col0;
    return launch_pair256(kOutSplit, true, xq, xsf, nullptr, wq, wsf, nullptr, bias, y_bf16, ldy, qo, M, N, K, stream, dev);
}

sol_status_t launch_pair256_nvfp4_quant_out(const void *xq, const void *xsf, const float *xts, const void *wq,
                                            const void *wsf, const float *wts, const void *bias, int act,
                                            const float *ts_out, void *hq, void *hsf, uint32_t *amax_out,
                                            int64_t M, int64_t N, int64_t K, cudaStream_t stream,
                                            const DeviceInfo *dev) {
    QuantOut qo;
    qo.act = act;
    qo.ts_out = ts_out;
    qo.hq = hq;
    qo.hsf = hsf;
    qo.amax_out = amax_out;
    qo.dest_K = N;
    return launch_pair256(kOutQuant, false, xq, xsf, xts, wq, wsf, wts, bias, nullptr, 0, qo, M, N, K, stream, dev);
}

sol_status_t launch_pair256_nvfp4_split_out(const void *xq, const void *xsf, const float *xts, const void *wq,
                                            const void *wsf, const float *wts, const void *bias, void *y_bf16,
                                            int64_t ldy, int64_t n_split, int act, const float *ts_out, void *hq,
                                            void *hsf, int64_t dest_K, int64_t dest_col0, uint32_t *amax_out,
                                            int64_t M, int64_t N, int64_t K, cudaStream_t stream,
                                            const DeviceInfo *dev) {
    QuantOut qo;
    qo.act = act;
    qo.ts_out = ts_out;
    qo.hq = hq;
    qo.hsf = hsf;
    qo.amax_out = amax_out;
    qo.n_split = n_split;
    qo.dest_K = dest_K;
    qo.dest_col0 = dest_col0;
    return launch_pair256(kOutSplit, false, xq, xsf, xts, wq, wsf, wts, bias, y_bf16, ldy, qo, M, N, K, stream, dev);
}

}  // namespace gemm
}  // namespace sol

#ifdef SOL_TUNING
extern "C" int sol_debug_trace256(long long *host_out) {
    return cudaMemcpyFromSymbol(host_out, sol::gemm::g_trace, sizeof(sol::gemm::g_trace)) == cudaSuccess ? 0 : 1;
}
#endif

#ifdef SOL_SPAN
extern "C" int sol_debug_span(long long *host_out) {
    return cudaMemcpyFromSymbol(host_out, sol::gemm::g_span, 16) == cudaSuccess ? 0 : 1;
}
#endif
