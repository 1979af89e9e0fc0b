// Persistent, warp-specialised tcgen05 GEMM for sm_100a: Y[M,N] = A[M,K] . B[N,K]^T (+ bias),
// BF16 output, FP32 accumulation in TMEM.  Two instantiations share the skeleton:
//   - BF16 inputs            (tcgen05.mma kind::f16), the stage-2 reference linear;
//   - NVFP4 inputs           (tcgen05.mma kind::mxf4nvf4.block_scale.scale_vec::4X), packed E2M1
//     data with one E4M3 scale per 16 elements along K held in TMEM, the stage-1 rollout linear.
//
// CTA = 6 warps.  Warp 0: TMA producer (one lane).  Warp 1: TMEM owner and MMA issuer (one
// lane).  Warps 2..5: epilogue, one TMEM lane quadrant each: tcgen05.ld -> alpha*acc + bias ->
// BF16 -> swizzled shared memory -> TMA store.  A ring of kStages shared-memory stages feeds
// the tensor core; two accumulator stages in TMEM let the epilogue of tile i overlap the
// main loop of tile i+1.  Each stage holds 128 bytes of K per row (64 BF16 or 256 FP4), i.e.
// four MMA instructions.  Every mbarrier wait is bounded: on expiry the CTA records a code in
// the device status word and leaves through the normal teardown.
#include "gemm_common.cuh"

namespace sol {
namespace gemm {
namespace {

template <Kind kKind, int kBN, int kStages>
struct Cfg {
    static constexpr bool kFp4 = kKind == Kind::kNvfp4;
    static constexpr int kBK = kFp4 ? 256 : 64;                 // elements of K per stage
    static constexpr int kMmaK = kBK / kMmasPerStage;
    static constexpr int kABytes = kBM * kRowBytes;
    static constexpr int kBBytes = kBN * kRowBytes;
    static constexpr int kSfRowChunksB = kFp4 ? (kBN > 128 ? 2 : 1) : 0;  // 128-row scale chunks of B
    static constexpr int kSfaBytes = kFp4 ? 2048 : 0;           // 4 chunks of 512 bytes
    static constexpr int kSfbBytes = kSfRowChunksB * 2048;
    static constexpr int kStageBytes = kABytes + kBBytes + kSfaBytes + kSfbBytes;
    // TMEM columns of one scale-factor buffer: 4 MMAs x (4 columns of A + 4 per 128-row chunk of B).
    // Two buffers, so the copies for k-tile i+1 run while the MMAs of k-tile i read the other one.
    static constexpr int kSfBufCols = kFp4 ? 16 + 16 * kSfRowChunksB : 0;
    static constexpr int kSfBufs = 2;
    static constexpr int kAccStages = (2 * kBN + kSfBufs * kSfBufCols <= kTmemCols) ? 2 : 1;
    static constexpr int kSfCol = kAccStages * kBN;             // first scale-factor column
    static constexpr int kSfWarps = kFp4 ? kMmasPerStage : 0;   // one copy warp per MMA of a stage
    static constexpr int kThreads = 192 + 32 * kSfWarps;
    static constexpr int kEpiBytes = kEpiWarps * 2 * kEpiBufBytes;
    static constexpr int kBarBytes = 256;
    static constexpr int kSmemBytes = kStages * kStageBytes + kEpiBytes + kBarBytes + 1024;
    static_assert(kStageBytes % 1024 == 0, "stage tiles must stay 1024-byte aligned");
    static_assert(kBN % 64 == 0 && kBN >= 64 && kBN <= 256, "tile N");
    static_assert(kSfCol + kSfBufs * kSfBufCols <= kTmemCols, "TMEM budget");
    static_assert(kSmemBytes <= 232448, "shared memory budget");
};

template <Kind kKind, int kBN, int kStages>
__global__ void __launch_bounds__((Cfg<kKind, kBN, kStages>::kThreads), 1)
gemm_kernel(const __grid_constant__ CUtensorMap tm_a, const __grid_constant__ CUtensorMap tm_b,
            const __grid_constant__ CUtensorMap tm_y, const Params p) {
    using C = Cfg<kKind, kBN, kStages>;
    extern __shared__ uint8_t smem_raw[];
    const uint32_t smem_base = (ptx::smem_u32(smem_raw) + 1023u) & ~1023u;
    uint8_t *smem_gen = smem_raw + (smem_base - ptx::smem_u32(smem_raw));

    const uint32_t epi_base = smem_base + kStages * C::kStageBytes;
    const uint32_t bar_base = epi_base + C::kEpiBytes;
    uint8_t *bar_gen = smem_gen + kStages * C::kStageBytes + C::kEpiBytes;
    // barrier block: full[kStages], empty[kStages], acc_full[2], acc_empty[2], sf_ready[2], tmem ptr, abort flag
    auto full_bar = [&](int s) { return bar_base + 8u * s; };
    auto empty_bar = [&](int s) { return bar_base + 8u * (kStages + s); };
    auto acc_full_bar = [&](int s) { return bar_base + 8u * (2 * kStages + s); };
    auto acc_empty_bar = [&](int s) { return bar_base + 8u * (2 * kStages + 2 + s); };
    auto sf_ready_bar = [&](int s) { return bar_base + 8u * (2 * kStages + 4 + s); };
    uint32_t *tmem_ptr_smem = reinterpret_cast<uint32_t *>(bar_gen + 8 * (2 * kStages + 6));
    volatile uint32_t *abort_flag = reinterpret_cast<volatile uint32_t *>(bar_gen + 8 * (2 * kStages + 6) + 4);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int total_tiles = p.m_tiles * p.n_tiles;
    const int k_tiles = (p.K + C::kBK - 1) / C::kBK;

    if (threadIdx.x == 0) {
        for (int s = 0; s < kStages; ++s) {
            ptx::mbar_init(full_bar(s), 1);
            ptx::mbar_init(empty_bar(s), 1);
        }
        for (int s = 0; s < 2; ++s) {
            ptx::mbar_init(acc_full_bar(s), 1);
            ptx::mbar_init(acc_empty_bar(s), kEpiWarps);
            ptx::mbar_init(sf_ready_bar(s), C::kSfWarps > 0 ? C::kSfWarps : 1);
        }
        *abort_flag = 0;
        ptx::fence_mbar_init();
        ptx::prefetch_tmap(&tm_a);
        ptx::prefetch_tmap(&tm_b);
        ptx::prefetch_tmap(&tm_y);
    }
    if (warp == 1) {
        ptx::tmem_alloc(ptx::smem_u32(tmem_ptr_smem), kTmemCols);
        ptx::tmem_relinquish();
    }
    ptx::tc_fence_before_sync();
    __syncthreads();
    ptx::tc_fence_after_sync();
    const uint32_t tmem_base = *tmem_ptr_smem;

    if (warp == 0) {
        // ------------------------------------------------------------ TMA producer
        if (lane == 0) {
            int stage = 0;
            uint32_t phase = 0;
            bool ok = true;
            for (int t = blockIdx.x; ok && t < total_tiles; t += gridDim.x) {
                int mt, nt;
                tile_coords(t, p.m_tiles, p.n_tiles, mt, nt);
                const int m0 = mt * kBM, n0 = nt * kBN;
                for (int kt = 0; kt < k_tiles; ++kt) {
                    if (!wait_bounded(empty_bar(stage), phase ^ 1u, abort_flag, p.status, 0x100u | stage)) {
                        ok = false;
                        break;
                    }
                    const uint32_t sa = smem_base + stage * C::kStageBytes;
                    const uint32_t sb = sa + C::kABytes;
                    uint32_t tx = C::kABytes + C::kBBytes;
                    if (C::kFp4) {
                        const int chunks_k = (p.K + 63) >> 6;
                        const int nchunk = min(4, chunks_k - kt * 4);
                        const int row_chunks_n = (p.N + 127) >> 7;
                        const int rc0 = n0 >> 7;
                        int n_rc = 0;
                        for (int rc = 0; rc < C::kSfRowChunksB; ++rc) n_rc += (rc0 + rc < row_chunks_n);
                        const bool sf_load = !(kTuning && (p.dbg & kDbgNoSfLoad));
                        if (sf_load) tx += static_cast<uint32_t>(nchunk * 512 * (1 + n_rc));
                        ptx::mbar_arrive_expect_tx(full_bar(stage), tx);
                        const uint32_t ssfa = sb + C::kBBytes;
                        const uint32_t ssfb = ssfa + C::kSfaBytes;
                        if (sf_load)
                            ptx::bulk_load_1d(ssfa, p.sfa + (static_cast<int64_t>(mt) * chunks_k + kt * 4) * 512,
                                              nchunk * 512, full_bar(stage));
                        for (int rc = 0; rc < C::kSfRowChunksB; ++rc) {
                            if (sf_load && rc0 + rc < row_chunks_n)
                                ptx::bulk_load_1d(ssfb + rc * 2048,
                                                  p.sfb + (static_cast<int64_t>(rc0 + rc) * chunks_k + kt * 4) * 512,
                                                  nchunk * 512, full_bar(stage));
                        }
                    } else {
                        ptx::mbar_arrive_expect_tx(full_bar(stage), tx);
                    }
                    // inner coordinate in elements of the tensor map (BF16 elements, or bytes of packed FP4)
                    const int kx = C::kFp4 ? kt * kRowBytes : kt * C::kBK;
                    ptx::tma_load_2d(sa, &tm_a, kx, m0, full_bar(stage));
                    ptx::tma_load_2d(sb, &tm_b, kx, n0, full_bar(stage));
                    if (++stage == kStages) {
                        stage = 0;
                        phase ^= 1u;
                    }
                }
            }
        }
        __syncwarp();
    } else if (warp == 1) {
        // ------------------------------------------------------------ MMA issuer
        if (lane == 0) {
            uint32_t idesc;
            if (C::kFp4) {
                idesc = (1u << 7) | (1u << 10) | (static_cast<uint32_t>(kBN >> 3) << 17) |
                        (static_cast<uint32_t>(kBM >> 4) << 24);  // E2M1 x E2M1, UE4M3 scales
            } else {
                idesc = (1u << 4) | (1u << 7) | (1u << 10) | (static_cast<uint32_t>(kBN >> 3) << 17) |
                        (static_cast<uint32_t>(kBM >> 4) << 24);  // FP32 accum, BF16 x BF16, K-major
            }
            int stage = 0;
            uint32_t phase = 0;
            uint32_t gi = 0;  // k-tiles issued so far by this CTA
            bool ok = true;
            int it = 0;
            for (int t = blockIdx.x; ok && t < total_tiles; t += gridDim.x, ++it) {
                int mt, nt;
                tile_coords(t, p.m_tiles, p.n_tiles, mt, nt);
                const int as = it % C::kAccStages;
                const uint32_t acc_parity = static_cast<uint32_t>(it / C::kAccStages) & 1u;
                if (!wait_bounded(acc_empty_bar(as), acc_parity ^ 1u, abort_flag, p.status, 0x200u | as)) break;
                ptx::tc_fence_after_sync();
                const uint32_t d_tmem = tmem_base + as * kBN;
                const uint32_t sfb_shift = C::kFp4 ? static_cast<uint32_t>(((nt * kBN) & 127) >> 5) : 0u;
                for (int kt = 0; kt < k_tiles; ++kt) {
                    if (!wait_bounded(full_bar(stage), phase, abort_flag, p.status, 0x300u | stage)) {
                        ok = false;
                        break;
                    }
                    ptx::tc_fence_after_sync();
                    const uint32_t sa = smem_base + stage * C::kStageBytes;
                    const uint32_t sb = sa + C::kABytes;
                    const uint64_t a_desc = ptx::smem_desc_sw128(sa);
                    const uint64_t b_desc = ptx::smem_desc_sw128(sb);
                    const int k_left = p.K - kt * C::kBK;
                    const int nmma = min(kMmasPerStage, (k_left + C::kMmaK - 1) / C::kMmaK);
                    if (C::kFp4) {
                        // scale factors of this k-tile were copied into TMEM buffer gi&1 by the copy warps
                        const uint32_t sf_buf = gi & 1u;
                        if (!(kTuning && (p.dbg & kDbgNoSfCopy)) &&
                            !wait_bounded(sf_ready_bar(sf_buf), (gi >> 1) & 1u, abort_flag, p.status, 0x500u | sf_buf)) {
                            ok = false;
                            break;
                        }
                        ptx::tc_fence_after_sync();
                        const uint32_t sfa_t = tmem_base + C::kSfCol + sf_buf * C::kSfBufCols;
                        const uint32_t sfb_t = sfa_t + 16 + sfb_shift;
                        for (int j = 0; j < nmma && !(kTuning && (p.dbg & kDbgNoMma)); ++j)
                            ptx::mma_nvfp4(d_tmem, a_desc + 2u * j, b_desc + 2u * j, idesc, sfa_t + 4 * j,
                                           sfb_t + 4 * C::kSfRowChunksB * j, (kt | j) != 0);
                    } else {
                        for (int j = 0; j < nmma && !(kTuning && (p.dbg & kDbgNoMma)); ++j)
                            ptx::mma_bf16(d_tmem, a_desc + 2u * j, b_desc + 2u * j, idesc, (kt | j) != 0);
                    }
                    ptx::tc_commit(empty_bar(stage));  // frees the stage once these MMAs have read it
                    ++gi;
                    if (++stage == kStages) {
                        stage = 0;
                        phase ^= 1u;
                    }
                }
                if (ok) ptx::tc_commit(acc_full_bar(as));
            }
        }
        __syncwarp();
    } else if (warp >= 6) {
        // ------------------------------------------------------------ scale-factor copy warps (NVFP4)
        // tcgen05.cp holds its issuing warp for ~100 cycles, so the copies are spread over four
        // warps (one per MMA of a stage) and kept off the MMA-issuing thread.  Warp j copies the
        // scales of k-block j: one 512-byte chunk of A and one per 128-row chunk of B.
        if (lane == 0 && !(kTuning && (p.dbg & kDbgNoSfCopy))) {
            const int j = warp - 6;
            int stage = 0;
            uint32_t phase = 0;
            uint32_t gi = 0;
            bool ok = true;
            for (int t = blockIdx.x; ok && t < total_tiles; t += gridDim.x) {
                for (int kt = 0; kt < k_tiles; ++kt) {
                    if (!wait_bounded(full_bar(stage), phase, abort_flag, p.status, 0x600u | stage)) {
                        ok = false;
                        break;
                    }
                    if (gi >= 2) {
                        // buffer gi&1 was last read by the MMAs of k-tile gi-2; their commit frees its stage
                        const uint32_t g2 = gi - 2;
                        if (!wait_bounded(empty_bar(g2 % kStages), (g2 / kStages) & 1u, abort_flag, p.status,
                                          0x700u | (g2 % kStages))) {
                            ok = false;
                            break;
                        }
                    }
                    ptx::tc_fence_after_sync();
                    const int k_left = p.K - kt * C::kBK;
                    const int nmma = min(kMmasPerStage, (k_left + C::kMmaK - 1) / C::kMmaK);
                    const uint32_t sf_buf = gi & 1u;
                    if (j < nmma) {
                        const uint32_t ssfa = smem_base + stage * C::kStageBytes + C::kABytes + C::kBBytes;
                        const uint32_t ssfb = ssfa + C::kSfaBytes;
                        const uint32_t sfa_t = tmem_base + C::kSfCol + sf_buf * C::kSfBufCols;
                        ptx::tc_copy_sf(sfa_t + 4 * j, ptx::smem_desc_sf(ssfa + j * 512));
                        for (int rc = 0; rc < C::kSfRowChunksB; ++rc)
                            ptx::tc_copy_sf(sfa_t + 16 + 4 * C::kSfRowChunksB * j + 4 * rc,
                                            ptx::smem_desc_sf(ssfb + rc * 2048 + j * 512));
                    }
                    ptx::tc_commit(sf_ready_bar(sf_buf));
                    ++gi;
                    if (++stage == kStages) {
                        stage = 0;
                        phase ^= 1u;
                    }
                }
            }
        }
        __syncwarp();
    } else {
        // ------------------------------------------------------------ epilogue (warps 2..5)
        const int quad = warp & 3;  // TMEM lanes [32*quad, 32*quad+32) are this warp's
        const uint32_t epi_warp = epi_base + (warp - 2) * 2 * kEpiBufBytes;
        const float alpha = C::kFp4 ? __fmul_rn(__ldcg(p.ts_a), __ldcg(p.ts_b)) : 1.0f;
        int it = 0;
        uint32_t buf = 0;
        for (int t = blockIdx.x; t < total_tiles; t += gridDim.x, ++it) {
            int mt, nt;
            tile_coords(t, p.m_tiles, p.n_tiles, mt, nt);
            const int m0 = mt * kBM + quad * 32, n0 = nt * kBN;
            const int as = it % C::kAccStages;
            const uint32_t acc_parity = static_cast<uint32_t>(it / C::kAccStages) & 1u;
            if (!wait_bounded(acc_full_bar(as), acc_parity, abort_flag, p.status, 0x400u | as)) break;
            ptx::tc_fence_after_sync();
            const uint32_t t_acc = tmem_base + (static_cast<uint32_t>(quad * 32) << 16) + as * kBN;
            if (kTuning && (p.dbg & kDbgNoEpilogue)) {
                ptx::tc_fence_before_sync();
                __syncwarp();
                if (lane == 0) ptx::mbar_arrive(acc_empty_bar(as));
                continue;
            }
            epilogue_tile<kBN>(&tm_y, p, t_acc, m0, n0, alpha, epi_warp, buf, lane,
                               [&] { ptx::mbar_arrive(acc_empty_bar(as)); });
        }
        if (lane == 0) ptx::tma_store_wait_all<0>();
    }

    // ---------------------------------------------------------------- teardown
    if (*abort_flag) __nanosleep(2000000);  // let copies already in flight land before the CTA exits
    ptx::tc_fence_before_sync();
    __syncthreads();
    if (warp == 1) {
        ptx::tc_fence_after_sync();
        ptx::tmem_dealloc(tmem_base, kTmemCols);
    }
}

template <Kind kKind, int kBN, int kStages>
sol_status_t launch(const CUtensorMap &tm_a, const CUtensorMap &tm_b, const CUtensorMap &tm_y, Params p,
                    cudaStream_t stream, const DeviceInfo *dev) {
    using C = Cfg<kKind, kBN, kStages>;
    static bool configured[64] = {};
    auto kern = gemm_kernel<kKind, kBN, kStages>;
    if (dev->device < 64 && !configured[dev->device]) {
        if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, C::kSmemBytes) != cudaSuccess)
            return SOL_ERR_CUDA;
        configured[dev->device] = true;
    }
#ifdef SOL_TUNING
    if (const char *e = getenv("SOL_DBG")) p.dbg = static_cast<uint32_t>(atoi(e));
#endif
    p.m_tiles = static_cast<int>(ceil_div(p.M, kBM));
    p.n_tiles = static_cast<int>(ceil_div(p.N, kBN));
    const int64_t tiles = static_cast<int64_t>(p.m_tiles) * p.n_tiles;
    const int grid = static_cast<int>(tiles < dev->sm_count ? tiles : dev->sm_count);
    kern<<<grid, C::kThreads, C::kSmemBytes, stream>>>(tm_a, tm_b, tm_y, p);
    return launch_status();
}

}  // namespace

sol_status_t launch_single_bf16(const void *x, const void *w, const void *bias, void *y, int64_t M, int64_t N,
                              int64_t K, int64_t ldx, int64_t ldw, int64_t ldy, cudaStream_t stream,
                              const DeviceInfo *dev) {
    constexpr int kBN = 256;
    CUtensorMap tm_a, tm_b, tm_y;
    if (!make_tmap_2d(&tm_a, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, x, K, M, ldx * 2, 64, kBM,
                      CU_TENSOR_MAP_SWIZZLE_128B) ||
        !make_tmap_2d(&tm_b, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, w, K, N, ldw * 2, 64, kBN,
                      CU_TENSOR_MAP_SWIZZLE_128B) ||
        !make_tmap_2d(&tm_y, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, y, N, M, ldy * 2, 64, 32,
                      CU_TENSOR_MAP_SWIZZLE_128B))
        return SOL_ERR_CUDA;
    Params p{};
    p.bias = static_cast<const uint16_t *>(bias);
    p.status = device_status_word();
    p.M = static_cast<int>(M);
    p.N = static_cast<int>(N);
    p.K = static_cast<int>(K);
    return launch<Kind::kBf16, kBN, 4>(tm_a, tm_b, tm_y, p, stream, dev);
}

sol_status_t launch_single_nvfp4(const void *xq, const void *xsf, const float *xts, const void *wq,
                               const void *wsf, const float *wts, const void *bias, void *y, int64_t M,
                               int64_t N, int64_t K, int64_t ldy, cudaStream_t stream,
                               const DeviceInfo *dev) {
    constexpr int kBN = 192;
    CUtensorMap tm_a, tm_b, tm_y;
    if (!make_tmap_2d(&tm_a, CU_TENSOR_MAP_DATA_TYPE_UINT8, 1, xq, K / 2, M, K / 2, 128, kBM,
                      CU_TENSOR_MAP_SWIZZLE_128B) ||
        !make_tmap_2d(&tm_b, CU_TENSOR_MAP_DATA_TYPE_UINT8, 1, wq, K / 2, N, K / 2, 128, kBN,
                      CU_TENSOR_MAP_SWIZZLE_128B) ||
        !make_tmap_2d(&tm_y, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, y, N, M, ldy * 2, 64, 32,
                      CU_TENSOR_MAP_SWIZZLE_128B))
        return SOL_ERR_CUDA;
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
    return launch<Kind::kNvfp4, kBN, 4>(tm_a, tm_b, tm_y, p, stream, dev);
}

}  // namespace gemm

// Pair tiles (two CTAs per MMA) halve the weight-tile traffic per SM; a single 128-row tile is
// enough when the whole problem has at most 128 rows.
sol_status_t launch_gemm_bf16(const void *x, const void *w, const void *bias, void *y, int64_t M, int64_t N,
                              int64_t K, int64_t ldx, int64_t ldw, int64_t ldy, cudaStream_t stream,
                              const DeviceInfo *dev) {
#ifdef SOL_TUNING
    if (getenv("SOL_FORCE_SINGLE")) return gemm::launch_single_bf16(x, w, bias, y, M, N, K, ldx, ldw, ldy, stream, dev);
#endif
    if (M <= 128) return gemm::launch_single_bf16(x, w, bias, y, M, N, K, ldx, ldw, ldy, stream, dev);
    return gemm::launch_pair_bf16(x, w, bias, y, M, N, K, ldx, ldw, ldy, stream, dev);
}

sol_status_t launch_gemm_nvfp4(const void *xq, const void *xsf, const float *xts, const void *wq,
                               const void *wsf, const float *wts, const void *bias, void *y, int64_t M,
                               int64_t N, int64_t K, int64_t ldy, cudaStream_t stream,
                               const DeviceInfo *dev) {
#ifdef SOL_TUNING
    if (getenv("SOL_FORCE_SINGLE"))
        return gemm::launch_single_nvfp4(xq, xsf, xts, wq, wsf, wts, bias, y, M, N, K, ldy, stream, dev);
#endif
    if (M <= 128) return gemm::launch_single_nvfp4(xq, xsf, xts, wq, wsf, wts, bias, y, M, N, K, ldy, stream, dev);
#ifdef SOL_TUNING
    if (getenv("SOL_PAIR192")) return gemm::launch_pair_nvfp4(xq, xsf, xts, wq, wsf, wts, bias, y, M, N, K, ldy, stream, dev);
#endif
    return gemm::launch_pair256_nvfp4(xq, xsf, xts, wq, wsf, wts, bias, y, M, N, K, ldy, stream, dev);
}

}  // namespace sol
