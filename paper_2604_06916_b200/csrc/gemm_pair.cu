// CTA-pair tcgen05 GEMM for sm_100a (tcgen05.mma.cta_group::2): two CTAs of a cluster compute one
// 256 x kBN tile of Y = A . B^T.  Each CTA holds 128 rows of A and half of the B tile in shared
// memory and its 128 x kBN slice of the accumulator in its own TMEM; the even CTA issues the MMAs
// for both.  Halving the B traffic per SM is what lets the FP4 main loop keep up with the L2 -> SM
// path.  No multicast loads are used: each CTA fetches its own tiles, and only the byte counts are
// reported to the even CTA's barrier.
//
// Warps per CTA: 0 = TMA producer, 1 = TMEM owner (+ MMA issuer in the even CTA), 2..5 = epilogue,
// 6..17 = scale-factor copy warps (NVFP4, even CTA only; tcgen05.cp holds its issuing warp for
// ~100 cycles, so each of the twelve copies of a k-tile has its own warp, off the MMA thread),
// 18 = TMA producer of the scale-factor tiles (NVFP4).
// Barriers: full[s] (even CTA; bytes of both CTAs' loads), empty[s] and acc_full[a] (both CTAs,
// signalled by multicast tcgen05.commit), acc_empty[a] (even CTA, 8 epilogue warps arrive),
// sf_ready[b] (even CTA).  All waits are bounded.
#include "gemm_common.cuh"

namespace sol {
namespace gemm {
namespace {

template <Kind kKind, int kBN, int kStages>
struct PairCfg {
    static constexpr bool kFp4 = kKind == Kind::kNvfp4;
    static constexpr int kBK = kFp4 ? 256 : 64;
    static constexpr int kMmaK = kBK / kMmasPerStage;
    static constexpr int kABytes = kBM * kRowBytes;             // this CTA's 128 rows of A
    static constexpr int kBBytes = (kBN / 2) * kRowBytes;       // this CTA's half of the B tile
    static constexpr int kSfRowChunksB = kFp4 ? (kBN > 128 ? 2 : 1) : 0;
    static constexpr int kSfaBytes = kFp4 ? 2048 : 0;
    static constexpr int kSfbBytes = kSfRowChunksB * 2048;      // scales of all kBN rows of B, in each CTA
    static constexpr int kStageBytes = kABytes + kBBytes + kSfaBytes + kSfbBytes;
    static constexpr int kSfBufCols = kFp4 ? 16 + 16 * kSfRowChunksB : 0;
    static constexpr int kSfBufs = 2;
    static constexpr int kAccStages = (2 * kBN + kSfBufs * kSfBufCols <= kTmemCols) ? 2 : 1;
    static constexpr int kSfCol = kAccStages * kBN;
    static constexpr int kSfCopiesPerMma = 1 + kSfRowChunksB;          // one 512-byte chunk of A, one per row chunk of B
    static constexpr int kSfWarps = kFp4 ? kMmasPerStage * kSfCopiesPerMma : 0;  // one tcgen05.cp per warp per k-tile
    static constexpr int kThreads = 192 + (kFp4 ? 32 * (kSfWarps + 1) : 0);  // + one scale-factor TMA warp
    static constexpr int kEpiBytes = kEpiWarps * 2 * kEpiBufBytes;
    static constexpr int kBarBytes = 256;
    static constexpr int kSmemBytes = kStages * kStageBytes + kEpiBytes + kBarBytes + 1024;
    static_assert(kStageBytes % 1024 == 0, "stage tiles must stay 1024-byte aligned");
    static_assert(kBN % 64 == 0 && kBN >= 64 && kBN <= 256, "tile N");
    static_assert(kSfCol + kSfBufs * kSfBufCols <= kTmemCols, "TMEM budget");
    static_assert(kSmemBytes <= 232448, "shared memory budget");
};

template <Kind kKind, int kBN, int kStages>
__global__ void __launch_bounds__((PairCfg<kKind, kBN, kStages>::kThreads), 1)
gemm_pair_kernel(const __grid_constant__ CUtensorMap tm_a, const __grid_constant__ CUtensorMap tm_b,
                 const __grid_constant__ CUtensorMap tm_y, const __grid_constant__ CUtensorMap tm_sfa,
                 const __grid_constant__ CUtensorMap tm_sfb, const Params p) {
    using C = PairCfg<kKind, kBN, kStages>;
    extern __shared__ uint8_t smem_raw[];
    const uint32_t smem_base = (ptx::smem_u32(smem_raw) + 1023u) & ~1023u;
    uint8_t *smem_gen = smem_raw + (smem_base - ptx::smem_u32(smem_raw));

    const uint32_t epi_base = smem_base + kStages * C::kStageBytes;
    const uint32_t bar_base = epi_base + C::kEpiBytes;
    uint8_t *bar_gen = smem_gen + kStages * C::kStageBytes + C::kEpiBytes;
    auto full_bar = [&](int s) { return bar_base + 8u * s; };
    auto empty_bar = [&](int s) { return bar_base + 8u * (kStages + s); };
    auto acc_full_bar = [&](int s) { return bar_base + 8u * (2 * kStages + s); };
    auto acc_empty_bar = [&](int s) { return bar_base + 8u * (2 * kStages + 2 + s); };
    auto sf_ready_bar = [&](int s) { return bar_base + 8u * (2 * kStages + 4 + s); };
    uint32_t *tmem_ptr_smem = reinterpret_cast<uint32_t *>(bar_gen + 8 * (2 * kStages + 6));
    volatile uint32_t *abort_flag = reinterpret_cast<volatile uint32_t *>(bar_gen + 8 * (2 * kStages + 6) + 4);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const uint32_t rank = ptx::cluster_ctarank();  // 0 = even CTA (issues the MMAs), 1 = its partner
    const bool leader = rank == 0;
    const int pair = blockIdx.x >> 1, num_pairs = gridDim.x >> 1;
    const int total_tiles = p.m_tiles * p.n_tiles;
    const int k_tiles = (p.K + C::kBK - 1) / C::kBK;

    if (threadIdx.x == 0) {
        for (int s = 0; s < kStages; ++s) {
            ptx::mbar_init(full_bar(s), 1);
            ptx::mbar_init(empty_bar(s), 1);
        }
        for (int s = 0; s < 2; ++s) {
            ptx::mbar_init(acc_full_bar(s), 1);
            ptx::mbar_init(acc_empty_bar(s), 2 * kEpiWarps);
            ptx::mbar_init(sf_ready_bar(s), C::kSfWarps > 0 ? C::kSfWarps : 1);
        }
        *abort_flag = 0;
        ptx::fence_mbar_init();
        ptx::prefetch_tmap(&tm_a);
        ptx::prefetch_tmap(&tm_b);
        ptx::prefetch_tmap(&tm_y);
        if (C::kFp4) {
            ptx::prefetch_tmap(&tm_sfa);
            ptx::prefetch_tmap(&tm_sfb);
        }
    }
    if (warp == 1) {
        ptx::tmem_alloc_pair(ptx::smem_u32(tmem_ptr_smem), kTmemCols);
        ptx::tmem_relinquish_pair();
    }
    ptx::tc_fence_before_sync();
    __syncthreads();
    ptx::cluster_sync();  // both CTAs' barriers and TMEM exist before anything crosses the pair
    ptx::tc_fence_after_sync();
    const uint32_t tmem_base = *tmem_ptr_smem;
    ptx::grid_dependency_wait();  // set-up above overlaps the previous kernel; its results are read below

    if (warp == 0) {
        // ------------------------------------------------------------ TMA producer: A and B tiles (both CTAs)
        // The whole warp runs the loop so that addresses and coordinates stay warp-uniform (they are
        // then handed to the copy engine without per-instruction register shuffling); one elected lane
        // issues.
        {
            const bool elected = ptx::elect_one();
            const uint32_t full0 = ptx::map_to_cta(full_bar(0), 0);  // the even CTA's barriers
            const bool sf_load = C::kFp4 && !(kTuning && (p.dbg & kDbgNoSfLoad));
            const uint32_t tx = 2u * (C::kStageBytes - (sf_load ? 0 : C::kSfaBytes + C::kSfbBytes));
            const bool trace = kTuning && (p.dbg & kDbgTrace);
            int stage = 0;
            uint32_t phase = 0;
            bool ok = !loads_held(p.status);
            [[maybe_unused]] int pgi = 0;
            for (int t = pair; ok && t < total_tiles; t += num_pairs) {
                int mt, nt;
                tile_coords(t, p.m_tiles, p.n_tiles, mt, nt);
                const int m0 = mt * 2 * kBM + static_cast<int>(rank) * kBM;
                const int nb0 = nt * kBN + static_cast<int>(rank) * (kBN / 2);
                int kx = 0;
                for (int kt = 0; kt < k_tiles; ++kt, kx += C::kFp4 ? kRowBytes : C::kBK) {
                    if (!wait_bounded(empty_bar(stage), phase ^ 1u, abort_flag, p.status, 0x100u | stage)) {
                        ok = false;
                        break;
                    }
                    if (trace) SOL_TRACE(leader ? 0 : 4, pgi);
                    const uint32_t sa = smem_base + stage * C::kStageBytes;
                    if (elected) {
                        if (leader) ptx::mbar_arrive_expect_tx(full_bar(stage), tx);
                        ptx::tma_load_2d_pair(sa, &tm_a, kx, m0, full0 + 8u * stage);
                        ptx::tma_load_2d_pair(sa + C::kABytes, &tm_b, kx, nb0, full0 + 8u * stage);
                    }
                    if (trace) SOL_TRACE(leader ? 1 : 5, pgi);
                    ++pgi;
                    if (++stage == kStages) {
                        stage = 0;
                        phase ^= 1u;
                    }
                }
            }
        }
        __syncwarp();
    } else if (warp == 6 + C::kSfWarps) {
        // ------------------------------------------------------------ TMA producer: scale factors (NVFP4, both CTAs)
        // Each tensor-copy instruction costs its issuing thread tens of cycles, so the scale tiles get
        // their own thread.  The byte count was announced by the A/B producer of the even CTA.
        if (!(kTuning && (p.dbg & kDbgNoSfLoad))) {
            const bool elected = ptx::elect_one();
            const uint32_t full0 = ptx::map_to_cta(full_bar(0), 0);
            int stage = 0;
            uint32_t phase = 0;
            bool ok = true;
            for (int t = pair; ok && t < total_tiles; t += num_pairs) {
                int mt, nt;
                tile_coords(t, p.m_tiles, p.n_tiles, mt, nt);
                const int rca = mt * 2 + static_cast<int>(rank);  // 128-row chunk of A owned by this CTA
                const int rcb = (nt * kBN) >> 7;                   // first 128-row chunk of B the tile touches
                for (int kt = 0; kt < k_tiles; ++kt) {
                    if (!wait_bounded(empty_bar(stage), phase ^ 1u, abort_flag, p.status, 0x800u | stage)) {
                        ok = false;
                        break;
                    }
                    const uint32_t ssfa = smem_base + stage * C::kStageBytes + C::kABytes + C::kBBytes;
                    if (elected) {
                        ptx::tma_load_3d_pair(ssfa, &tm_sfa, 0, kt * 4, rca, full0 + 8u * stage);
                        ptx::tma_load_3d_pair(ssfa + C::kSfaBytes, &tm_sfb, 0, kt * 4, rcb, full0 + 8u * stage);
                    }
                    if (++stage == kStages) {
                        stage = 0;
                        phase ^= 1u;
                    }
                }
            }
        }
        __syncwarp();
    } else if (warp == 1) {
        // ------------------------------------------------------------ MMA issuer (even CTA)
        if (leader) {
            const bool elected = ptx::elect_one();
            uint32_t idesc;
            if (C::kFp4) {
                idesc = (1u << 7) | (1u << 10) | (static_cast<uint32_t>(kBN >> 3) << 17) |
                        (static_cast<uint32_t>((2 * kBM) >> 4) << 24);
            } else {
                idesc = (1u << 4) | (1u << 7) | (1u << 10) | (static_cast<uint32_t>(kBN >> 3) << 17) |
                        (static_cast<uint32_t>((2 * kBM) >> 4) << 24);
            }
            // Everything that does not depend on the k-tile is computed once: the issue loop below is a
            // single thread's instruction stream, and its latency is what bounds the tensor pipe.
            const uint64_t desc_hi = ptx::smem_desc_sw128(0);           // swizzle / stride / version fields
            const uint32_t a_lo0 = (smem_base & 0x3FFFFu) >> 4;         // start-address field of stage 0's A tile
            const uint32_t b_lo0 = ((smem_base + C::kABytes) & 0x3FFFFu) >> 4;
            constexpr uint32_t kStageLo = C::kStageBytes >> 4;
            const uint32_t sf_t0 = tmem_base + C::kSfCol;
            const bool trace = kTuning && (p.dbg & kDbgTrace);
            const bool no_sf_wait = kTuning && (p.dbg & kDbgNoSfCopy);
            const bool no_mma = kTuning && (p.dbg & kDbgNoMma);
            const int tail_mmas = (p.K - (k_tiles - 1) * C::kBK + C::kMmaK - 1) / C::kMmaK;  // MMAs of the last k-tile
            int stage = 0;
            uint32_t phase = 0;
            uint32_t gi = 0;
            bool ok = true;
            int it = 0;
            for (int t = pair; ok && t < total_tiles; t += num_pairs, ++it) {
                const int as = it % C::kAccStages;
                const uint32_t acc_parity = static_cast<uint32_t>(it / C::kAccStages) & 1u;
                if (!wait_bounded(acc_empty_bar(as), acc_parity ^ 1u, abort_flag, p.status, 0x200u | as)) break;
                ptx::tc_fence_after_sync();
                const uint32_t d_tmem = tmem_base + as * kBN;
                uint32_t sfb_shift = 0;
                if (C::kFp4) {
                    int mt, nt;
                    tile_coords(t, p.m_tiles, p.n_tiles, mt, nt);
                    sfb_shift = static_cast<uint32_t>(((nt * kBN) & 127) >> 5);
                }
                for (int kt = 0; kt < k_tiles; ++kt) {
                    const uint32_t sf_buf = gi & 1u;
                    if (C::kFp4 && !no_sf_wait) {
                        // The copy warps waited for this stage's loads before copying its scale factors, so
                        // their barrier also covers the A/B tiles: one wait per k-tile on this thread.
                        if (!wait_bounded(sf_ready_bar(sf_buf), (gi >> 1) & 1u, abort_flag, p.status, 0x500u | sf_buf)) {
                            ok = false;
                            break;
                        }
                    } else if (!wait_bounded(full_bar(stage), phase, abort_flag, p.status, 0x300u | stage)) {
                        ok = false;
                        break;
                    }
                    ptx::tc_fence_after_sync();
                    if (trace) SOL_TRACE(6, gi);
                    const uint64_t a_desc = desc_hi | (a_lo0 + static_cast<uint32_t>(stage) * kStageLo);
                    const uint64_t b_desc = desc_hi | (b_lo0 + static_cast<uint32_t>(stage) * kStageLo);
                    const uint32_t sfa_t = sf_t0 + sf_buf * C::kSfBufCols;
                    const uint32_t sfb_t = sfa_t + 16 + sfb_shift;
                    const uint32_t acc0 = kt != 0;
                    if (elected && !no_mma) {
                        if (kt + 1 < k_tiles || tail_mmas == kMmasPerStage) {
                            if (C::kFp4) {
                                ptx::mma_nvfp4_pair(d_tmem, a_desc, b_desc, idesc, sfa_t, sfb_t, acc0);
                                ptx::mma_nvfp4_pair(d_tmem, a_desc + 2, b_desc + 2, idesc, sfa_t + 4,
                                                    sfb_t + 4 * C::kSfRowChunksB, 1);
                                ptx::mma_nvfp4_pair(d_tmem, a_desc + 4, b_desc + 4, idesc, sfa_t + 8,
                                                    sfb_t + 8 * C::kSfRowChunksB, 1);
                                ptx::mma_nvfp4_pair(d_tmem, a_desc + 6, b_desc + 6, idesc, sfa_t + 12,
                                                    sfb_t + 12 * C::kSfRowChunksB, 1);
                            } else {
                                ptx::mma_bf16_pair(d_tmem, a_desc, b_desc, idesc, acc0);
                                ptx::mma_bf16_pair(d_tmem, a_desc + 2, b_desc + 2, idesc, 1);
                                ptx::mma_bf16_pair(d_tmem, a_desc + 4, b_desc + 4, idesc, 1);
                                ptx::mma_bf16_pair(d_tmem, a_desc + 6, b_desc + 6, idesc, 1);
                            }
                        } else {
                            for (int j = 0; j < tail_mmas; ++j) {  // ragged K: fewer than four 32-byte slices are valid
                                if (C::kFp4)
                                    ptx::mma_nvfp4_pair(d_tmem, a_desc + 2u * j, b_desc + 2u * j, idesc, sfa_t + 4 * j,
                                                        sfb_t + 4 * C::kSfRowChunksB * j, (kt | j) != 0);
                                else
                                    ptx::mma_bf16_pair(d_tmem, a_desc + 2u * j, b_desc + 2u * j, idesc, (kt | j) != 0);
                            }
                        }
                    }
                    if (elected) ptx::tc_commit_pair_mcast(empty_bar(stage), 3);  // frees the stage in both CTAs
                    if (trace) SOL_TRACE(3, gi);
                    ++gi;
                    if (++stage == kStages) {
                        stage = 0;
                        phase ^= 1u;
                    }
                }
                if (ok && elected) ptx::tc_commit_pair_mcast(acc_full_bar(as), 3);
            }
        }
        __syncwarp();
    } else if (warp >= 6) {
        // ------------------------------------------------------------ scale-factor copy warps 6..9 (even CTA)
        if (leader && !(kTuning && (p.dbg & kDbgNoSfCopy))) {
            const bool elected = ptx::elect_one();
            // warp w copies part (w % copies-per-MMA) of MMA j = w / copies-per-MMA: part 0 = scales of A,
            // part 1.. = scales of the B tile's 128-row chunks
            const int j = (warp - 6) / C::kSfCopiesPerMma, part = (warp - 6) % C::kSfCopiesPerMma;
            int stage = 0;
            uint32_t phase = 0;
            uint32_t gi = 0;
            bool ok = true;
            for (int t = pair; ok && t < total_tiles; t += num_pairs) {
                for (int kt = 0; kt < k_tiles; ++kt) {
                    if (!wait_bounded(full_bar(stage), phase, abort_flag, p.status, 0x600u | stage)) {
                        ok = false;
                        break;
                    }
                    if (gi >= 2) {
                        const uint32_t g2 = gi - 2;  // last k-tile whose MMAs read this TMEM buffer
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
                    if (elected) {
                        if (j < nmma) {
                            const uint32_t ssf = smem_base + stage * C::kStageBytes + C::kABytes + C::kBBytes;
                            const uint32_t sf_t = tmem_base + C::kSfCol + sf_buf * C::kSfBufCols;
                            const uint32_t src = part == 0 ? ssf + j * 512 : ssf + C::kSfaBytes + (part - 1) * 2048 + j * 512;
                            const uint32_t dst = part == 0 ? sf_t + 4 * j
                                                           : sf_t + 16 + 4 * C::kSfRowChunksB * j + 4 * (part - 1);
                            ptx::tc_copy_sf_pair(dst, ptx::smem_desc_sf(src));
                        }
                        ptx::tc_commit_pair(sf_ready_bar(sf_buf));
                    }
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
        // ------------------------------------------------------------ epilogue (warps 2..5, both CTAs)
        const int quad = warp & 3;
        const uint32_t epi_warp = epi_base + (warp - 2) * 2 * kEpiBufBytes;
        const float alpha = C::kFp4 ? __fmul_rn(__ldcg(p.ts_a), __ldcg(p.ts_b)) : 1.0f;
        int it = 0;
        uint32_t buf = 0;
        for (int t = pair; t < total_tiles; t += num_pairs, ++it) {
            int mt, nt;
            tile_coords(t, p.m_tiles, p.n_tiles, mt, nt);
            const int m0 = mt * 2 * kBM + static_cast<int>(rank) * kBM + quad * 32, n0 = nt * kBN;
            const int as = it % C::kAccStages;
            const uint32_t acc_parity = static_cast<uint32_t>(it / C::kAccStages) & 1u;
            if (!wait_bounded(acc_full_bar(as), acc_parity, abort_flag, p.status, 0x400u | as)) break;
            ptx::tc_fence_after_sync();
            const uint32_t t_acc = tmem_base + (static_cast<uint32_t>(quad * 32) << 16) + as * kBN;
            const uint32_t release_bar = ptx::map_to_cta(acc_empty_bar(as), 0);
            if (kTuning && (p.dbg & kDbgNoEpilogue)) {
                ptx::tc_fence_before_sync();
                __syncwarp();
                if (lane == 0) ptx::mbar_arrive_cluster(release_bar);
                continue;
            }
            epilogue_tile<kBN>(&tm_y, p, t_acc, m0, n0, alpha, epi_warp, buf, lane,
                               [&] { ptx::mbar_arrive_cluster(release_bar); });
        }
        if (lane == 0) ptx::tma_store_wait_all<0>();
    }

    // ---------------------------------------------------------------- teardown
    if (*abort_flag) __nanosleep(2000000);
    ptx::tc_fence_before_sync();
    __syncthreads();
    ptx::cluster_sync();  // neither CTA frees TMEM or exits while its partner may still touch it
    if (warp == 1) {
        ptx::tc_fence_after_sync();
        ptx::tmem_dealloc_pair(tmem_base, kTmemCols);
    }
}

template <Kind kKind, int kBN, int kStages>
sol_status_t launch_pair(const CUtensorMap &tm_a, const CUtensorMap &tm_b, const CUtensorMap &tm_y,
                         const CUtensorMap &tm_sfa, const CUtensorMap &tm_sfb, Params p, cudaStream_t stream,
                         const DeviceInfo *dev) {
    using C = PairCfg<kKind, kBN, kStages>;
    static bool configured[64] = {};
    auto kern = gemm_pair_kernel<kKind, kBN, kStages>;
    if (dev->device < 64 && !configured[dev->device]) {
        if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, C::kSmemBytes) != cudaSuccess)
            return SOL_ERR_CUDA;
        configured[dev->device] = true;
    }
#ifdef SOL_TUNING
    if (const char *e = getenv("SOL_DBG")) p.dbg = static_cast<uint32_t>(atoi(e));
#endif
    p.m_tiles = static_cast<int>(ceil_div(p.M, 2 * kBM));
    p.n_tiles = static_cast<int>(ceil_div(p.N, kBN));
    const int64_t tiles = static_cast<int64_t>(p.m_tiles) * p.n_tiles;
    const int max_pairs = dev->sm_count / 2;
    const int pairs = static_cast<int>(tiles < max_pairs ? tiles : max_pairs);
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(static_cast<unsigned>(2 * pairs), 1, 1);
    cfg.blockDim = dim3(C::kThreads, 1, 1);
    cfg.dynamicSmemBytes = C::kSmemBytes;
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
    if (cudaLaunchKernelEx(&cfg, kern, tm_a, tm_b, tm_y, tm_sfa, tm_sfb, p) != cudaSuccess) {
        cudaGetLastError();
        return SOL_ERR_CUDA;
    }
    return SOL_OK;
}

}  // namespace

sol_status_t launch_pair_bf16(const void *x, const void *w, const void *bias, void *y, int64_t M, int64_t N,
                              int64_t K, int64_t ldx, int64_t ldw, int64_t ldy, cudaStream_t stream,
                              const DeviceInfo *dev) {
    constexpr int kBN = 256;
    CUtensorMap tm_a, tm_b, tm_y;
    if (!make_tmap_2d(&tm_a, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, x, K, M, ldx * 2, 64, kBM,
                      CU_TENSOR_MAP_SWIZZLE_128B) ||
        !make_tmap_2d(&tm_b, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, w, K, N, ldw * 2, 64, kBN / 2,
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
    return launch_pair<Kind::kBf16, kBN, 6>(tm_a, tm_b, tm_y, tm_a, tm_a, p, stream, dev);
}

#ifdef SOL_TUNING  // the 256 x 192 NVFP4 pair tile is kept for A/B timing only; the product uses gemm_pair_fp4.cu
sol_status_t launch_pair_nvfp4(const void *xq, const void *xsf, const float *xts, const void *wq,
                               const void *wsf, const float *wts, const void *bias, void *y, int64_t M,
                               int64_t N, int64_t K, int64_t ldy, cudaStream_t stream, const DeviceInfo *dev) {
    constexpr int kBN = 192;
    const uint64_t chunks_k = static_cast<uint64_t>(ceil_div(K, 64));
    CUtensorMap tm_a, tm_b, tm_y, tm_sfa, tm_sfb;
    if (!make_tmap_2d(&tm_a, CU_TENSOR_MAP_DATA_TYPE_UINT8, 1, xq, K / 2, M, K / 2, 128, kBM,
                      CU_TENSOR_MAP_SWIZZLE_128B) ||
        !make_tmap_2d(&tm_b, CU_TENSOR_MAP_DATA_TYPE_UINT8, 1, wq, K / 2, N, K / 2, 128, kBN / 2,
                      CU_TENSOR_MAP_SWIZZLE_128B) ||
        !make_tmap_2d(&tm_y, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, y, N, M, ldy * 2, 64, 32,
                      CU_TENSOR_MAP_SWIZZLE_128B) ||
        // scale buffers as [128-row chunk][k chunk][128 x u32]: a box is 4 k-chunks of 1 (A) or 2 (B) row chunks
        !make_tmap_sf(&tm_sfa, xsf, chunks_k, static_cast<uint64_t>(ceil_div(M, 128)), 1) ||
        !make_tmap_sf(&tm_sfb, wsf, chunks_k, static_cast<uint64_t>(ceil_div(N, 128)), kBN > 128 ? 2 : 1))
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
#ifdef SOL_TUNING
    if (const char *e = getenv("SOL_PAIR_STAGES")) {
        const int st = atoi(e);
        if (st == 3) return launch_pair<Kind::kNvfp4, kBN, 3>(tm_a, tm_b, tm_y, tm_sfa, tm_sfb, p, stream, dev);
        if (st == 4) return launch_pair<Kind::kNvfp4, kBN, 4>(tm_a, tm_b, tm_y, tm_sfa, tm_sfb, p, stream, dev);
    }
#endif
    return launch_pair<Kind::kNvfp4, kBN, 5>(tm_a, tm_b, tm_y, tm_sfa, tm_sfb, p, stream, dev);
}
#endif

}  // namespace gemm
}  // namespace sol

#ifdef SOL_TUNING
extern "C" int sol_debug_trace(long long *host_out) {
    return cudaMemcpyFromSymbol(host_out, sol::gemm::g_trace, sizeof(sol::gemm::g_trace)) == cudaSuccess ? 0 : 1;
}
#endif
