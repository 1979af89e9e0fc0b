// Scaled-dot-product attention of a DiT block (BF16 in and out, head dimension 128, no mask):
//     O = softmax(Q K^T / sqrt(128)) V   per batch element and head.
// The linear layers around it run in NVFP4; attention itself stays in BF16 in both the FP4 and the
// BF16 path of the method, so this kernel is what a whole-block forward needs besides the linears.
//
// One CTA per 256 query rows of one (batch, head), one CTA per SM: two query tiles of 128 rows, each
// with its own softmax warpgroup, share the K and V tiles, which stream through two-stage rings (a
// tile is requested more than a whole tile period before it is used: loads take ~2 500 cycles here).
// Per 128-key tile j and query tile t:
//     S_t = Q_t K_j^T          tcgen05.mma kind::f16, 128 x 128 x 128, accumulator in TMEM
//     softmax                  one thread per query row (= TMEM lane): tcgen05.ld of the row, running
//                              max m and sum l (online softmax), p = exp2(s c - m); P goes back into
//                              the columns S occupied, as packed BF16 pairs (tcgen05.st)
//     O_t = alpha O_t + P V_j  O rescaled in TMEM by the row's alpha when its max moved (tcgen05.ld /
//                              st), then tcgen05.mma with A = P from TMEM and V as an MN-major
//                              shared-memory operand (V is [kv][d])
// The MMA thread alternates between the two query tiles (P_0 V, next S_0, P_1 V, next S_1), so the
// tensor pipe works for one tile while the other is in its softmax.  TMEM: S_t/P_t and O_t, 128
// columns each.  The epilogue divides by l and leaves through TMA stores (staged where Q_t was).
//
// Warps: 0 = TMA producer, 1 = TMEM owner and MMA issuer, 2..5 and 6..9 = softmax / epilogue of query
// tile 0 and 1 (one warp per TMEM lane quadrant).  Every mbarrier wait is bounded.
#include "gemm_common.cuh"
#include "quant_math.cuh"
#include "sol_internal.h"

namespace sol {
namespace attn {
namespace {

using gemm::wait_bounded;

constexpr int kBQ = 128;                // query rows per query tile
constexpr int kQTiles = 2;              // query tiles per CTA
constexpr int kBKV = 128;               // keys per tile
constexpr int kBox = 128 * 128;         // bytes of a [128 rows][64 BF16] box
constexpr int kStages = 2;              // K ring and V ring
constexpr int kThreads = 32 * (2 + 4 * kQTiles);
constexpr float kLazyLog2 = 8.0f;       // slack of the softmax reference maximum, in powers of two
constexpr int smem_bytes(int head_dim) { return (kQTiles + 2 * kStages) * (head_dim / 64) * kBox + 256; }
constexpr uint32_t kTmemCols = 512;
constexpr uint32_t kColS = 0, kColO = 128, kColTile = 256;   // per query tile; P overwrites columns [0, 64) of S
static_assert(smem_bytes(128) <= 232448, "shared memory budget");

#ifdef SOL_TUNING
__device__ long long g_attn_trace[12][64];
#define ATTN_TRACE(type, idx) do { if ((blockIdx.x | blockIdx.y | blockIdx.z) == 0 && (idx) < 64 && (threadIdx.x & 31) == 0) g_attn_trace[type][idx] = clock64(); } while (0)
#else
#define ATTN_TRACE(type, idx) do { } while (0)
#endif

struct Params {
    int seq_q;             // query rows and keys of the joint sequence (stream a first, then stream b)
    int seq_kv;
    int q_split;           // rows / keys that come from stream a (0: one stream); multiples of 256 and 128
    int kv_split;
    float scale_log2;      // log2(e) / sqrt(d)
    uint32_t *status;
    // quantized output (kQuantOut): the rows of all samples stacked, [batch * seq_q, dest_K] in NVFP4
    uint8_t *q_dest;       // packed nibbles, dest_K / 2 bytes per row
    uint8_t *sf_dest;      // chunked scale layout of a [batch * seq_q, dest_K] tensor
    const float *ts_out;   // tensor scale of the destination (caller supplied)
    uint32_t *amax_out;    // nullable: running max |h| as FP32 bits
    int dest_pitch;        // dest_K / 2
    int dest_col0;         // first destination column of head 0
    int dest_chunks_k;     // dest_K / 64
};

__device__ __forceinline__ float ex2(float x) {
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}
__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi) {
    uint32_t r;
    asm("cvt.rn.bf16x2.f32 %0, %1, %2;" : "=r"(r) : "f"(hi), "f"(lo));
    return r;
}
__device__ __forceinline__ void sts128(uint32_t addr, uint32_t a, uint32_t b, uint32_t c, uint32_t d) {
    asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(addr), "r"(a), "r"(b), "r"(c), "r"(d) : "memory");
}

// kD: head dimension, 64 or 128 (a tile of kD columns is kD / 64 boxes of [128 rows][64 BF16]).
// kQuantOut: the output leaves as the next linear's NVFP4 activations (h = bf16(O / l), then the
// quantizer's FP32 sequence per 16 columns) instead of BF16 -- one stream only.
template <int kD, bool kQuantOut>
__global__ void __launch_bounds__(kThreads, 1)
attention_kernel(const __grid_constant__ CUtensorMap tm_qa, const __grid_constant__ CUtensorMap tm_ka,
                 const __grid_constant__ CUtensorMap tm_va, const __grid_constant__ CUtensorMap tm_oa,
                 const __grid_constant__ CUtensorMap tm_qb, const __grid_constant__ CUtensorMap tm_kb,
                 const __grid_constant__ CUtensorMap tm_vb, const __grid_constant__ CUtensorMap tm_ob, const Params p) {
    constexpr int kBoxes = kD / 64;
    constexpr int kTile = kBoxes * kBox;    // bytes of a [128][kD] BF16 tile
    extern __shared__ __align__(1024) uint8_t smem_raw[];
    const uint32_t smem_base = ptx::smem_u32(smem_raw);
    if (smem_base & 1023u) {  // the swizzled operand layout needs 1024-byte alignment
        if (threadIdx.x == 0) atomicExch(p.status, 0xB00u);
        return;
    }
    const uint32_t sQ = smem_base;                        // kQTiles tiles; later the output staging buffers
    const uint32_t sK = sQ + kQTiles * kTile;             // kStages tiles
    const uint32_t sV = sK + kStages * kTile;
    const uint32_t bar_base = sV + kStages * kTile;
    uint8_t *bar_gen = smem_raw + (bar_base - smem_base);
    auto bar = [&](int i) { return bar_base + 8u * i; };
    // K / V rings: [stage]; S, P, PV-done: [query tile]
    constexpr int kQFull = 0, kKFull = 1, kKEmpty = 3, kVFull = 5, kVEmpty = 7, kSFull = 9, kPFull = 11, kPvDone = 13,
                  kNumBars = 15;
    uint32_t *tmem_ptr_smem = reinterpret_cast<uint32_t *>(bar_gen + 8 * kNumBars);
    volatile uint32_t *abort_flag = reinterpret_cast<volatile uint32_t *>(bar_gen + 8 * kNumBars + 4);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int q0_joint = blockIdx.x * (kQTiles * kBQ), head = blockIdx.y, batch = blockIdx.z;
    const int n_tiles = (p.seq_kv + kBKV - 1) / kBKV;
    // the CTA's queries come from one stream (the split is a multiple of the CTA's 256 rows)
    const bool q_in_a = q0_joint < p.q_split;
    const CUtensorMap *tm_q = q_in_a ? &tm_qa : &tm_qb;
    const CUtensorMap *tm_o = q_in_a ? &tm_oa : &tm_ob;
    const int q0 = q_in_a ? q0_joint : q0_joint - p.q_split;                 // row within its stream
    const int q_rows = q_in_a ? p.q_split : p.seq_q - p.q_split;             // rows of that stream

    if (threadIdx.x == 0) {
        for (int i = 0; i < kNumBars; ++i) ptx::mbar_init(bar(i), (i == kPFull || i == kPFull + 1) ? 4 : 1);
        *abort_flag = 0;
        ptx::fence_mbar_init();
        ptx::prefetch_tmap(tm_q);
        ptx::prefetch_tmap(tm_o);
        ptx::prefetch_tmap(&tm_kb);
        ptx::prefetch_tmap(&tm_vb);
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
        if (ptx::elect_one()) {
            const int x0 = head * kD;
            ptx::mbar_arrive_expect_tx(bar(kQFull), kQTiles * kTile);
#pragma unroll
            for (int t = 0; t < kQTiles; ++t) {
#pragma unroll
                for (int bx = 0; bx < kBoxes; ++bx)
                    ptx::tma_load_3d(sQ + t * kTile + bx * kBox, tm_q, x0 + 64 * bx, q0 + t * kBQ, batch, bar(kQFull));
            }
            for (int j = 0; j < n_tiles; ++j) {
                const int st = j & 1;
                const uint32_t par = static_cast<uint32_t>(j >> 1) & 1u;
                if (!wait_bounded(bar(kKEmpty + st), par ^ 1u, abort_flag, p.status, 0xB10u | st)) break;
                ATTN_TRACE(10, j);
                ptx::mbar_arrive_expect_tx(bar(kKFull + st), kTile);
                // key tile j of the joint sequence: stream a up to the split (a multiple of the tile), then stream b
                const bool kv_in_a = j * kBKV < p.kv_split;
                const int kv0 = kv_in_a ? j * kBKV : j * kBKV - p.kv_split;
                const CUtensorMap *tm_k = kv_in_a ? &tm_ka : &tm_kb;
                const CUtensorMap *tm_v = kv_in_a ? &tm_va : &tm_vb;
#pragma unroll
                for (int bx = 0; bx < kBoxes; ++bx)
                    ptx::tma_load_3d(sK + st * kTile + bx * kBox, tm_k, x0 + 64 * bx, kv0, batch, bar(kKFull + st));
                if (!wait_bounded(bar(kVEmpty + st), par ^ 1u, abort_flag, p.status, 0xB20u | st)) break;
                ATTN_TRACE(11, j);
                ptx::mbar_arrive_expect_tx(bar(kVFull + st), kTile);
#pragma unroll
                for (int bx = 0; bx < kBoxes; ++bx)
                    ptx::tma_load_3d(sV + st * kTile + bx * kBox, tm_v, x0 + 64 * bx, kv0, batch, bar(kVFull + st));
            }
        }
        __syncwarp();
    } else if (warp == 1) {
        // ------------------------------------------------------------ MMA issuer
        if (ptx::elect_one()) {
            // BF16 x BF16 -> FP32, M = 128; scores N = 128 keys, output N = kD with B MN-major (bit 16: V is [kv][d])
            const uint32_t idesc_base = (1u << 4) | (1u << 7) | (1u << 10) | (static_cast<uint32_t>(128 >> 4) << 24);
            const uint32_t idesc_qk = idesc_base | (static_cast<uint32_t>(kBKV >> 3) << 17);
            const uint32_t idesc_pv = idesc_base | (static_cast<uint32_t>(kD >> 3) << 17) | (1u << 16);
            auto issue_qk = [&](int t, int st) {  // S_t = Q_t K^T, 16 elements of d per instruction
#pragma unroll
                for (int i = 0; i < kD / 16; ++i) {
                    const uint64_t a = ptx::smem_desc_sw128(sQ + t * kTile + (i >> 2) * kBox) + 2u * (i & 3);
                    const uint64_t b = ptx::smem_desc_sw128(sK + st * kTile + (i >> 2) * kBox) + 2u * (i & 3);
                    ptx::mma_bf16(tmem_base + t * kColTile + kColS, a, b, idesc_qk, i > 0);
                }
                ptx::tc_commit(bar(kSFull + t));   // also: every earlier MMA of this tile has completed
            };
            auto issue_pv = [&](int t, int st, bool acc) {  // O_t += P_t V, 16 keys (8 columns of packed P) per instruction
#pragma unroll
                for (int i = 0; i < 8; ++i) {
                    const uint64_t b = ptx::smem_desc_sw128_mn(sV + st * kTile + i * 2048, kBox, 1024);
                    ptx::mma_bf16_a_tmem(tmem_base + t * kColTile + kColO, tmem_base + t * kColTile + kColS + 8 * i, b,
                                         idesc_pv, acc || i > 0);
                }
            };
            bool ok = wait_bounded(bar(kQFull), 0, abort_flag, p.status, 0xB30u) &&
                      wait_bounded(bar(kKFull), 0, abort_flag, p.status, 0xB31u);
            if (ok) {
                ptx::tc_fence_after_sync();
                issue_qk(0, 0);
                issue_qk(1, 0);
                ptx::tc_commit(bar(kKEmpty));
            }
            for (int j = 0; ok && j < n_tiles; ++j) {
                const int st = j & 1, nst = st ^ 1;
                const uint32_t par = static_cast<uint32_t>(j) & 1u;            // per-tile barriers flip every tile
                const uint32_t ring = static_cast<uint32_t>(j >> 1) & 1u;      // ring barriers every second tile
                const bool more = j + 1 < n_tiles;
                // query tile 0: P_0 V_j, then the next scores
                if (!wait_bounded(bar(kPFull), par, abort_flag, p.status, 0xB60u)) break;
                if (!wait_bounded(bar(kVFull + st), ring, abort_flag, p.status, 0xB70u | st)) break;
                ptx::tc_fence_after_sync();
                ATTN_TRACE(2, j);
                issue_pv(0, st, j > 0);
                if (more) {
                    if (!wait_bounded(bar(kKFull + nst), static_cast<uint32_t>((j + 1) >> 1) & 1u, abort_flag, p.status,
                                      0xB40u | nst))
                        break;
                    ptx::tc_fence_after_sync();
                    ATTN_TRACE(0, j + 1);
                    issue_qk(0, nst);
                } else {
                    ptx::tc_commit(bar(kPvDone));
                }
                // query tile 1
                if (!wait_bounded(bar(kPFull + 1), par, abort_flag, p.status, 0xB61u)) break;
                ptx::tc_fence_after_sync();
                issue_pv(1, st, j > 0);
                ptx::tc_commit(bar(kVEmpty + st));
                if (more) {
                    issue_qk(1, nst);
                    ptx::tc_commit(bar(kKEmpty + nst));
                } else {
                    ptx::tc_commit(bar(kPvDone + 1));
                }
                ATTN_TRACE(3, j);
            }
        }
        __syncwarp();
    } else {
        // ------------------------------------------------------------ softmax and epilogue: thread = query row
        const int t = (warp - 2) >> 2;                        // query tile of this warpgroup
        const int quad = warp & 3;
        const int r = quad * 32 + lane;                       // row of the tile = TMEM lane
        const uint32_t t_lane = tmem_base + t * kColTile + (static_cast<uint32_t>(quad * 32) << 16);
        const uint32_t sw = static_cast<uint32_t>(r & 7);
        const bool tracer = warp == 2;
        float m = -INFINITY, l = 0.0f;
        bool ok = true;
        for (int j = 0; j < n_tiles; ++j) {
            // S_j is complete, and with it every earlier MMA of this tile: O holds the sum over tiles 0..j-1
            if (!wait_bounded(bar(kSFull + t), static_cast<uint32_t>(j) & 1u, abort_flag, p.status, 0xB80u | t)) {
                ok = false;
                break;
            }
            ptx::tc_fence_after_sync();
            if (tracer) ATTN_TRACE(4, j);
            uint32_t s[4][32];
#pragma unroll
            for (int c = 0; c < 4; ++c) ptx::tmem_ld_32x32(t_lane + kColS + 32 * c, s[c]);
            ptx::tmem_ld_wait();
            if (tracer) ATTN_TRACE(5, j);
            const int valid = p.seq_kv - j * kBKV;              // keys of this tile that exist (>= 1)
            if (valid < kBKV) {  // the last tile of a ragged sequence: keys that do not exist score -inf
#pragma unroll
                for (int c = 0; c < 4; ++c)
#pragma unroll
                    for (int e = 0; e < 32; ++e)
                        if (c * 32 + e >= valid) s[c][e] = 0xFF800000u;
            }
            float mx8[8];
#pragma unroll
            for (int e = 0; e < 8; ++e) mx8[e] = __uint_as_float(s[0][e]);
#pragma unroll
            for (int c = 0; c < 4; ++c)
#pragma unroll
                for (int e = 0; e < 32; e += 8)
#pragma unroll
                    for (int k = 0; k < 8; ++k)
                        if (c + e > 0) mx8[k] = fmaxf(mx8[k], __uint_as_float(s[c][e + k]));
            const float mx = fmaxf(fmaxf(fmaxf(mx8[0], mx8[1]), fmaxf(mx8[2], mx8[3])),
                                   fmaxf(fmaxf(mx8[4], mx8[5]), fmaxf(mx8[6], mx8[7])));
            // The reference maximum m only follows the row maximum when that has grown by more than 2^8:
            // until then the probabilities are up to 256 times larger (exact in FP32 and BF16 alike, l carries
            // the same factor) and O, which lives in TMEM, does not have to be rescaled.
            const float m_tile = mx * p.scale_log2;
            const bool move = m_tile > m + kLazyLog2;
            const float m_new = move ? m_tile : m;
            const float alpha = move ? ex2(m - m_new) : 1.0f;   // 0 on the first tile (m = -inf)
            if (tracer) ATTN_TRACE(6, j);
            float sum = 0.0f;
            const uint64_t c2 = qmath::f32x2(p.scale_log2, p.scale_log2), nm2 = qmath::f32x2(-m_new, -m_new);
#pragma unroll
            for (int c = 0; c < 4; ++c)
#pragma unroll
                for (int e = 0; e < 32; e += 2) {
                    // s c - m for two scores in one two-lane FMA (each lane rounded as the scalar form would be)
                    float x0, x1;
                    qmath::f32x2_split(qmath::fma2(qmath::f32x2(__uint_as_float(s[c][e]), __uint_as_float(s[c][e + 1])), c2, nm2), x0, x1);
                    const float p0 = ex2(x0), p1 = ex2(x1);
                    sum += p0 + p1;
                    s[c][e >> 1] = pack_bf16(p0, p1);  // 16 words per 32 keys, packed in place
                }
            l = fmaf(l, alpha, sum);
            m = m_new;
            if (tracer) ATTN_TRACE(7, j);
            if (j > 0 && __any_sync(0xFFFFFFFFu, move)) {
#pragma unroll
                for (int c = 0; c < kD / 32; ++c) {
                    uint32_t o[32];
                    ptx::tmem_ld_32x32(t_lane + kColO + 32 * c, o);
                    ptx::tmem_ld_wait();
#pragma unroll
                    for (int e = 0; e < 32; ++e) o[e] = __float_as_uint(__uint_as_float(o[e]) * alpha);
                    ptx::tmem_st_32x32(t_lane + kColO + 32 * c, o);
                }
            }
            if (tracer) ATTN_TRACE(8, j);
            // P row: keys 2c and 2c+1 in column c, over the row's own scores (all of them are in registers)
#pragma unroll
            for (int c = 0; c < 4; ++c) ptx::tmem_st_32x16(t_lane + kColS + 16 * c, s[c]);
            ptx::tc_wait_st();
            ptx::tc_fence_before_sync();
            __syncwarp();
            if (lane == 0) ptx::mbar_arrive(bar(kPFull + t));
            if (tracer) ATTN_TRACE(9, j);
        }
        if (ok && wait_bounded(bar(kPvDone + t), 0, abort_flag, p.status, 0xBA0u | t)) {
            ptx::tc_fence_after_sync();
            const float inv = 1.0f / l;
            if constexpr (kQuantOut) {
                // thread = row: the kD columns of one head are whole 16-element blocks, quantized from registers
                const int row = q0 + t * kBQ + r;
                const bool row_ok = row < q_rows;
                const int64_t m = static_cast<int64_t>(batch) * p.seq_q + row;
                const float T = __ldcg(p.ts_out);
                const float c6T = __fmul_rn(6.0f, T);
                const int col0 = p.dest_col0 + head * kD;
                uint8_t *qrow = p.q_dest + m * p.dest_pitch + (col0 >> 1);
                uint32_t amax2 = 0, sfw[kD / 64] = {};
                uint32_t codes[kD / 8];  // the row's nibbles: stored in one go so that its 32-byte sectors fill at once
#pragma unroll
                for (int c = 0; c < kD / 32; ++c) {
                    uint32_t o[32];
                    ptx::tmem_ld_32x32(t_lane + kColO + 32 * c, o);
                    ptx::tmem_ld_wait();
                    uint32_t w[16];
                    uint32_t *code = codes + 4 * c;
#pragma unroll
                    for (int e = 0; e < 16; ++e)
                        w[e] = pack_bf16(__uint_as_float(o[2 * e]) * inv, __uint_as_float(o[2 * e + 1]) * inv);
#pragma unroll
                    for (int blk = 0; blk < 2; ++blk) {
                        const uint32_t *b = w + 8 * blk;
                        uint32_t a2 = qmath::absmax2(qmath::absmax2(qmath::absmax2(b[0], b[1]), qmath::absmax2(b[2], b[3])),
                                                     qmath::absmax2(qmath::absmax2(b[4], b[5]), qmath::absmax2(b[6], b[7])));
                        a2 &= 0x7FFF7FFFu;
                        amax2 = qmath::absmax2(amax2, a2);
                        const float a = fmaxf(qmath::bf16_lo(a2), qmath::bf16_hi(a2));
                        float rcp;
                        const uint32_t sb = qmath::block_scale(a, c6T, T, rcp);
                        code[2 * blk] = qmath::quantize8(b[0], b[1], b[2], b[3], rcp);
                        code[2 * blk + 1] = qmath::quantize8(b[4], b[5], b[6], b[7], rcp);
                        sfw[c >> 1] |= sb << (8 * ((c & 1) * 2 + blk));
                    }
                }
                if (row_ok) {
#pragma unroll
                    for (int c = 0; c < kD / 32; ++c)
                        *reinterpret_cast<uint4 *>(qrow + 16 * c) = make_uint4(codes[4 * c], codes[4 * c + 1], codes[4 * c + 2], codes[4 * c + 3]);
                }
                if (row_ok) {
#pragma unroll
                    for (int kc = 0; kc < kD / 64; ++kc) {  // the four scale bytes of a (row, 64-column chunk) slot are one word
                        const int64_t chunk = (m >> 7) * p.dest_chunks_k + (col0 >> 6) + kc;
                        *reinterpret_cast<uint32_t *>(p.sf_dest + chunk * 512 + (m & 31) * 16 + ((m & 127) >> 5) * 4) = sfw[kc];
                    }
                }
                if (p.amax_out != nullptr) {
                    amax2 &= 0x7FFF7FFFu;
                    uint32_t mx = row_ok ? max(amax2 & 0xFFFFu, amax2 >> 16) : 0u;
                    mx = __reduce_max_sync(0xFFFFFFFFu, mx);
                    if (lane == 0 && mx) atomicMax(p.amax_out, mx << 16);
                }
            } else {
            const uint32_t o_row = sQ + t * kTile + r * 128;  // Q_t is no longer read: its MMAs have completed
#pragma unroll
            for (int c = 0; c < kD / 32; ++c) {
                uint32_t o[32];
                ptx::tmem_ld_32x32(t_lane + kColO + 32 * c, o);
                ptx::tmem_ld_wait();
#pragma unroll
                for (int q = 0; q < 4; ++q) {
                    uint32_t w[4];
#pragma unroll
                    for (int e = 0; e < 4; ++e)
                        w[e] = pack_bf16(__uint_as_float(o[8 * q + 2 * e]) * inv, __uint_as_float(o[8 * q + 2 * e + 1]) * inv);
                    const int ch = c * 4 + q;
                    sts128(o_row + (ch >> 3) * kBox + ((static_cast<uint32_t>(ch & 7) ^ sw) << 4), w[0], w[1], w[2], w[3]);
                }
            }
            ptx::fence_proxy_async_smem();
            __syncwarp();
            const int row0 = q0 + t * kBQ + quad * 32;
            if (lane == 0 && row0 < q_rows) {  // this warp's 32 rows, boxes of 64 columns (clipped at the end of the stream)
#pragma unroll
                for (int bx = 0; bx < kBoxes; ++bx)
                    ptx::tma_store_3d(tm_o, head * kD + 64 * bx, row0, batch, sQ + t * kTile + bx * kBox + quad * 32 * 128);
                ptx::tma_store_commit();
                ptx::tma_store_wait_all<0>();
            }
            }
        }
    }

    // ---------------------------------------------------------------- teardown
    ptx::tc_fence_before_sync();
    __syncthreads();
    if (warp == 1) {
        ptx::tc_fence_after_sync();
        ptx::tmem_dealloc(tmem_base, kTmemCols);
    }
}

}  // namespace

sol_status_t launch_attention(const Stream *a, const Stream &b, int64_t batch, int64_t heads, int64_t head_dim,
                              const QuantDest *qd, cudaStream_t stream) {
    CUtensorMap tm[8];
    const uint64_t cols = static_cast<uint64_t>(heads) * static_cast<uint64_t>(head_dim);
    auto make = [&](CUtensorMap *t, const void *base, int64_t seq, int64_t ld, uint32_t box_rows) {
        return make_tmap_3d_bf16(t, base, cols, static_cast<uint64_t>(seq), static_cast<uint64_t>(batch),
                                 static_cast<uint64_t>(ld) * 2, static_cast<uint64_t>(seq) * ld * 2, 64, box_rows);
    };
    auto make4 = [&](CUtensorMap *t, const Stream &s) {
        // a quantized destination has no BF16 output tensor: the (unused) output map is a copy of the query map
        return make(t, s.q, s.seq_q, s.ld_q, kBQ) && make(t + 1, s.k, s.seq_kv, s.ld_k, kBKV) &&
               make(t + 2, s.v, s.seq_kv, s.ld_v, kBKV) &&
               (qd != nullptr ? make(t + 3, s.q, s.seq_q, s.ld_q, 32) : make(t + 3, s.out, s.seq_q, s.ld_out, 32));
    };
    if (!make4(tm + 4, b) || !make4(tm, a != nullptr ? *a : b)) return SOL_ERR_CUDA;  // one stream: the a maps are never used
    Params p{};
    p.q_split = a != nullptr ? static_cast<int>(a->seq_q) : 0;
    p.kv_split = a != nullptr ? static_cast<int>(a->seq_kv) : 0;
    p.seq_q = p.q_split + static_cast<int>(b.seq_q);
    p.seq_kv = p.kv_split + static_cast<int>(b.seq_kv);
    p.scale_log2 = 1.4426950408889634f / sqrtf(static_cast<float>(head_dim));
    p.status = device_status_word();
    if (qd != nullptr) {
        p.q_dest = static_cast<uint8_t *>(qd->q);
        p.sf_dest = static_cast<uint8_t *>(qd->sf);
        p.ts_out = qd->tscale;
        p.amax_out = qd->amax_out;
        p.dest_pitch = static_cast<int>(qd->dest_K / 2);
        p.dest_col0 = static_cast<int>(qd->dest_col0);
        p.dest_chunks_k = static_cast<int>(qd->dest_K / 64);
    }
    const bool quant = qd != nullptr, wide = head_dim == 128;
    auto kern = wide ? (quant ? attention_kernel<128, true> : attention_kernel<128, false>)
                     : (quant ? attention_kernel<64, true> : attention_kernel<64, false>);
    const int smem = smem_bytes(static_cast<int>(head_dim));
    static bool configured[4][64] = {};
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return SOL_ERR_CUDA;
    const int slot = (wide ? 2 : 0) + (quant ? 1 : 0);
    if (!configured[slot][dev]) {
        if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, smem) != cudaSuccess)
            return SOL_ERR_CUDA;
        configured[slot][dev] = true;
    }
    const dim3 grid(static_cast<unsigned>((p.seq_q + kQTiles * kBQ - 1) / (kQTiles * kBQ)), static_cast<unsigned>(heads),
                    static_cast<unsigned>(batch));
    kern<<<grid, kThreads, smem, stream>>>(tm[0], tm[1], tm[2], tm[3], tm[4], tm[5], tm[6], tm[7], p);
    return launch_status();
}

}  // namespace attn
}  // namespace sol

#ifdef SOL_TUNING
extern "C" int sol_debug_attention_trace(long long *host_out) {
    return cudaMemcpyFromSymbol(host_out, sol::attn::g_attn_trace, sizeof(sol::attn::g_attn_trace)) == cudaSuccess ? 0 : 1;
}
#endif
