// Stage-1 selection and rank-consistency metrics for sm_100a.
//
// After the NVFP4 rollout has scored N candidates per prompt, the K/2 best and K/2 worst are kept
// and their initial-noise seeds preserved for the BF16 regeneration (paper Section 3.4, Section 4.1:
// N = 96, K = 24); advantages are the group-standardised rewards (Section 2, GRPO equation).  The
// appendix on ranking consistency compares proxy and reference rewards with Kendall's tau,
// Spearman's rho and the Top/Bottom-k match.  The work is tiny (N^2 comparisons per prompt): one
// block per prompt, rewards in shared memory, ranks by counting, so that every result except the
// advantages is an exact integer.  Ties: the lower candidate index ranks higher.
#include "sol_internal.h"

namespace sol {
namespace {

constexpr int kSelThreads = 128;
constexpr int kMaxCandidates = 4096;   // rewards of one prompt held in shared memory

// rank = number of candidates that beat i (higher reward, or equal reward and lower index)
__device__ __forceinline__ int descending_rank(const float *r, int n, int i) {
    const float ri = r[i];
    int rank = 0;
    for (int j = 0; j < n; ++j) {
        const float rj = r[j];
        rank += (rj > ri) || (rj == ri && j < i);
    }
    return rank;
}

__global__ void __launch_bounds__(kSelThreads)
select_contrastive_kernel(const float *__restrict__ rewards, const uint64_t *__restrict__ seeds, int N, int K,
                          int32_t *__restrict__ idx_out, uint64_t *__restrict__ seeds_out,
                          float *__restrict__ adv_out) {
    extern __shared__ float sh[];
    float *r = sh;
    __shared__ double red[2][kSelThreads / 32];
    const int64_t p = blockIdx.x;
    const float *rp = rewards + p * N;
    double s1 = 0.0;
    for (int i = threadIdx.x; i < N; i += kSelThreads) {
        const float v = rp[i];
        r[i] = v;
        s1 += v;
    }
    __syncthreads();
    const int half = K >> 1;
    for (int i = threadIdx.x; i < N; i += kSelThreads) {
        const int rank = descending_rank(r, N, i);
        int pos = -1;
        if (rank < half) pos = rank;                           // the best, in descending order
        else if (rank >= N - half) pos = half + (N - 1 - rank);  // the worst, from the lowest
        if (pos >= 0) {
            idx_out[p * K + pos] = i;
            if (seeds_out != nullptr) seeds_out[p * K + pos] = seeds[p * N + i];
        }
    }
    if (adv_out == nullptr) return;
    // group statistics in FP64 (N values): mean, then the population variance around it
    for (int o = 16; o > 0; o >>= 1) s1 += __shfl_xor_sync(0xFFFFFFFFu, s1, o);
    if ((threadIdx.x & 31) == 0) red[0][threadIdx.x >> 5] = s1;
    __syncthreads();
    double mu = 0.0;
    for (int w = 0; w < kSelThreads / 32; ++w) mu += red[0][w];
    mu /= N;
    double s2 = 0.0;
    for (int i = threadIdx.x; i < N; i += kSelThreads) {
        const double d = r[i] - mu;
        s2 += d * d;
    }
    for (int o = 16; o > 0; o >>= 1) s2 += __shfl_xor_sync(0xFFFFFFFFu, s2, o);
    if ((threadIdx.x & 31) == 0) red[1][threadIdx.x >> 5] = s2;
    __syncthreads();
    double var = 0.0;
    for (int w = 0; w < kSelThreads / 32; ++w) var += red[1][w];
    const double sd = sqrt(var / N);
    for (int i = threadIdx.x; i < N; i += kSelThreads)
        adv_out[p * N + i] = sd > 0.0 ? static_cast<float>((r[i] - mu) / sd) : 0.0f;
}

__global__ void __launch_bounds__(kSelThreads)
rank_consistency_kernel(const float *__restrict__ ref, const float *__restrict__ proxy, int N, int k,
                        int64_t *__restrict__ counts_out, float *__restrict__ metrics_out) {
    extern __shared__ float sh[];
    float *a = sh, *b = sh + N;
    __shared__ long long red[4][kSelThreads / 32];
    const int64_t p = blockIdx.x;
    for (int i = threadIdx.x; i < N; i += kSelThreads) {
        a[i] = ref[p * N + i];
        b[i] = proxy[p * N + i];
    }
    __syncthreads();
    long long s = 0, d2 = 0, top = 0, bot = 0;
    for (int i = threadIdx.x; i < N; i += kSelThreads) {
        const int ra = descending_rank(a, N, i), rb = descending_rank(b, N, i);
        const long long d = ra - rb;
        d2 += d * d;
        top += (ra < k) && (rb < k);
        bot += (ra >= N - k) && (rb >= N - k);
        const float ai = a[i], bi = b[i];
        for (int j = i + 1; j < N; ++j) {   // concordant minus discordant pairs; a tie in either counts 0
            const int sa = (ai > a[j]) - (ai < a[j]), sb = (bi > b[j]) - (bi < b[j]);
            s += sa * sb;
        }
    }
    long long v[4] = {s, d2, top, bot};
#pragma unroll
    for (int q = 0; q < 4; ++q) {
        for (int o = 16; o > 0; o >>= 1) v[q] += __shfl_xor_sync(0xFFFFFFFFu, v[q], o);
        if ((threadIdx.x & 31) == 0) red[q][threadIdx.x >> 5] = v[q];
    }
    __syncthreads();
    if (threadIdx.x == 0) {
        long long t[4] = {0, 0, 0, 0};
        for (int q = 0; q < 4; ++q)
            for (int w = 0; w < kSelThreads / 32; ++w) t[q] += red[q][w];
        for (int q = 0; q < 4; ++q) counts_out[p * 4 + q] = t[q];
        if (metrics_out != nullptr) {
            const double n = N;
            metrics_out[p * 4 + 0] = static_cast<float>(t[0] / (n * (n - 1.0) / 2.0));
            metrics_out[p * 4 + 1] = static_cast<float>(1.0 - 6.0 * t[1] / (n * (n * n - 1.0)));
            metrics_out[p * 4 + 2] = static_cast<float>(static_cast<double>(t[2]) / k);
            metrics_out[p * 4 + 3] = static_cast<float>(static_cast<double>(t[3]) / k);
        }
    }
}

}  // namespace

int selection_max_candidates() { return kMaxCandidates; }

sol_status_t launch_select_contrastive(const float *rewards, const uint64_t *seeds, int64_t P, int64_t N, int64_t K,
                                       int32_t *idx_out, uint64_t *seeds_out, float *adv_out, cudaStream_t stream) {
    select_contrastive_kernel<<<static_cast<unsigned>(P), kSelThreads, N * sizeof(float), stream>>>(
        rewards, seeds, static_cast<int>(N), static_cast<int>(K), idx_out, seeds_out, adv_out);
    return launch_status();
}

sol_status_t launch_rank_consistency(const float *ref, const float *proxy, int64_t P, int64_t N, int64_t k,
                                     int64_t *counts_out, float *metrics_out, cudaStream_t stream) {
    rank_consistency_kernel<<<static_cast<unsigned>(P), kSelThreads, 2 * N * sizeof(float), stream>>>(
        ref, proxy, static_cast<int>(N), static_cast<int>(k), counts_out, metrics_out);
    return launch_status();
}

}  // namespace sol
