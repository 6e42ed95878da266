// Preparation stage (paper Section 3.3.1 "Preparation Stage": the effective rank of every head averaged over
// the samples; Algorithm 1: every sample puts each head into one of M clusters, the final label of a head is
// the majority vote over the samples).
//
// Input: erank [S, L, H], the output of the entropy stage for S samples.  A ranking set is one layer (H heads)
// or the whole model (L*H heads).  Grouping is the budget rule's: rank r by descending value (equal values:
// lower index first) goes to group g with floor(g n / M) <= r < floor((g + 1) n / M).
//   vote kernel    a thread per (sample, head) ranks the head inside its set by counting and adds one vote
//                  (integer atomics: the totals do not depend on the order);
//   finish kernel  grid (sets): mean over the samples with fp64 accumulation in a fixed order, grouping of the
//                  means, arg-max of the votes (lowest group on a tie).
#include "common.cuh"

namespace uncomp {

namespace {
constexpr int kPrepThreads = 256;

__device__ __forceinline__ int group_of_rank(int r, int n, int M) {
    int g = (int)(((int64_t)r * M) / n);
    while (g + 1 < M && (int)(((int64_t)(g + 1) * n) / M) <= r) ++g;
    while (g > 0 && (int)(((int64_t)g * n) / M) > r) --g;
    return g;
}

__device__ __forceinline__ int rank_in_set(const float *v, int n, int i) {
    const float e = v[i];
    int r = 0;
    for (int j = 0; j < n; ++j) r += (v[j] > e) || (v[j] == e && j < i);
    return r;
}

// one thread per (sample, head): the set's values are read straight from global memory (a set is at most
// 32 KB and stays in L1)
__global__ void __launch_bounds__(kPrepThreads) prepare_vote_kernel(const float *__restrict__ erank, int S, int LH, int n,
                                                                   int M, int32_t *__restrict__ votes) {
    const int64_t idx = (int64_t)blockIdx.x * kPrepThreads + threadIdx.x;
    if (idx >= (int64_t)S * LH) return;
    const int h = (int)(idx % LH), set = h / n, i = h % n;
    const float *vals = erank + (idx - h) + (size_t)set * n;
    const int g = group_of_rank(rank_in_set(vals, n, i), n, M);
    atomicAdd(&votes[(size_t)h * M + g], 1);
}

// grid (sets): a warp per head sums its samples (lane-strided fp64 partial sums, then a butterfly: a fixed order)
__global__ void __launch_bounds__(kPrepThreads) prepare_finish_kernel(const float *__restrict__ erank, int S, int LH,
                                                                     int n, int M, const int32_t *__restrict__ votes,
                                                                     float *__restrict__ mean,
                                                                     int32_t *__restrict__ group_mean,
                                                                     int32_t *__restrict__ group_vote) {
    extern __shared__ float vals[];
    const int set = blockIdx.x, lane = threadIdx.x & 31, wid = threadIdx.x >> 5;
    for (int i = wid; i < n; i += kPrepThreads / 32) {
        const size_t h = (size_t)set * n + i;
        double acc = 0.0;
        for (int s = lane; s < S; s += 32) acc += (double)erank[(size_t)s * LH + h];
        acc = warp_sum(acc);
        if (lane == 0) {
            const float m = (float)(acc / (double)S);
            vals[i] = m;
            mean[h] = m;
            const int32_t *v = votes + h * M;
            int best = 0;
            for (int g = 1; g < M; ++g)
                if (v[g] > v[best]) best = g;
            group_vote[h] = best;
        }
    }
    __syncthreads();
    for (int i = threadIdx.x; i < n; i += kPrepThreads)
        group_mean[(size_t)set * n + i] = group_of_rank(rank_in_set(vals, n, i), n, M);
}
// Retrieval layer (paper Section 3.3.2, "Retrieval Layer"): the layer after the largest rise of the layer mean.
// One CTA: a thread per layer forms the mean over heads in fp64 (head order), thread 0 scans the rises in layer order.
__global__ void __launch_bounds__(kPrepThreads) retrieval_layer_kernel(const float *__restrict__ values, int L, int H,
                                                                      int32_t *__restrict__ layer,
                                                                      float *__restrict__ increase) {
    extern __shared__ double lmean[];
    for (int l = threadIdx.x; l < L; l += kPrepThreads) {
        double e = 0.0;
        for (int h = 0; h < H; ++h) e += (double)values[(size_t)l * H + h];
        lmean[l] = e / (double)H;
    }
    __syncthreads();
    for (int l = threadIdx.x; l + 1 < L; l += kPrepThreads)
        if (increase) increase[l] = (float)(lmean[l + 1] - lmean[l]);
    if (threadIdx.x == 0) {
        int best = 1;
        double best_inc = lmean[1] - lmean[0];
        for (int l = 2; l < L; ++l) {
            const double inc = lmean[l] - lmean[l - 1];
            if (inc > best_inc) { best_inc = inc; best = l; }
        }
        *layer = best;
    }
}
}  // namespace

cudaError_t launch_retrieval_layer(const float *d_values, int L, int H, int32_t *d_layer, float *d_increase,
                                   cudaStream_t st) {
    retrieval_layer_kernel<<<1, kPrepThreads, (size_t)L * sizeof(double), st>>>(d_values, L, H, d_layer, d_increase);
    return cudaGetLastError();
}

cudaError_t launch_prepare_groups(const float *d_erank, int S, int L, int H, int M, int scope, float *d_mean,
                                  int32_t *d_group_mean, int32_t *d_votes, int32_t *d_group_vote, Profiler *prof,
                                  cudaStream_t st) {
    const int LH = L * H, n = scope ? LH : H, sets = scope ? 1 : L;
    cudaError_t e = cudaMemsetAsync(d_votes, 0, (size_t)LH * M * sizeof(int32_t), st);
    if (e != cudaSuccess) return e;
    {
        ProfScope ps(prof, kSlotPrepareVote, st);
        const int64_t total = (int64_t)S * LH;
        prepare_vote_kernel<<<(unsigned)((total + kPrepThreads - 1) / kPrepThreads), kPrepThreads, 0, st>>>(d_erank, S, LH, n,
                                                                                                            M, d_votes);
    }
    {
        ProfScope ps(prof, kSlotPrepareFinish, st);
        prepare_finish_kernel<<<sets, kPrepThreads, n * sizeof(float), st>>>(d_erank, S, LH, n, M, d_votes, d_mean,
                                                                             d_group_mean, d_group_vote);
    }
    return cudaGetLastError();
}

}  // namespace uncomp
