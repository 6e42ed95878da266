// Head-group token budgets and the layer-group partition (paper Section 3.3.3 and 3.3.2).
//
// A single CTA: the input is at most a few thousand effective ranks, and the kernel exists so that the
// pass needs no host synchronisation between the entropy stage and the selection stage.
//
// Ranking is by counting (rank = number of heads of the ranking set that come first), the group target
// t_g = n_max - g * n (n_max - avg) / S, S = sum_g n_g g, is kept as the exact fraction num_g / S, heads
// get floor(t_g) and the tokens still missing go to the largest remainders (ties: better rank).  Every
// step is integer arithmetic, so the budgets are reproducible bit for bit.
#include "common.cuh"

namespace uncomp {

constexpr int kBudThreads = 1024;

__host__ __device__ __forceinline__ int group_lo(int g, int n, int M) { return (int)(((int64_t)g * n) / M); }

__global__ void __launch_bounds__(kBudThreads) budgets_kernel(const float *__restrict__ erank, int B, int L, int H,
                                                             int N, int w, uncomp_budget_params bp,
                                                             int32_t *__restrict__ budgets,
                                                             int64_t *__restrict__ offsets,
                                                             int32_t *__restrict__ layer_group,
                                                             int32_t *__restrict__ layer_ctx,
                                                             int32_t *__restrict__ rank_ws,
                                                             int64_t *__restrict__ rem_ws) {
    const int tid = threadIdx.x;
    const int units = B * L * H;
    const int n = bp.scope ? L * H : H;          // ranking-set size
    const int M = bp.M;
    const int64_t avg = bp.avg_budget, n_max = bp.n_max;

    // S = sum_g n_g * g and the tokens the floors leave undistributed (same for every ranking set)
    int64_t S = 0, floor_total = 0;
    for (int g = 0; g < M; ++g) S += (int64_t)(group_lo(g + 1, n, M) - group_lo(g, n, M)) * g;
    for (int g = 0; g < M; ++g) {
        const int64_t ng = group_lo(g + 1, n, M) - group_lo(g, n, M);
        const int64_t fl = M == 1 ? avg : (n_max * S - (int64_t)g * n * (n_max - avg)) / S;
        floor_total += ng * fl;
    }
    const int missing = (int)((int64_t)n * avg - floor_total);

    // phase 1: rank within the set, group, floor and remainder
    for (int u = tid; u < units; u += kBudThreads) {
        const int set_base = (u / n) * n;
        const float e = erank[u];
        int r = 0;
        for (int j = 0; j < n; ++j) {
            const float ej = erank[set_base + j];
            r += (ej > e) || (ej == e && set_base + j < u);
        }
        int g = (int)(((int64_t)r * M) / n);
        while (g + 1 < M && group_lo(g + 1, n, M) <= r) ++g;
        while (g > 0 && group_lo(g, n, M) > r) --g;
        int64_t fl, rem;
        if (M == 1) { fl = avg; rem = 0; }
        else {
            const int64_t num = n_max * S - (int64_t)g * n * (n_max - avg);
            fl = num / S;
            rem = num % S;
        }
        rank_ws[u] = r;
        rem_ws[u] = rem;
        budgets[u] = (int32_t)fl;
    }
    __syncthreads();
    // phase 2: largest remainders
    for (int u = tid; u < units; u += kBudThreads) {
        const int set_base = (u / n) * n;
        const int64_t rem = rem_ws[u];
        const int r = rank_ws[u];
        int ahead = 0;
        for (int j = 0; j < n; ++j) {
            const int64_t rj = rem_ws[set_base + j];
            ahead += (rj > rem) || (rj == rem && rank_ws[set_base + j] < r);
        }
        if (ahead < missing) budgets[u] += 1;
    }
    __syncthreads();
    // phase 3: exclusive prefix sum over units, a block scan per 1024 units with a running carry
    __shared__ int64_t scan[kBudThreads];
    __shared__ int64_t carry;
    if (tid == 0) { carry = 0; offsets[0] = 0; }
    __syncthreads();
    for (int base = 0; base < units; base += kBudThreads) {
        const int u = base + tid;
        scan[tid] = u < units ? (int64_t)budgets[u] : 0;
        __syncthreads();
        for (int o = 1; o < kBudThreads; o <<= 1) {
            const int64_t add = tid >= o ? scan[tid - o] : 0;
            __syncthreads();
            scan[tid] += add;
            __syncthreads();
        }
        if (u < units) offsets[u + 1] = carry + scan[tid];
        __syncthreads();
        if (tid == 0) carry += scan[kBudThreads - 1];
        __syncthreads();
    }
    // phase 4: layer groups
    if (layer_group && layer_ctx) {
        for (int b = tid; b < B; b += kBudThreads) {
            int32_t *lg = layer_group + (size_t)b * L, *lc = layer_ctx + (size_t)b * L;
            if (bp.dn <= 0) {
                for (int l = 0; l < L; ++l) { lg[l] = 0; lc[l] = N; }
                continue;
            }
            int boundaries = 0;
            lg[0] = 0;
            double prev = 0.0;
            for (int h = 0; h < H; ++h) prev += (double)erank[((size_t)b * L) * H + h];
            prev /= (double)H;
            for (int l = 0; l + 1 < L; ++l) {
                double next = 0.0;
                for (int h = 0; h < H; ++h) next += (double)erank[((size_t)b * L + l + 1) * H + h];
                next /= (double)H;
                if (prev - next > (double)bp.eps) ++boundaries;
                lg[l + 1] = boundaries;
                prev = next;
            }
            for (int l = 0; l < L; ++l) {
                if (lg[l] == 0) lc[l] = N;
                else {
                    const int64_t c = (int64_t)bp.n_last + (int64_t)(boundaries - lg[l]) * bp.dn;
                    lc[l] = (int32_t)(c < N ? c : N);
                }
            }
        }
    }
}

// Host-side check of the schedule's preconditions; mirrors the arithmetic of the kernel.
int check_budget_params(const uncomp_shape &s, const uncomp_budget_params &bp) {
    const int n = bp.scope ? s.L * s.H : s.H;
    if (bp.M < 1 || bp.M > n) return UNCOMP_E_PARAM;
    if (bp.avg_budget < s.w || bp.n_max < bp.avg_budget || bp.n_max > s.N) return UNCOMP_E_PARAM;
    if (bp.dn < 0 || (bp.dn > 0 && bp.n_last < 1)) return UNCOMP_E_PARAM;
    if (bp.M > 1) {
        int64_t S = 0;
        for (int g = 0; g < bp.M; ++g) S += (int64_t)(group_lo(g + 1, n, bp.M) - group_lo(g, n, bp.M)) * g;
        const int64_t num_last = (int64_t)bp.n_max * S - (int64_t)(bp.M - 1) * n * (bp.n_max - bp.avg_budget);
        if (num_last < (int64_t)s.w * S) return UNCOMP_E_PARAM;
    }
    return UNCOMP_OK;
}

cudaError_t launch_budgets(const Plan &p, const float *d_erank, const uncomp_budget_params &bp, int32_t *d_budgets,
                           int64_t *d_offsets, int32_t *d_layer_group, int32_t *d_layer_ctx, int32_t *d_rank,
                           int64_t *d_rem, cudaStream_t st) {
    budgets_kernel<<<1, kBudThreads, 0, st>>>(d_erank, p.shape.B, p.shape.L, p.shape.H, p.shape.N, p.shape.w, bp,
                                              d_budgets, d_offsets, d_layer_group, d_layer_ctx, d_rank, d_rem);
    return cudaGetLastError();
}

}  // namespace uncomp
