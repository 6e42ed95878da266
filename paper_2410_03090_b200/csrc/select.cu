// Pooling of the raw window scores and variable-k top-k selection per unit (paper Section 3.3.3:
// the tokens with the highest cumulative window attention are kept within the head's budget; the w
// window tokens are part of the budget).
//
// One CTA of 1024 threads per unit.
//   1. pooled[j] = max / mean of raw over the pool window clipped to the prefix (written out: it is the
//      `d_scores` output of the pass).
//   2. Radix select of the k-th largest pooled score, k = budget - w, on the order-preserving 32-bit
//      image of the float: three histogram passes (11 + 11 + 10 bits) give the exact threshold T, the
//      number of scores above it and how many scores equal to T are still needed.
//   3. Ordered compaction: each warp owns a contiguous segment; ballots and population counts give every
//      kept position its output slot, so the kept positions come out ascending, and among scores equal to
//      T the lowest positions win.  The window positions follow.
// Counting is integer work: the result does not depend on the order in which threads run.
#include <cooperative_groups.h>

#include "common.cuh"

namespace uncomp {

constexpr int kSelThreads = 1024;
constexpr int kSelWarps = kSelThreads / 32;

__device__ __forceinline__ uint32_t ordered_bits(float f) {
    const uint32_t b = __float_as_uint(f);
    return (b & 0x80000000u) ? ~b : (b | 0x80000000u);
}

struct SelSmem {
    int hist[2048];
    int scan[kSelThreads];
    int warp_gt[kSelWarps], warp_eq[kSelWarps];
    int bin, above;
};

// What a unit may write: its slab of d_indices is offsets[u] .. offsets[u+1].  The budget should equal the slab
// length and lie in [w, P + w]; whatever disagrees raises UNCOMP_STATUS_BOUNDS and the unit is cut to what the
// slab and the budget both allow, so that every slot of the slab holds a valid position and nothing outside it
// is touched: k top positions, then wn window positions, then `fill` copies of the last position.
struct Slab {
    int64_t begin, seg;
    int k, wn;
    int64_t fill;
};

__device__ __forceinline__ Slab slab_of(const int32_t *__restrict__ budgets, const int64_t *__restrict__ offsets,
                                        int units, int u, int P, int w, bool reporter, uint32_t *status) {
    const int64_t o0 = offsets[u], o1 = offsets[u + 1], oend = offsets[units];
    const int budget = budgets[u];
    const bool off_ok = o0 >= 0 && o1 >= o0 && o1 <= oend;
    const int64_t seg = off_ok ? o1 - o0 : 0;
    if (!(off_ok && (int64_t)budget == seg && budget >= w && budget <= P + w) && reporter)
        atomicOr(status, (uint32_t)UNCOMP_STATUS_BOUNDS);
    int64_t b = min(max(budget, 0), P + w);
    b = min(b, seg);
    Slab s;
    s.begin = off_ok ? o0 : 0;
    s.seg = seg;
    s.k = (int)max((int64_t)0, min(b - w, (int64_t)P));
    s.wn = (int)min((int64_t)w, b - s.k);
    s.fill = seg - s.k - s.wn;
    return s;
}

// Finds the bin (counting down from the top) that holds the kr-th largest element.  All threads call it.
__device__ void find_bin(SelSmem &S, int nbins, int kr, int tid) {
    // thread t covers bins nbins-1-2t and nbins-2-2t
    const int b0 = nbins - 1 - 2 * tid;
    const int h0 = b0 >= 0 ? S.hist[b0] : 0;
    const int h1 = b0 - 1 >= 0 ? S.hist[b0 - 1] : 0;
    S.scan[tid] = h0 + h1;
    __syncthreads();
    for (int o = 1; o < kSelThreads; o <<= 1) {
        const int add = tid >= o ? S.scan[tid - o] : 0;
        __syncthreads();
        S.scan[tid] += add;
        __syncthreads();
    }
    const int excl = S.scan[tid] - (h0 + h1);
    if (b0 >= 0 && excl < kr && kr <= excl + h0) { S.bin = b0; S.above = excl; }
    else if (b0 - 1 >= 0 && excl + h0 < kr && kr <= excl + h0 + h1) { S.bin = b0 - 1; S.above = excl + h0; }
    __syncthreads();
}

__global__ void __launch_bounds__(kSelThreads) pool_select_kernel(const float *__restrict__ raw,
                                                                 float *__restrict__ pooled, int P, int w,
                                                                 int pool_kernel, int pool_mode,
                                                                 const int32_t *__restrict__ budgets,
                                                                 const int64_t *__restrict__ offsets,
                                                                 int units, int32_t *__restrict__ indices,
                                                                 uint32_t *__restrict__ status) {
    __shared__ SelSmem S;
    const int u = blockIdx.x, tid = threadIdx.x, lane = tid & 31, wid = tid >> 5;
    const float *r = raw + (size_t)u * P;
    float *s = pooled + (size_t)u * P;

    // ---- 1. pooling ------------------------------------------------------------------------------
    const int half = pool_kernel >> 1;
    for (int j = tid; j < P; j += kSelThreads) {
        const int lo = max(0, j - half), hi = min(P - 1, j + half);
        float acc = pool_mode ? 0.f : r[lo];
        for (int t = lo; t <= hi; ++t) acc = pool_mode ? acc + r[t] : fmaxf(acc, r[t]);
        s[j] = pool_mode ? acc / (float)(hi - lo + 1) : acc;
    }
    const Slab slab = slab_of(budgets, offsets, units, u, P, w, tid == 0, status);
    const int k = slab.k;
    int32_t *out = indices + slab.begin;
    for (int i = tid; i < slab.wn; i += kSelThreads)
            if (UNCOMP_INDEX_OK(k + i, slab.seg, status)) out[k + i] = P + i;
    for (int64_t i = tid; i < slab.fill; i += kSelThreads)
            if (UNCOMP_INDEX_OK(k + slab.wn + i, slab.seg, status)) out[k + slab.wn + i] = P + w - 1;
    if (k == 0) return;   // uniform over the CTA
    __syncthreads();      // pooled scores of this unit are visible to the whole CTA

    // ---- 2. threshold ----------------------------------------------------------------------------
    uint32_t prefix = 0;      // bits of the threshold fixed so far
    int kr = k;               // rank still to resolve inside the current bin
    if (k < P) {
#pragma unroll 1
        for (int pass = 0; pass < 3; ++pass) {
            const int shift = pass == 0 ? 21 : (pass == 1 ? 10 : 0);
            const int nbits = pass == 2 ? 10 : 11;
            const int nbins = 1 << nbits;
            const uint32_t himask = pass == 0 ? 0u : (0xffffffffu << (shift + nbits));
            for (int b = tid; b < 2048; b += kSelThreads) S.hist[b] = 0;
            __syncthreads();
            for (int j = tid; j < P; j += kSelThreads) {
                const uint32_t v = ordered_bits(s[j]);
                if ((v & himask) == prefix && UNCOMP_INDEX_OK((v >> shift) & (nbins - 1), 2048, status))
                    atomicAdd(&S.hist[(v >> shift) & (nbins - 1)], 1);
            }
            __syncthreads();
            find_bin(S, nbins, kr, tid);
            prefix |= (uint32_t)S.bin << shift;
            kr -= S.above;
            __syncthreads();
        }
    }
    // k >= P keeps every prefix position: threshold below everything
    const uint32_t T = k < P ? prefix : 0u;
    const int need_eq = k < P ? kr : P;   // scores equal to T that are still kept (lowest positions first)

    // ---- 3. ordered compaction -------------------------------------------------------------------
    const int seg = ((P + kSelWarps - 1) / kSelWarps + 31) & ~31;
    const int j0 = min(P, wid * seg), j1 = min(P, j0 + seg);
    int cg = 0, ce = 0;
    for (int j = j0 + lane; j < j1; j += 32) {
        const uint32_t v = ordered_bits(s[j]);
        cg += v > T;
        ce += v == T;
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        cg += __shfl_xor_sync(0xffffffffu, cg, o);
        ce += __shfl_xor_sync(0xffffffffu, ce, o);
    }
    if (lane == 0) { S.warp_gt[wid] = cg; S.warp_eq[wid] = ce; }
    __syncthreads();
    int gt_run = 0, eq_run = 0;
    for (int x = 0; x < wid; ++x) { gt_run += S.warp_gt[x]; eq_run += S.warp_eq[x]; }
    const unsigned lt = (1u << lane) - 1u;
    for (int jb = j0; jb < j1; jb += 32) {
        const int j = jb + lane;
        const uint32_t v = j < j1 ? ordered_bits(s[j]) : 0u;
        const bool gt = j < j1 && v > T;
        const bool eq = j < j1 && v == T;
        const unsigned mg = __ballot_sync(0xffffffffu, gt), me = __ballot_sync(0xffffffffu, eq);
        const int gtb = gt_run + __popc(mg & lt);
        const int eqb = eq_run + __popc(me & lt);
        if ((gt || (eq && eqb < need_eq)) && UNCOMP_INDEX_OK(gtb + min(eqb, need_eq), k, status))
            out[gtb + min(eqb, need_eq)] = j;
        gt_run += __popc(mg);
        eq_run += __popc(me);
    }
}

// The same selection with a unit spread over a cluster of 8 CTAs, for calls with few units (a layer of one sequence,
// the hidden-state eviction with one unit per sequence), where one CTA per unit would leave most SMs idle.  CTA r of
// the cluster owns the r-th eighth of the positions; histograms and counts are combined through distributed shared
// memory by CTA 0 and read back by the others.  The result is identical to the single-CTA kernel.
constexpr int kSelCluster = 8;

__global__ void __cluster_dims__(kSelCluster, 1, 1) __launch_bounds__(kSelThreads)
pool_select_cluster_kernel(const float *__restrict__ raw, float *__restrict__ pooled, int P, int w, int pool_kernel,
                           int pool_mode, const int32_t *__restrict__ budgets, const int64_t *__restrict__ offsets,
                           int units, int32_t *__restrict__ indices, uint32_t *__restrict__ status) {
    namespace cg = cooperative_groups;
    __shared__ SelSmem S;
    __shared__ int slice_gt, slice_eq;
    cg::cluster_group cluster = cg::this_cluster();
    const int rank = (int)cluster.block_rank();
    const int u = blockIdx.x / kSelCluster, tid = threadIdx.x, lane = tid & 31, wid = tid >> 5;
    const float *r = raw + (size_t)u * P;
    float *s = pooled + (size_t)u * P;
    // this CTA's positions: a multiple of 1024 per CTA, so that warps own aligned segments of 32
    const int per = ((P + kSelCluster - 1) / kSelCluster + kSelThreads - 1) / kSelThreads * kSelThreads;
    const int p0 = min(P, rank * per), p1 = min(P, p0 + per);

    const int half = pool_kernel >> 1;
    for (int j = p0 + tid; j < p1; j += kSelThreads) {
        const int lo = max(0, j - half), hi = min(P - 1, j + half);
        float acc = pool_mode ? 0.f : r[lo];
        for (int t = lo; t <= hi; ++t) acc = pool_mode ? acc + r[t] : fmaxf(acc, r[t]);
        s[j] = pool_mode ? acc / (float)(hi - lo + 1) : acc;
    }
    const Slab slab = slab_of(budgets, offsets, units, u, P, w, tid == 0 && rank == 0, status);
    const int k = slab.k;
    int32_t *out = indices + slab.begin;
    if (rank == 0) {
        for (int i = tid; i < slab.wn; i += kSelThreads)
            if (UNCOMP_INDEX_OK(k + i, slab.seg, status)) out[k + i] = P + i;
        for (int64_t i = tid; i < slab.fill; i += kSelThreads)
            if (UNCOMP_INDEX_OK(k + slab.wn + i, slab.seg, status)) out[k + slab.wn + i] = P + w - 1;
    }
    if (k == 0) return;   // uniform over the cluster
    __syncthreads();      // this CTA reads only the pooled scores it wrote itself

    SelSmem *S0 = cluster.map_shared_rank(&S, 0);
    uint32_t prefix = 0;
    int kr = k;
    if (k < P) {
#pragma unroll 1
        for (int pass = 0; pass < 3; ++pass) {
            const int shift = pass == 0 ? 21 : (pass == 1 ? 10 : 0);
            const int nbits = pass == 2 ? 10 : 11;
            const int nbins = 1 << nbits;
            const uint32_t himask = pass == 0 ? 0u : (0xffffffffu << (shift + nbits));
            for (int b = tid; b < 2048; b += kSelThreads) S.hist[b] = 0;
            __syncthreads();
            for (int j = p0 + tid; j < p1; j += kSelThreads) {
                const uint32_t v = ordered_bits(s[j]);
                if ((v & himask) == prefix && UNCOMP_INDEX_OK((v >> shift) & (nbins - 1), 2048, status))
                    atomicAdd(&S.hist[(v >> shift) & (nbins - 1)], 1);
            }
            cluster.sync();                       // every CTA's histogram is complete
            if (rank == 0) {
                for (int b = tid; b < nbins; b += kSelThreads) {
                    int sum = S.hist[b];
                    for (int c = 1; c < kSelCluster; ++c) sum += cluster.map_shared_rank(&S, c)->hist[b];
                    S.hist[b] = sum;              // only this thread reads or writes bin b of CTA 0 here
                }
                __syncthreads();
                find_bin(S, nbins, kr, tid);
            }
            cluster.sync();                       // bin and count above it are published by CTA 0
            prefix |= (uint32_t)S0->bin << shift;
            kr -= S0->above;
            cluster.sync();                       // all have read them before the next pass clears the histograms
        }
    }
    const uint32_t T = k < P ? prefix : 0u;
    const int need_eq = k < P ? kr : P;

    // ordered compaction: counts of the lower CTAs first, then of the lower warps of this CTA
    const int seg = per / kSelWarps;              // a multiple of 32
    const int j0 = min(p1, p0 + wid * seg), j1 = min(p1, j0 + seg);
    int cg_ = 0, ce = 0;
    for (int j = j0 + lane; j < j1; j += 32) {
        const uint32_t v = ordered_bits(s[j]);
        cg_ += v > T;
        ce += v == T;
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        cg_ += __shfl_xor_sync(0xffffffffu, cg_, o);
        ce += __shfl_xor_sync(0xffffffffu, ce, o);
    }
    if (lane == 0) { S.warp_gt[wid] = cg_; S.warp_eq[wid] = ce; }
    __syncthreads();
    if (tid == 0) {
        int a = 0, b = 0;
        for (int x = 0; x < kSelWarps; ++x) { a += S.warp_gt[x]; b += S.warp_eq[x]; }
        slice_gt = a;
        slice_eq = b;
    }
    cluster.sync();
    int gt_run = 0, eq_run = 0;
    for (int c = 0; c < rank; ++c) {
        gt_run += *cluster.map_shared_rank(&slice_gt, c);
        eq_run += *cluster.map_shared_rank(&slice_eq, c);
    }
    for (int x = 0; x < wid; ++x) { gt_run += S.warp_gt[x]; eq_run += S.warp_eq[x]; }
    const unsigned lt = (1u << lane) - 1u;
    for (int jb = j0; jb < j1; jb += 32) {
        const int j = jb + lane;
        const uint32_t v = j < j1 ? ordered_bits(s[j]) : 0u;
        const bool gt = j < j1 && v > T;
        const bool eq = j < j1 && v == T;
        const unsigned mg = __ballot_sync(0xffffffffu, gt), me = __ballot_sync(0xffffffffu, eq);
        const int gtb = gt_run + __popc(mg & lt);
        const int eqb = eq_run + __popc(me & lt);
        if ((gt || (eq && eqb < need_eq)) && UNCOMP_INDEX_OK(gtb + min(eqb, need_eq), k, status))
            out[gtb + min(eqb, need_eq)] = j;
        gt_run += __popc(mg);
        eq_run += __popc(me);
    }
    cluster.sync();       // no CTA leaves while another may still read its shared memory
}

cudaError_t launch_pool_select(const Plan &p, const float *d_raw, float *d_pooled, int pool_kernel, int pool_mode,
                               const int32_t *d_budgets, const int64_t *d_offsets, int32_t *d_indices,
                               uint32_t *d_status, cudaStream_t st) {
    int dev = 0, sms = 148;
    cudaGetDevice(&dev);
    cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
    if (p.units * kSelCluster <= 2 * sms && p.prefix >= 4096)      // few units: a cluster of CTAs per unit
        pool_select_cluster_kernel<<<p.units * kSelCluster, kSelThreads, 0, st>>>(
            d_raw, d_pooled, p.prefix, p.shape.w, pool_kernel, pool_mode, d_budgets, d_offsets, p.units, d_indices,
            d_status);
    else
        pool_select_kernel<<<p.units, kSelThreads, 0, st>>>(d_raw, d_pooled, p.prefix, p.shape.w, pool_kernel, pool_mode,
                                                            d_budgets, d_offsets, p.units, d_indices, d_status);
    return cudaGetLastError();
}

}  // namespace uncomp
