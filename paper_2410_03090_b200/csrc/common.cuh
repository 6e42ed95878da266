// Shared device/host helpers of the uncomp CUDA library (sm_100a only).
#pragma once

#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "../../include/uncomp.h"

namespace uncomp {

constexpr int kD = 128;          // head dimension supported by every kernel
constexpr int kMaxRows = 512;    // G * w upper bound (window rows of all grouped query heads)
constexpr int kTargetSms = 148;  // SM count of the part the grids are sized for (B200)

// Carve-up of the caller's workspace, decided by the shape alone (see api.cu).
struct Plan {
    uncomp_shape shape;
    int units;          // B * L * H
    int G;              // query heads per KV head
    int rows;           // G * w
    int prefix;         // N - w
    int gram_splits;    // token chunks per unit in the Gram stage (P)
    int gram_chunk;     // tokens per chunk
    int score_splits;   // token chunks per unit in the scorer's statistics pass
    int score_chunk;    // tokens per chunk
    size_t off_status, off_gram, off_stats_part, off_stats, off_raw, off_pooled, off_rank, off_rem;
    size_t off_ev_logits, off_ev_stats, off_ev_raw, off_ev_pooled, off_ev_budgets, off_ev_offsets;   // hidden-state eviction
    size_t off_dec_stats, off_dec_part, off_dec_new;   // decode-time update (its logits reuse off_raw .. off_rank)
    size_t bytes;
};

Plan make_plan(const uncomp_shape &s);

struct UnitAddr {
    int L, H;
    int64_t sB, sL, sH, sN;
    __host__ __device__ inline int64_t base(int u) const {
        const int h = u % H;
        const int l = (u / H) % L;
        const int b = u / (H * L);
        return (int64_t)b * sB + (int64_t)l * sL + (int64_t)h * sH;
    }
};

inline UnitAddr make_addr(const uncomp_shape &s, const uncomp_strides &st) {
    UnitAddr a;
    a.L = s.L; a.H = s.H; a.sB = st.sB; a.sL = st.sL; a.sH = st.sH; a.sN = st.sN;
    return a;
}

// Debug library (-DUNCOMP_DEBUG, built as libuncomp_debug.so): the kernels that place data at computed positions
// (selection, compaction, decode-time commit, hidden-state gather) check every such
// index against the extent it must stay in.  A violation raises UNCOMP_STATUS_BOUNDS and the access is skipped:
// no trap, no assert.  In the release library the check is the constant `true`.
#ifdef UNCOMP_DEBUG
__device__ __forceinline__ bool debug_index_ok(int64_t i, int64_t extent, uint32_t *status) {
    if (i >= 0 && i < extent) return true;
    atomicOr(status, (uint32_t)UNCOMP_STATUS_BOUNDS);
    return false;
}
#define UNCOMP_INDEX_OK(i, extent, status) (::uncomp::debug_index_ok((int64_t)(i), (int64_t)(extent), (status)))
#else
#define UNCOMP_INDEX_OK(i, extent, status) (true)
#endif

__device__ __forceinline__ float to_float(float x) { return x; }
__device__ __forceinline__ float to_float(__nv_bfloat16 x) { return __bfloat162float(x); }

__device__ __forceinline__ double warp_sum(double v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    return v;
}
__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    return v;
}

// Optional per-kernel timing with CUDA events on the launching stream (host objects only).
enum Slot { kSlotGram = 0, kSlotEigen, kSlotBudgets, kSlotScoreStats, kSlotStatsMerge, kSlotScoreColsum,
            kSlotPoolSelect, kSlotCompact, kSlotGramStats, kSlotEvictLogits, kSlotEvictScores, kSlotEvictGather,
            kSlotDecodeLogits, kSlotDecodeAccumulate, kSlotDecodeCommit, kSlotPrepareVote,
            kSlotPrepareFinish, kSlotWideGram, kSlotWideAssemble, kSlotWideTridiag, kSlotWideSturm, kSlotGramColsum, kSlotCount };
enum { kScorePhaseStats = 1, kScorePhaseColsum = 2 };
struct Profiler;
void prof_begin(Profiler *p, int slot, cudaStream_t st);
void prof_end(Profiler *p, cudaStream_t st);
struct ProfScope {
    Profiler *p; cudaStream_t st;
    ProfScope(Profiler *p_, int slot, cudaStream_t st_) : p(p_), st(st_) { if (p) prof_begin(p, slot, st); }
    ~ProfScope() { if (p) prof_end(p, st); }
};

// ---- kernel launchers (each returns the cudaError_t of its launches) -------------------------------
cudaError_t launch_gram_simt(const Plan &p, const void *dK, const UnitAddr &addr, void *d_partials, cudaStream_t st);
cudaError_t launch_gram_tc(const Plan &p, const void *dK, const UnitAddr &addr, void *d_partials, uint32_t *d_status,
                           cudaStream_t st);
cudaError_t launch_eigen_entropy(const Plan &p, const void *d_partials, const uncomp_entropy_params &ep,
                                 float *d_entropy, float *d_erank, double *d_spectrum, uint32_t *d_status,
                                 cudaStream_t st);
cudaError_t launch_eigen_f32(const Plan &p, const void *d_partials, int partials_per_unit, const uncomp_entropy_params &ep,
                             float *d_entropy, float *d_erank, double *d_spectrum, uint32_t *d_status, cudaStream_t st);
cudaError_t launch_gram_reduce(const Plan &p, const void *d_partials, double *d_out, cudaStream_t st);
int check_budget_params(const uncomp_shape &s, const uncomp_budget_params &bp);
cudaError_t launch_budgets(const Plan &p, const float *d_erank, const uncomp_budget_params &bp, int32_t *d_budgets,
                           int64_t *d_offsets, int32_t *d_layer_group, int32_t *d_layer_ctx, int32_t *d_rank,
                           int64_t *d_rem, cudaStream_t st);
// d_lse != NULL: the caller's log-sum-exp per window row replaces the statistics pass and the merge
cudaError_t launch_scores_simt(const Plan &p, const void *dQw, const void *dK, const UnitAddr &addr, float scale,
                               const float *d_lse, float *d_stats_part, float *d_stats, float *d_raw,
                               uint32_t *d_status, Profiler *prof, cudaStream_t st);
// Caller-supplied ln-sum-exp [units, rows] -> the merged statistics the column-sum kernels read: m' = lse * log2(e)
// per row (log2_domain, tensor-core kernels) or the pair (lse, 1) (CUDA-core kernels).  A non-finite entry raises
// UNCOMP_STATUS_NONFINITE and becomes +inf, so that its row adds nothing.
cudaError_t launch_lse_import(const Plan &p, const float *d_lse, float *d_stats, bool log2_domain, uint32_t *d_status,
                              cudaStream_t st);
struct TmapCache;
// phases: kScorePhaseStats (pass A; with d_gram_part != NULL the Gram partials of every (unit, scorer chunk) are
// produced in the same sweep) and / or kScorePhaseColsum (merge, or the import of d_lse when given, + pass B).
// kScorePhaseColsum alone with d_gram_part != NULL: pass B and the Gram partials from one sweep (needs d_lse).
cudaError_t launch_scores_tc(const Plan &p, const void *dQw, const void *dK, const UnitAddr &addr, float scale,
                             const float *d_lse, float *d_stats_part, float *d_stats, float *d_raw, float *d_gram_part,
                             int phases, uint32_t *d_status, TmapCache *cache, Profiler *prof, cudaStream_t st);
cudaError_t launch_pool_select(const Plan &p, const float *d_raw, float *d_pooled, int pool_kernel, int pool_mode,
                               const int32_t *d_budgets, const int64_t *d_offsets, int32_t *d_indices,
                               uint32_t *d_status, cudaStream_t st);
int evict_chunks(const uncomp_shape &s);
cudaError_t launch_evict_hidden(const Plan &p, const void *d_qlast, const void *d_K, int64_t sB, int64_t sH, int64_t sN,
                                const void *d_X, int64_t row_bytes, int n_keep, float scale, float *d_logits,
                                float *d_stats, float *d_raw, int32_t *d_budgets, int64_t *d_offsets, float *d_scores,
                                int32_t *d_indices, void *d_Xout, uint32_t *d_status, Profiler *prof, cudaStream_t st);
cudaError_t launch_decode_seed(const Plan &p, const float *d_scores, const int32_t *d_indices, const int64_t *d_offsets,
                               float *d_cum, cudaStream_t st);
int decode_chunks(int max_cap);
size_t decode_partial_bytes();
cudaError_t launch_decode_update(const Plan &p, const void *d_q, const void *d_knew, const void *d_vnew,
                                 const int32_t *d_new_pos, const int64_t *d_offsets, int32_t *d_lens, int max_cap,
                                 int protect, float scale, void *d_Kc, void *d_Vc, int32_t *d_pos, float *d_cum,
                                 float *d_p, int32_t *d_evicted, float *d_logits, float *d_stats, void *d_partial,
                                 float *d_new_cum, uint32_t *d_status, Profiler *prof, cudaStream_t st);
cudaError_t launch_retrieval_layer(const float *d_values, int L, int H, int32_t *d_layer, float *d_increase,
                                   cudaStream_t st);
cudaError_t launch_prepare_groups(const float *d_erank, int S, int L, int H, int M, int scope, float *d_mean,
                                  int32_t *d_group_mean, int32_t *d_votes, int32_t *d_group_vote, Profiler *prof,
                                  cudaStream_t st);
size_t entropy_wide_scratch_bytes(int N, int D);
cudaError_t launch_entropy_wide(const void *d_X, int64_t sN, int N, int D, const uncomp_entropy_params &ep,
                                unsigned char *scratch, float *d_entropy, float *d_erank, double *d_spectrum,
                                uint32_t *d_status, Profiler *prof, cudaStream_t st);
cudaError_t launch_l2_sweep(float *d_A, int rows, int cols, int passes, cudaStream_t st);
cudaError_t launch_compact(const Plan &p, const void *dK, const void *dV, const UnitAddr &aK, const UnitAddr &aV,
                           const int32_t *d_indices, const int64_t *d_offsets, void *dKc, void *dVc,
                           uint32_t *d_status, cudaStream_t st);

}  // namespace uncomp
