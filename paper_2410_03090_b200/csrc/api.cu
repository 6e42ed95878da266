// Host side of the C ABI declared in include/uncomp.h: argument checks, the workspace plan and the
// kernel launches of the four calls.  No device memory is allocated here.
#include <math.h>
#include <new>
#include <vector>

#include "tc_common.cuh"

namespace uncomp {

static size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

static bool shape_ok(const uncomp_shape &s) {
    if (s.B < 1 || s.L < 1 || s.H < 1 || s.Hq < 1 || s.N < 2) return false;
    if (s.d != kD) return false;
    if (s.Hq % s.H != 0) return false;
    if (s.w < 1 || s.w > 64 || s.w >= s.N) return false;
    if ((s.Hq / s.H) * s.w > kMaxRows) return false;
    if (s.dtype != UNCOMP_BF16 && s.dtype != UNCOMP_FP32) return false;
    if ((int64_t)s.B * s.L * s.H > (1 << 20)) return false;
    if (s.N > (1 << 24)) return false;
    return true;
}

Plan make_plan(const uncomp_shape &s) {
    Plan p;
    p.shape = s;
    p.units = s.B * s.L * s.H;
    p.G = s.Hq / s.H;
    p.rows = p.G * s.w;
    p.prefix = s.N - s.w;
    // Four CTAs per SM of the target part.  The plan (and with it the workspace size) must not depend on the
    // device that happens to be present: uncomp_workspace_bytes is a pure host function.
    const int target_ctas = 4 * kTargetSms;
    {
        int want = (target_ctas + p.units - 1) / p.units;
        int most = (s.N + 1023) / 1024;
        int P = want < 1 ? 1 : (want > most ? most : want);
        int chunk = (int)align_up((size_t)(s.N + P - 1) / P, 128);
        p.gram_chunk = chunk;
        p.gram_splits = (s.N + chunk - 1) / chunk;
    }
    {
        // scorer: chunks of 8192 tokens (a multiple of the 128-token tile), halved while the grid is small
        int chunk = 8192;
        while (chunk > 512 && (int64_t)p.units * ((s.N + chunk - 1) / chunk) < target_ctas) chunk >>= 1;
        p.score_chunk = chunk;
        p.score_splits = (s.N + chunk - 1) / chunk;
    }
    const size_t acc = s.dtype == UNCOMP_FP32 ? sizeof(double) : sizeof(float);
    size_t o = 0;
    p.off_status = o;      o = align_up(o + 256, 256);
    const int gram_parts = p.gram_splits > p.score_splits ? p.gram_splits : p.score_splits;   // fused path: one per scorer chunk
    p.off_gram = o;        o = align_up(o + (size_t)p.units * gram_parts * (kD * kD + kD) * acc, 256);
    p.off_stats_part = o;  o = align_up(o + (size_t)p.units * p.score_splits * 2 * kMaxRows * 2 * sizeof(float), 256);
    p.off_stats = o;       o = align_up(o + (size_t)p.units * kMaxRows * 2 * sizeof(float), 256);
    p.off_raw = o;         o = align_up(o + (size_t)p.units * p.prefix * sizeof(float), 256);
    p.off_pooled = o;      o = align_up(o + (size_t)p.units * p.prefix * sizeof(float), 256);
    p.off_rank = o;        o = align_up(o + (size_t)p.units * sizeof(int32_t), 256);
    p.off_rem = o;         o = align_up(o + (size_t)p.units * sizeof(int64_t), 256);
    p.off_ev_logits = o;   o = align_up(o + (size_t)s.B * s.Hq * s.N * sizeof(float), 256);
    p.off_ev_stats = o;    o = align_up(o + (size_t)s.B * s.Hq * evict_chunks(s) * 2 * sizeof(float), 256);
    p.off_ev_raw = o;      o = align_up(o + (size_t)s.B * s.N * sizeof(float), 256);
    p.off_ev_pooled = o;   o = align_up(o + (size_t)s.B * s.N * sizeof(float), 256);
    p.off_ev_budgets = o;  o = align_up(o + (size_t)s.B * sizeof(int32_t), 256);
    p.off_ev_offsets = o;  o = align_up(o + (size_t)(s.B + 1) * sizeof(int64_t), 256);
    p.off_dec_stats = o;   o = align_up(o + (size_t)p.units * decode_chunks(s.N) * 16 * 2 * sizeof(float), 256);
    p.off_dec_part = o;    o = align_up(o + (size_t)p.units * decode_chunks(s.N) * decode_partial_bytes(), 256);
    p.off_dec_new = o;     o = align_up(o + (size_t)p.units * sizeof(float), 256);
    p.bytes = o;
    return p;
}

// Per-kernel timing: one (start, stop) event pair per launch, appended while profiling is on.
struct Profiler {
    struct Rec { int slot; cudaEvent_t start, stop; };
    std::vector<Rec> recs;     // records in use
    std::vector<Rec> pool;     // event pairs created earlier, reused after a reset
    static constexpr size_t kMaxRecs = 1 << 16;
};

void prof_begin(Profiler *p, int slot, cudaStream_t st) {
    if (p->recs.size() >= Profiler::kMaxRecs) return;
    Profiler::Rec r;
    if (!p->pool.empty()) { r = p->pool.back(); p->pool.pop_back(); }
    else {
        if (cudaEventCreate(&r.start) != cudaSuccess) return;
        if (cudaEventCreate(&r.stop) != cudaSuccess) { cudaEventDestroy(r.start); return; }
    }
    r.slot = slot;
    cudaEventRecord(r.start, st);
    p->recs.push_back(r);
}

void prof_end(Profiler *p, cudaStream_t st) {
    if (!p->recs.empty()) cudaEventRecord(p->recs.back().stop, st);
}

}  // namespace uncomp

using namespace uncomp;

struct uncomp_ctx {
    Plan plan;
    unsigned char *ws;
    int last_cuda;
    int device;
    Profiler *prof;   // NULL unless profiling is on
    Profiler prof_store;
    int force_simt;   // UNCOMP_OPT_CUDA_CORES
    // row statistics left in the workspace by a fused uncomp_entropy call, valid for exactly these inputs
    int stats_valid;
    const void *stats_K, *stats_Qw;
    uncomp_strides stats_sK;
    float stats_scale;
    TmapCache tmaps;  // tensor maps of the last key / query tensors the scorer saw
    // second stream and fork / join events of uncomp_compress (host objects, created on first use)
    cudaStream_t side;
    cudaEvent_t ev_fork, ev_join;
    int side_ready;
};

// Host objects only: a non-blocking stream and two events without timing.
static cudaError_t ensure_side_stream(uncomp_ctx *ctx) {
    if (ctx->side_ready) return cudaSuccess;
    cudaError_t e = cudaStreamCreateWithFlags(&ctx->side, cudaStreamNonBlocking);
    if (e != cudaSuccess) return e;
    e = cudaEventCreateWithFlags(&ctx->ev_fork, cudaEventDisableTiming);
    if (e != cudaSuccess) { cudaStreamDestroy(ctx->side); return e; }
    e = cudaEventCreateWithFlags(&ctx->ev_join, cudaEventDisableTiming);
    if (e != cudaSuccess) { cudaEventDestroy(ctx->ev_fork); cudaStreamDestroy(ctx->side); return e; }
    ctx->side_ready = 1;
    return cudaSuccess;
}

static int cuda_fail(uncomp_ctx *ctx, cudaError_t e) {
    ctx->last_cuda = (int)e;
    return UNCOMP_E_CUDA;
}

static bool aligned16(const void *p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

static int check_strides(const uncomp_shape &s, const uncomp_strides &st) {
    const int64_t eb = s.dtype == UNCOMP_FP32 ? 4 : 2;
    const int64_t v[4] = {st.sB, st.sL, st.sH, st.sN};
    for (int i = 0; i < 4; ++i) {
        if (v[i] < 0) return UNCOMP_E_SHAPE;
        if ((v[i] * eb) % 16 != 0) return UNCOMP_E_ALIGN;
    }
    if (st.sN < s.d) return UNCOMP_E_SHAPE;
    return UNCOMP_OK;
}

extern "C" {

int uncomp_version(void) { return 100; }

const char *uncomp_strerror(int code) {
    switch (code) {
        case UNCOMP_OK: return "ok";
        case UNCOMP_E_NULL: return "a required pointer is NULL";
        case UNCOMP_E_SHAPE: return "unsupported shape or stride";
        case UNCOMP_E_ALIGN: return "pointer or stride is not 16-byte aligned";
        case UNCOMP_E_WORKSPACE: return "workspace too small or misaligned";
        case UNCOMP_E_PARAM: return "invalid hyper-parameter";
        case UNCOMP_E_CUDA: return "CUDA call failed";
        case UNCOMP_E_LIMIT: return "size beyond a documented maximum";
        default: return "unknown error code";
    }
}

size_t uncomp_workspace_bytes(const uncomp_shape *shape) {
    if (!shape || !shape_ok(*shape)) return 0;
    return make_plan(*shape).bytes;
}

int uncomp_create(uncomp_ctx **out, const uncomp_shape *shape, void *d_workspace, size_t workspace_bytes) {
    if (!out || !shape || !d_workspace) return UNCOMP_E_NULL;
    *out = nullptr;
    if (!shape_ok(*shape)) return UNCOMP_E_SHAPE;
    Plan p = make_plan(*shape);
    if (workspace_bytes < p.bytes || (reinterpret_cast<uintptr_t>(d_workspace) & 255u)) return UNCOMP_E_WORKSPACE;
    uncomp_ctx *ctx = new (std::nothrow) uncomp_ctx;
    if (!ctx) return UNCOMP_E_LIMIT;
    ctx->plan = p;
    ctx->ws = static_cast<unsigned char *>(d_workspace);
    ctx->last_cuda = 0;
    ctx->device = 0;
    ctx->prof = nullptr;
    ctx->force_simt = 0;
    ctx->stats_valid = 0;
    ctx->tmaps.k_valid = ctx->tmaps.q_valid = false;
    ctx->side_ready = 0;
    cudaError_t e = cudaGetDevice(&ctx->device);
    if (e == cudaSuccess) e = cudaMemset(ctx->ws + p.off_status, 0, 256);
    if (e == cudaSuccess) e = cudaDeviceSynchronize();
    if (e != cudaSuccess) {
        delete ctx;
        return UNCOMP_E_CUDA;
    }
    *out = ctx;
    return UNCOMP_OK;
}

void uncomp_destroy(uncomp_ctx *ctx) {
    if (!ctx) return;
    for (auto &r : ctx->prof_store.recs) { cudaEventDestroy(r.start); cudaEventDestroy(r.stop); }
    for (auto &r : ctx->prof_store.pool) { cudaEventDestroy(r.start); cudaEventDestroy(r.stop); }
    if (ctx->side_ready) {
        cudaEventDestroy(ctx->ev_fork);
        cudaEventDestroy(ctx->ev_join);
        cudaStreamDestroy(ctx->side);
    }
    delete ctx;
}

int uncomp_set_option(uncomp_ctx *ctx, int option, int value) {
    if (!ctx) return UNCOMP_E_NULL;
    if (option == UNCOMP_OPT_CUDA_CORES) {
        ctx->force_simt = value != 0;
        ctx->stats_valid = 0;      // the two kernel families keep their statistics in different formats
        return UNCOMP_OK;
    }
    return UNCOMP_E_PARAM;
}

int uncomp_profile_enable(uncomp_ctx *ctx, int on) {
    if (!ctx) return UNCOMP_E_NULL;
    ctx->prof = on ? &ctx->prof_store : nullptr;
    return UNCOMP_OK;
}

int uncomp_profile_slots(void) { return kSlotCount; }

const char *uncomp_profile_slot_name(int slot) {
    static const char *names[kSlotCount] = {"gram", "eigen_entropy", "budgets", "score_stats", "stats_merge",
                                            "score_colsum", "pool_select", "compact", "gram_score_stats",
                                            "evict_logits", "evict_scores", "evict_gather",
                                            "decode_logits", "decode_accumulate", "decode_commit",
                                            "prepare_vote", "prepare_finish",
                                            "wide_gram", "wide_assemble", "wide_tridiag", "wide_eigen_entropy",
                                            "gram_score_colsum"};
    return slot >= 0 && slot < kSlotCount ? names[slot] : "";
}

int uncomp_profile_read(uncomp_ctx *ctx, int max_slots, float *ms_sum, int32_t *launches) {
    if (!ctx || !ms_sum || !launches) return UNCOMP_E_NULL;
    for (int i = 0; i < max_slots; ++i) { ms_sum[i] = 0.f; launches[i] = 0; }
    Profiler &P = ctx->prof_store;
    for (auto &r : P.recs) {
        cudaError_t e = cudaEventSynchronize(r.stop);
        float ms = 0.f;
        if (e == cudaSuccess) e = cudaEventElapsedTime(&ms, r.start, r.stop);
        if (e != cudaSuccess) return cuda_fail(ctx, e);
        if (r.slot < max_slots) { ms_sum[r.slot] += ms; launches[r.slot] += 1; }
        P.pool.push_back(r);
    }
    P.recs.clear();
    return UNCOMP_OK;
}

int uncomp_last_cuda_error(const uncomp_ctx *ctx) { return ctx ? ctx->last_cuda : 0; }

static float effective_scale(float scale, int d) { return scale > 0.f ? scale : 1.0f / sqrtf((float)d); }

static bool same_strides(const uncomp_strides &a, const uncomp_strides &b) {
    return a.sB == b.sB && a.sL == b.sL && a.sH == b.sH && a.sN == b.sN;
}

int uncomp_entropy(uncomp_ctx *ctx, const void *d_K, uncomp_strides sK, const uncomp_entropy_params *params,
                   const void *d_Qw, float scale, float *d_entropy, float *d_erank, double *d_spectrum,
                   void *stream) {
    if (!ctx || !d_K || !params || !d_entropy) return UNCOMP_E_NULL;
    const Plan &p = ctx->plan;
    if (!aligned16(d_K) || (d_Qw && !aligned16(d_Qw))) return UNCOMP_E_ALIGN;
    int rc = check_strides(p.shape, sK);
    if (rc != UNCOMP_OK) return rc;
    if (params->k_trunc < 1 || params->max_iters < 0 || (params->center != 0 && params->center != 1) ||
        (params->norm != 0 && params->norm != 1) || !(scale >= 0.f) || isinf(scale))
        return UNCOMP_E_PARAM;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    uint32_t *d_status = reinterpret_cast<uint32_t *>(ctx->ws + p.off_status);
    void *partials = ctx->ws + p.off_gram;
    const UnitAddr addr = make_addr(p.shape, sK);
    const bool tensor_path = p.shape.dtype == UNCOMP_BF16 && !ctx->force_simt;
    ctx->stats_valid = 0;
    cudaError_t e;
    int parts = p.gram_splits;
    if (tensor_path && d_Qw) {
        // one sweep over K: Gram partials per scorer chunk and the scorer's row statistics
        const float sc = effective_scale(scale, p.shape.d);
        e = launch_scores_tc(p, d_Qw, d_K, addr, sc, nullptr, reinterpret_cast<float *>(ctx->ws + p.off_stats_part),
                             reinterpret_cast<float *>(ctx->ws + p.off_stats), nullptr,
                             reinterpret_cast<float *>(partials), kScorePhaseStats, d_status, &ctx->tmaps, ctx->prof, st);
        if (e != cudaSuccess) return cuda_fail(ctx, e);
        parts = p.score_splits;
        ctx->stats_valid = 1;
        ctx->stats_K = d_K;
        ctx->stats_Qw = d_Qw;
        ctx->stats_sK = sK;
        ctx->stats_scale = sc;
    } else {
        ProfScope ps(ctx->prof, kSlotGram, st);
        if (tensor_path) e = launch_gram_tc(p, d_K, addr, partials, d_status, st);
        else e = launch_gram_simt(p, d_K, addr, partials, st);
        if (e != cudaSuccess) return cuda_fail(ctx, e);
    }
    {
        ProfScope ps(ctx->prof, kSlotEigen, st);
        if (tensor_path)
            e = launch_eigen_f32(p, partials, parts, *params, d_entropy, d_erank, d_spectrum, d_status, st);
        else
            e = launch_eigen_entropy(p, partials, *params, d_entropy, d_erank, d_spectrum, d_status, st);
    }
    if (e != cudaSuccess) return cuda_fail(ctx, e);
    return UNCOMP_OK;
}

int uncomp_gram(uncomp_ctx *ctx, const void *d_K, uncomp_strides sK, double *d_gram, void *stream) {
    if (!ctx || !d_K || !d_gram) return UNCOMP_E_NULL;
    const Plan &p = ctx->plan;
    if (!aligned16(d_K)) return UNCOMP_E_ALIGN;
    int rc = check_strides(p.shape, sK);
    if (rc != UNCOMP_OK) return rc;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    uint32_t *d_status = reinterpret_cast<uint32_t *>(ctx->ws + p.off_status);
    void *partials = ctx->ws + p.off_gram;
    const UnitAddr addr = make_addr(p.shape, sK);
    cudaError_t e;
    if (p.shape.dtype == UNCOMP_BF16 && !ctx->force_simt) e = launch_gram_tc(p, d_K, addr, partials, d_status, st);
    else e = launch_gram_simt(p, d_K, addr, partials, st);
    if (e != cudaSuccess) return cuda_fail(ctx, e);
    e = launch_gram_reduce(p, partials, d_gram, st);
    if (e != cudaSuccess) return cuda_fail(ctx, e);
    return UNCOMP_OK;
}

int uncomp_assign_budgets(uncomp_ctx *ctx, const float *d_erank, const uncomp_budget_params *params,
                          int32_t *d_budgets, int64_t *d_offsets, int32_t *d_layer_group,
                          int32_t *d_layer_ctx, void *stream) {
    if (!ctx || !d_erank || !params || !d_budgets || !d_offsets) return UNCOMP_E_NULL;
    const Plan &p = ctx->plan;
    if (params->scope != 0 && params->scope != 1) return UNCOMP_E_PARAM;
    const int rc = check_budget_params(p.shape, *params);
    if (rc != UNCOMP_OK) return rc;
    if ((d_layer_group == nullptr) != (d_layer_ctx == nullptr)) return UNCOMP_E_NULL;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    cudaError_t e;
    {
        ProfScope ps(ctx->prof, kSlotBudgets, st);
        e = launch_budgets(p, d_erank, *params, d_budgets, d_offsets, d_layer_group, d_layer_ctx,
                           reinterpret_cast<int32_t *>(ctx->ws + p.off_rank),
                           reinterpret_cast<int64_t *>(ctx->ws + p.off_rem), st);
    }
    if (e != cudaSuccess) return cuda_fail(ctx, e);
    return UNCOMP_OK;
}

int uncomp_score_select(uncomp_ctx *ctx, const void *d_Qw, const void *d_K, uncomp_strides sK, const float *d_lse,
                        const int32_t *d_budgets, const int64_t *d_offsets, const uncomp_score_params *params,
                        float *d_scores, int32_t *d_indices, void *stream) {
    if (!ctx || !d_Qw || !d_K || !d_budgets || !d_offsets || !params || !d_indices) return UNCOMP_E_NULL;
    const Plan &p = ctx->plan;
    if (!aligned16(d_K) || !aligned16(d_Qw)) return UNCOMP_E_ALIGN;
    if (d_lse && (reinterpret_cast<uintptr_t>(d_lse) & 3u)) return UNCOMP_E_ALIGN;
    int rc = check_strides(p.shape, sK);
    if (rc != UNCOMP_OK) return rc;
    if (params->pool_kernel < 1 || params->pool_kernel > 63 || (params->pool_kernel & 1) == 0 ||
        (params->pool_mode != 0 && params->pool_mode != 1) || !(params->scale >= 0.f) || isinf(params->scale) ||
        (params->reuse_stats != 0 && params->reuse_stats != 1))
        return UNCOMP_E_PARAM;
    const float scale = effective_scale(params->scale, p.shape.d);
    const bool tensor_path = p.shape.dtype == UNCOMP_BF16 && !ctx->force_simt;
    // row statistics: supplied by the caller (d_lse), left by a fused uncomp_entropy call (reuse_stats), or
    // produced here by a statistics sweep of their own
    const bool reuse = !d_lse && params->reuse_stats && tensor_path && ctx->stats_valid && ctx->stats_K == d_K &&
                       ctx->stats_Qw == d_Qw && same_strides(ctx->stats_sK, sK) && ctx->stats_scale == scale;
    ctx->stats_valid = 0;          // every path below overwrites the statistics region or consumes it
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    uint32_t *d_status = reinterpret_cast<uint32_t *>(ctx->ws + p.off_status);
    float *stats_part = reinterpret_cast<float *>(ctx->ws + p.off_stats_part);
    float *stats = reinterpret_cast<float *>(ctx->ws + p.off_stats);
    float *raw = reinterpret_cast<float *>(ctx->ws + p.off_raw);
    float *pooled = d_scores ? d_scores : reinterpret_cast<float *>(ctx->ws + p.off_pooled);
    const UnitAddr addr = make_addr(p.shape, sK);
    cudaError_t e;
    if (tensor_path) {
        const int phases = (reuse || d_lse) ? kScorePhaseColsum : (kScorePhaseStats | kScorePhaseColsum);
        e = launch_scores_tc(p, d_Qw, d_K, addr, scale, d_lse, stats_part, stats, raw, nullptr, phases, d_status,
                             &ctx->tmaps, ctx->prof, st);
    } else {
        e = launch_scores_simt(p, d_Qw, d_K, addr, scale, d_lse, stats_part, stats, raw, d_status, ctx->prof, st);
    }
    if (e != cudaSuccess) return cuda_fail(ctx, e);
    {
        ProfScope ps(ctx->prof, kSlotPoolSelect, st);
        e = launch_pool_select(p, raw, pooled, params->pool_kernel, params->pool_mode, d_budgets, d_offsets,
                               d_indices, d_status, st);
    }
    if (e != cudaSuccess) return cuda_fail(ctx, e);
    return UNCOMP_OK;
}

int uncomp_compact(uncomp_ctx *ctx, const void *d_K, const void *d_V, uncomp_strides sK, uncomp_strides sV,
                   const int32_t *d_indices, const int64_t *d_offsets, void *d_Kc, void *d_Vc, void *stream) {
    if (!ctx || !d_K || !d_V || !d_indices || !d_offsets || !d_Kc || !d_Vc) return UNCOMP_E_NULL;
    const Plan &p = ctx->plan;
    if (!aligned16(d_K) || !aligned16(d_V) || !aligned16(d_Kc) || !aligned16(d_Vc)) return UNCOMP_E_ALIGN;
    int rc = check_strides(p.shape, sK);
    if (rc != UNCOMP_OK) return rc;
    rc = check_strides(p.shape, sV);
    if (rc != UNCOMP_OK) return rc;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    cudaError_t e;
    {
        ProfScope ps(ctx->prof, kSlotCompact, st);
        e = launch_compact(p, d_K, d_V, make_addr(p.shape, sK), make_addr(p.shape, sV), d_indices, d_offsets, d_Kc,
                           d_Vc, reinterpret_cast<uint32_t *>(ctx->ws + p.off_status), st);
    }
    if (e != cudaSuccess) return cuda_fail(ctx, e);
    return UNCOMP_OK;
}

int uncomp_compress(uncomp_ctx *ctx, const void *d_K, const void *d_V, uncomp_strides sK, uncomp_strides sV,
                    const void *d_Qw, const float *d_lse, const uncomp_entropy_params *eparams,
                    const uncomp_budget_params *bparams, const uncomp_score_params *sparams, float *d_entropy,
                    float *d_erank, int32_t *d_budgets, int64_t *d_offsets, int32_t *d_layer_group, int32_t *d_layer_ctx,
                    float *d_scores, int32_t *d_indices, void *d_Kc, void *d_Vc, void *stream) {
    if (!ctx || !eparams || !bparams || !sparams || !d_erank) return UNCOMP_E_NULL;
    const Plan &p = ctx->plan;
    const bool tensor_path = p.shape.dtype == UNCOMP_BF16 && !ctx->force_simt;
    int rc;
    if (d_lse && tensor_path) {
        // One sweep over K: the window scores (the caller brings the row normalisers) and the Gram partials of the
        // entropy stage come out of the same kernel; then eigenvalues, budgets, selection, gather.
        if (!d_K || !d_Qw || !d_entropy || !d_budgets || !d_offsets || !d_indices) return UNCOMP_E_NULL;
        if (!aligned16(d_K) || !aligned16(d_Qw) || (reinterpret_cast<uintptr_t>(d_lse) & 3u)) return UNCOMP_E_ALIGN;
        rc = check_strides(p.shape, sK);
        if (rc != UNCOMP_OK) return rc;
        if (eparams->k_trunc < 1 || eparams->max_iters < 0 || (eparams->center != 0 && eparams->center != 1) ||
            (eparams->norm != 0 && eparams->norm != 1))
            return UNCOMP_E_PARAM;
        if (sparams->pool_kernel < 1 || sparams->pool_kernel > 63 || (sparams->pool_kernel & 1) == 0 ||
            (sparams->pool_mode != 0 && sparams->pool_mode != 1) || !(sparams->scale >= 0.f) || isinf(sparams->scale))
            return UNCOMP_E_PARAM;
        if (bparams->scope != 0 && bparams->scope != 1) return UNCOMP_E_PARAM;
        rc = check_budget_params(p.shape, *bparams);
        if (rc != UNCOMP_OK) return rc;
        if ((d_layer_group == nullptr) != (d_layer_ctx == nullptr)) return UNCOMP_E_NULL;
        cudaStream_t st = static_cast<cudaStream_t>(stream);
        uint32_t *d_status = reinterpret_cast<uint32_t *>(ctx->ws + p.off_status);
        float *partials = reinterpret_cast<float *>(ctx->ws + p.off_gram);
        float *raw = reinterpret_cast<float *>(ctx->ws + p.off_raw);
        float *pooled = d_scores ? d_scores : reinterpret_cast<float *>(ctx->ws + p.off_pooled);
        const UnitAddr addr = make_addr(p.shape, sK);
        ctx->stats_valid = 0;
        cudaError_t e = launch_scores_tc(p, d_Qw, d_K, addr, effective_scale(sparams->scale, p.shape.d), d_lse,
                                         reinterpret_cast<float *>(ctx->ws + p.off_stats_part),
                                         reinterpret_cast<float *>(ctx->ws + p.off_stats), raw, partials, kScorePhaseColsum,
                                         d_status, &ctx->tmaps, ctx->prof, st);
        if (e != cudaSuccess) return cuda_fail(ctx, e);
        {
            ProfScope ps(ctx->prof, kSlotEigen, st);
            e = launch_eigen_f32(p, partials, p.score_splits, *eparams, d_entropy, d_erank, nullptr, d_status, st);
        }
        if (e != cudaSuccess) return cuda_fail(ctx, e);
        {
            ProfScope ps(ctx->prof, kSlotBudgets, st);
            e = launch_budgets(p, d_erank, *bparams, d_budgets, d_offsets, d_layer_group, d_layer_ctx,
                               reinterpret_cast<int32_t *>(ctx->ws + p.off_rank),
                               reinterpret_cast<int64_t *>(ctx->ws + p.off_rem), st);
        }
        if (e != cudaSuccess) return cuda_fail(ctx, e);
        {
            ProfScope ps(ctx->prof, kSlotPoolSelect, st);
            e = launch_pool_select(p, raw, pooled, sparams->pool_kernel, sparams->pool_mode, d_budgets, d_offsets,
                                   d_indices, d_status, st);
        }
        if (e != cudaSuccess) return cuda_fail(ctx, e);
    } else if (tensor_path) {
        // Gram + statistics sweep; then eigenvalues and budgets on a second stream beside the merge and the column
        // sums: neither needs the other, only the selection needs both.  The eigenvalue kernel is a chain of
        // dependent steps that leaves most of an SM idle; beside the column sums it costs little (measured against
        // the staged order: 0.51 ms instead of 0.59 ms at 8K tokens, 1.88 instead of 1.93 ms at 32K tokens, no
        // change with four 32K-token sequences).
        if (!d_K || !d_Qw || !d_entropy || !d_budgets || !d_offsets || !d_indices) return UNCOMP_E_NULL;
        if (!aligned16(d_K) || !aligned16(d_Qw)) return UNCOMP_E_ALIGN;
        rc = check_strides(p.shape, sK);
        if (rc != UNCOMP_OK) return rc;
        if (eparams->k_trunc < 1 || eparams->max_iters < 0 || (eparams->center != 0 && eparams->center != 1) ||
            (eparams->norm != 0 && eparams->norm != 1))
            return UNCOMP_E_PARAM;
        if (sparams->pool_kernel < 1 || sparams->pool_kernel > 63 || (sparams->pool_kernel & 1) == 0 ||
            (sparams->pool_mode != 0 && sparams->pool_mode != 1) || !(sparams->scale >= 0.f) || isinf(sparams->scale))
            return UNCOMP_E_PARAM;
        if (bparams->scope != 0 && bparams->scope != 1) return UNCOMP_E_PARAM;
        rc = check_budget_params(p.shape, *bparams);
        if (rc != UNCOMP_OK) return rc;
        if ((d_layer_group == nullptr) != (d_layer_ctx == nullptr)) return UNCOMP_E_NULL;
        cudaStream_t st = static_cast<cudaStream_t>(stream);
        cudaError_t e = ensure_side_stream(ctx);
        if (e != cudaSuccess) return cuda_fail(ctx, e);
        uint32_t *d_status = reinterpret_cast<uint32_t *>(ctx->ws + p.off_status);
        float *partials = reinterpret_cast<float *>(ctx->ws + p.off_gram);
        float *stats_part = reinterpret_cast<float *>(ctx->ws + p.off_stats_part);
        float *stats = reinterpret_cast<float *>(ctx->ws + p.off_stats);
        float *raw = reinterpret_cast<float *>(ctx->ws + p.off_raw);
        float *pooled = d_scores ? d_scores : reinterpret_cast<float *>(ctx->ws + p.off_pooled);
        const UnitAddr addr = make_addr(p.shape, sK);
        const float sc = effective_scale(sparams->scale, p.shape.d);
        ctx->stats_valid = 0;
        e = launch_scores_tc(p, d_Qw, d_K, addr, sc, nullptr, stats_part, stats, nullptr, partials, kScorePhaseStats,
                             d_status, &ctx->tmaps, ctx->prof, st);
        if (e == cudaSuccess) e = cudaEventRecord(ctx->ev_fork, st);
        if (e == cudaSuccess) e = cudaStreamWaitEvent(ctx->side, ctx->ev_fork, 0);
        if (e != cudaSuccess) return cuda_fail(ctx, e);
        {
            ProfScope ps(ctx->prof, kSlotEigen, ctx->side);
            e = launch_eigen_f32(p, partials, p.score_splits, *eparams, d_entropy, d_erank, nullptr, d_status, ctx->side);
        }
        if (e != cudaSuccess) return cuda_fail(ctx, e);
        {
            ProfScope ps(ctx->prof, kSlotBudgets, ctx->side);
            e = launch_budgets(p, d_erank, *bparams, d_budgets, d_offsets, d_layer_group, d_layer_ctx,
                               reinterpret_cast<int32_t *>(ctx->ws + p.off_rank),
                               reinterpret_cast<int64_t *>(ctx->ws + p.off_rem), ctx->side);
        }
        if (e == cudaSuccess) e = cudaEventRecord(ctx->ev_join, ctx->side);
        if (e != cudaSuccess) return cuda_fail(ctx, e);
        e = launch_scores_tc(p, d_Qw, d_K, addr, sc, nullptr, stats_part, stats, raw, nullptr, kScorePhaseColsum, d_status,
                             &ctx->tmaps, ctx->prof, st);
        if (e == cudaSuccess) e = cudaStreamWaitEvent(st, ctx->ev_join, 0);
        if (e != cudaSuccess) return cuda_fail(ctx, e);
        {
            ProfScope ps(ctx->prof, kSlotPoolSelect, st);
            e = launch_pool_select(p, raw, pooled, sparams->pool_kernel, sparams->pool_mode, d_budgets, d_offsets,
                                   d_indices, d_status, st);
        }
        if (e != cudaSuccess) return cuda_fail(ctx, e);
    } else {
        // the four calls back to back; bf16 keys without normalisers take the fused Gram + statistics sweep
        const bool fuse = tensor_path && !d_lse;
        rc = uncomp_entropy(ctx, d_K, sK, eparams, fuse ? d_Qw : nullptr, sparams->scale, d_entropy, d_erank, nullptr, stream);
        if (rc != UNCOMP_OK) return rc;
        rc = uncomp_assign_budgets(ctx, d_erank, bparams, d_budgets, d_offsets, d_layer_group, d_layer_ctx, stream);
        if (rc != UNCOMP_OK) return rc;
        uncomp_score_params sp = *sparams;
        sp.reuse_stats = fuse ? 1 : 0;
        rc = uncomp_score_select(ctx, d_Qw, d_K, sK, d_lse, d_budgets, d_offsets, &sp, d_scores, d_indices, stream);
        if (rc != UNCOMP_OK) return rc;
    }
    return uncomp_compact(ctx, d_K, d_V, sK, sV, d_indices, d_offsets, d_Kc, d_Vc, stream);
}

int uncomp_decode_seed(uncomp_ctx *ctx, const float *d_scores, const int32_t *d_indices, const int64_t *d_offsets,
                       float *d_cum, void *stream) {
    if (!ctx || !d_scores || !d_indices || !d_offsets || !d_cum) return UNCOMP_E_NULL;
    cudaError_t e = launch_decode_seed(ctx->plan, d_scores, d_indices, d_offsets, d_cum, static_cast<cudaStream_t>(stream));
    if (e != cudaSuccess) return cuda_fail(ctx, e);
    return UNCOMP_OK;
}

int uncomp_decode_update(uncomp_ctx *ctx, const void *d_qnew, const void *d_knew, const void *d_vnew,
                         const int32_t *d_new_pos, const int64_t *d_offsets, int32_t *d_lens, int32_t max_cap,
                         int64_t total_cap, int32_t protect, float scale, void *d_Kc, void *d_Vc, int32_t *d_pos,
                         float *d_cum, float *d_p, int32_t *d_evicted, void *stream) {
    if (!ctx || !d_qnew || !d_knew || !d_vnew || !d_new_pos || !d_offsets || !d_lens || !d_Kc || !d_Vc || !d_pos ||
        !d_cum)
        return UNCOMP_E_NULL;
    const Plan &p = ctx->plan;
    if (!aligned16(d_qnew) || !aligned16(d_knew) || !aligned16(d_vnew) || !aligned16(d_Kc) || !aligned16(d_Vc))
        return UNCOMP_E_ALIGN;
    if (p.G != 1 && p.G != 2 && p.G != 4 && p.G != 8 && p.G != 16) return UNCOMP_E_SHAPE;
    if (max_cap < 1 || max_cap > p.shape.N || total_cap < 1 || protect < 1 || !(scale >= 0.f) || isinf(scale))
        return UNCOMP_E_PARAM;
    // the logits of every entry live in the region the prefill pass uses for its raw and pooled scores
    if ((size_t)(total_cap + p.units) * p.G * sizeof(float) > p.off_rank - p.off_raw) return UNCOMP_E_LIMIT;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    cudaError_t e = launch_decode_update(
        p, d_qnew, d_knew, d_vnew, d_new_pos, d_offsets, d_lens, max_cap, protect, effective_scale(scale, p.shape.d),
        d_Kc, d_Vc, d_pos, d_cum, d_p, d_evicted, reinterpret_cast<float *>(ctx->ws + p.off_raw),
        reinterpret_cast<float *>(ctx->ws + p.off_dec_stats), ctx->ws + p.off_dec_part,
        reinterpret_cast<float *>(ctx->ws + p.off_dec_new), reinterpret_cast<uint32_t *>(ctx->ws + p.off_status),
        ctx->prof, st);
    if (e != cudaSuccess) return cuda_fail(ctx, e);
    return UNCOMP_OK;
}

int uncomp_eviction_plan(const int32_t *layer_group, const int32_t *layer_ctx, int32_t L, int32_t *out_layer,
                         int32_t *out_keep) {
    if (L < 0) return UNCOMP_E_PARAM;
    if (L == 0) return 0;
    if (!layer_group || !layer_ctx || !out_layer || !out_keep) return UNCOMP_E_NULL;
    int n = 0;
    int32_t current = layer_ctx[0];
    for (int32_t l = 1; l < L; ++l) {
        if (layer_group[l] != layer_group[l - 1] && layer_ctx[l] < current) {
            out_layer[n] = l;
            out_keep[n] = layer_ctx[l];
            current = layer_ctx[l];
            ++n;
        }
    }
    return n;
}

int uncomp_retrieval_layer(uncomp_ctx *ctx, const float *d_values, int32_t *d_layer, float *d_increase, void *stream) {
    if (!ctx || !d_values || !d_layer) return UNCOMP_E_NULL;
    const uncomp_shape &s = ctx->plan.shape;
    if (s.L < 2) return UNCOMP_E_SHAPE;
    if (s.L > 4096) return UNCOMP_E_LIMIT;
    cudaError_t e = launch_retrieval_layer(d_values, s.L, s.H, d_layer, d_increase, static_cast<cudaStream_t>(stream));
    if (e != cudaSuccess) return cuda_fail(ctx, e);
    return UNCOMP_OK;
}

int uncomp_prepare_groups(uncomp_ctx *ctx, const float *d_erank, int32_t S, int32_t M, int32_t scope, float *d_mean,
                          int32_t *d_group_mean, int32_t *d_votes, int32_t *d_group_vote, void *stream) {
    if (!ctx || !d_erank || !d_mean || !d_group_mean || !d_votes || !d_group_vote) return UNCOMP_E_NULL;
    const uncomp_shape &s = ctx->plan.shape;
    const int n = scope ? s.L * s.H : s.H;
    if (S < 1 || M < 1 || M > n || (scope != 0 && scope != 1)) return UNCOMP_E_PARAM;
    if (n > 8192 || S > 65535) return UNCOMP_E_LIMIT;
    cudaError_t e = launch_prepare_groups(d_erank, S, s.L, s.H, M, scope, d_mean, d_group_mean, d_votes, d_group_vote,
                                          ctx->prof, static_cast<cudaStream_t>(stream));
    if (e != cudaSuccess) return cuda_fail(ctx, e);
    return UNCOMP_OK;
}

size_t uncomp_entropy_wide_scratch_bytes(int32_t N, int32_t D) {
    if (N < 2 || D < 128 || D > 4096 || D % 64 != 0) return 0;
    return entropy_wide_scratch_bytes(N, D);
}

int uncomp_entropy_wide(uncomp_ctx *ctx, const void *d_X, int32_t count, int64_t stride_matrix, int64_t stride_row,
                        int32_t N, int32_t D, const uncomp_entropy_params *params, void *d_scratch, size_t scratch_bytes,
                        float *d_entropy, float *d_erank, double *d_spectrum, void *stream) {
    if (!ctx || !d_X || !params || !d_scratch || !d_entropy) return UNCOMP_E_NULL;
    if (ctx->plan.shape.dtype != UNCOMP_BF16) return UNCOMP_E_SHAPE;
    if (count < 1 || N < 2 || D < 128 || D % 64 != 0) return UNCOMP_E_SHAPE;
    if (D > 4096) return UNCOMP_E_LIMIT;
    if (!aligned16(d_X) || !aligned16(d_scratch) || ((uintptr_t)d_scratch & 255) != 0 || stride_row < D ||
        stride_row % 8 != 0 || stride_matrix % 8 != 0)
        return UNCOMP_E_ALIGN;
    if (params->k_trunc < 1 || params->k_trunc > 256 || (params->center != 0 && params->center != 1) ||
        (params->norm != 0 && params->norm != 1) || params->max_iters < 0)
        return UNCOMP_E_PARAM;
    if (scratch_bytes < entropy_wide_scratch_bytes(N, D)) return UNCOMP_E_WORKSPACE;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const int k = params->k_trunc < D ? params->k_trunc : D;
    for (int i = 0; i < count; ++i) {
        const unsigned char *Xi = static_cast<const unsigned char *>(d_X) + (size_t)i * stride_matrix * 2;
        cudaError_t e = launch_entropy_wide(Xi, stride_row, N, D, *params, static_cast<unsigned char *>(d_scratch),
                                            d_entropy + i, d_erank ? d_erank + i : nullptr,
                                            d_spectrum ? d_spectrum + (size_t)i * k : nullptr,
                                            reinterpret_cast<uint32_t *>(ctx->ws + ctx->plan.off_status), ctx->prof, st);
        if (e != cudaSuccess) return cuda_fail(ctx, e);
    }
    return UNCOMP_OK;
}

int uncomp_measure_l2_sweep(float *d_A, int32_t rows, int32_t cols, int32_t passes, void *stream) {
    if (!d_A) return UNCOMP_E_NULL;
    if (rows < 1 || cols < 4 || cols % 4 != 0 || passes < 1) return UNCOMP_E_PARAM;
    if (!aligned16(d_A)) return UNCOMP_E_ALIGN;
    return launch_l2_sweep(d_A, rows, cols, passes, static_cast<cudaStream_t>(stream)) == cudaSuccess ? UNCOMP_OK
                                                                                                       : UNCOMP_E_CUDA;
}

int uncomp_evict_hidden(uncomp_ctx *ctx, const void *d_qlast, const void *d_K, uncomp_strides sK, const void *d_X,
                        int32_t D, int32_t n_keep, float scale, float *d_scores, int32_t *d_indices, void *d_Xout,
                        void *stream) {
    if (!ctx || !d_qlast || !d_K || !d_X || !d_indices || !d_Xout) return UNCOMP_E_NULL;
    const Plan &p = ctx->plan;
    const int64_t eb = p.shape.dtype == UNCOMP_FP32 ? 4 : 2;
    if (!aligned16(d_qlast) || !aligned16(d_K) || !aligned16(d_X) || !aligned16(d_Xout)) return UNCOMP_E_ALIGN;
    int rc = check_strides(p.shape, sK);
    if (rc != UNCOMP_OK) return rc;
    if (D < 1 || ((int64_t)D * eb) % 16 != 0) return UNCOMP_E_ALIGN;
    if (p.G != 1 && p.G != 2 && p.G != 4 && p.G != 8 && p.G != 16) return UNCOMP_E_SHAPE;
    if (n_keep < 1 || n_keep > p.shape.N || !(scale >= 0.f) || isinf(scale)) return UNCOMP_E_PARAM;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    float *pooled = d_scores ? d_scores : reinterpret_cast<float *>(ctx->ws + p.off_ev_pooled);
    cudaError_t e = launch_evict_hidden(
        p, d_qlast, d_K, sK.sB, sK.sH, sK.sN, d_X, (int64_t)D * eb, n_keep, effective_scale(scale, p.shape.d),
        reinterpret_cast<float *>(ctx->ws + p.off_ev_logits), reinterpret_cast<float *>(ctx->ws + p.off_ev_stats),
        reinterpret_cast<float *>(ctx->ws + p.off_ev_raw), reinterpret_cast<int32_t *>(ctx->ws + p.off_ev_budgets),
        reinterpret_cast<int64_t *>(ctx->ws + p.off_ev_offsets), pooled, d_indices, d_Xout,
        reinterpret_cast<uint32_t *>(ctx->ws + p.off_status), ctx->prof, st);
    if (e != cudaSuccess) return cuda_fail(ctx, e);
    return UNCOMP_OK;
}

int uncomp_status(uncomp_ctx *ctx, void *stream, uint32_t *host_bits) {
    if (!ctx || !host_bits) return UNCOMP_E_NULL;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    uint32_t *d_status = reinterpret_cast<uint32_t *>(ctx->ws + ctx->plan.off_status);
    cudaError_t e = cudaMemcpyAsync(host_bits, d_status, sizeof(uint32_t), cudaMemcpyDeviceToHost, st);
    if (e == cudaSuccess) e = cudaMemsetAsync(d_status, 0, sizeof(uint32_t), st);
    if (e == cudaSuccess) e = cudaStreamSynchronize(st);
    if (e != cudaSuccess) return cuda_fail(ctx, e);
    return UNCOMP_OK;
}

}  // extern "C"
