/*
 * TEST INFRASTRUCTURE -- the slow, plain fp64 CPU oracle of the UNComp prefill-end KV compression pass.
 *
 * This file states, as directly as C allows, what each stage of the pass computes according to the
 * paper (UNComp, arXiv 2410.03090).  It is deliberately unblocked, unfused and single-threaded; it is
 * what the CUDA library is compared against and it is never part of the product path.  It shares no
 * code, header, table or helper with the CUDA library.
 *
 * Stages and the passages they follow:
 *   covariance            Section 3.1, Eq. 1 (centred); the uncentred X^T X form used in the proof of Lemma 3
 *   eigenvalues           symmetric eigenvalues by the classical cyclic Jacobi rotation method
 *   truncated entropy     Section 3.2, the definitions of H_k and erank_k; Lemma 2 (eigenvalue form);
 *                         Appendix "Proofs": unit trace, natural logarithm (erank = exp H)
 *   budgets               Section 3.3.3 ("Head-Group Compression", N_{i,g+1} = N_{i,g} - dn_g) and
 *                         Section 3.3.2 (layer-group partition: Delta c_i, C, N_{i+1} = N_i + dn)
 *   window scores         Section 3.3.3, "Dynamic KV Cache Eviction": attention of the last l query
 *                         positions summed per key position; the log-sum-exp of each of those rows
 *   selection             same paragraph: keep the highest-scored tokens within the head's budget; the
 *                         recent (window) tokens are part of the budget (Section 4, recent/historical split)
 *   hidden-state eviction Section 3.3.2, "Hidden State Eviction": tokens kept for the next layer group by
 *                         the last token's attention scores
 *   compaction            per-head ragged cache (Section 3.3.3, "each head maintains its context window");
 *                         K and V share one selection (Table 1 caption)
 *
 * Readings taken where the paper is silent or ambiguous are listed next to each function.
 * Parity pins: every function below is pinned by tests/test_oracle_*.py; the rounding rule for
 * non-integer budget steps has no counterpart in the paper ("parity unpinned" for that rule only).
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

/* ------------------------------------------------------------------------------------------------
 * Covariance, Eq. 1:  Sigma = 1/(N-1) * sum_i (x_i - mean)(x_i - mean)^T.
 * The factor 1/(N-1) is left out: every later use normalises the spectrum, where it cancels.
 * center = 0 gives the uncentred X^T X of the appendix proof.
 * X is [N, d] row-major; C is [d, d].
 * ---------------------------------------------------------------------------------------------- */
void oracle_covariance(const double *X, int N, int d, int center, double *C)
{
    double *mean = (double *)calloc((size_t)d, sizeof(double));
    double *row = (double *)malloc((size_t)d * sizeof(double));
    if (center) {
        for (int i = 0; i < N; ++i)
            for (int a = 0; a < d; ++a) mean[a] += X[(size_t)i * d + a];
        for (int a = 0; a < d; ++a) mean[a] /= (double)N;
    }
    memset(C, 0, (size_t)d * d * sizeof(double));
    for (int i = 0; i < N; ++i) {
        for (int a = 0; a < d; ++a) row[a] = X[(size_t)i * d + a] - mean[a];
        for (int a = 0; a < d; ++a) {
            const double ra = row[a];
            double *Ca = C + (size_t)a * d;
            for (int c = 0; c < d; ++c) Ca[c] += ra * row[c];
        }
    }
    free(mean);
    free(row);
}

/* ------------------------------------------------------------------------------------------------
 * Eigenvalues of a symmetric matrix by cyclic Jacobi: sweep over all pairs p < q, annihilating A[p][q]
 * with a plane rotation, until the off-diagonal Frobenius norm is below 1e-14 of the matrix norm.
 * A is destroyed.  lam receives the d eigenvalues sorted in descending order.  Returns the number of
 * sweeps used, or -1 if 100 sweeps did not reach the tolerance.
 * ---------------------------------------------------------------------------------------------- */
static int cmp_desc(const void *a, const void *b)
{
    const double x = *(const double *)a, y = *(const double *)b;
    return (x < y) - (x > y);
}

int oracle_jacobi_eigenvalues(double *A, int d, double *lam)
{
    double fro = 0.0;
    for (int i = 0; i < d * d; ++i) fro += A[i] * A[i];
    fro = sqrt(fro);
    int sweep = 0, converged = 0;
    for (; sweep < 100; ++sweep) {
        double off = 0.0;
        for (int p = 0; p < d; ++p)
            for (int q = 0; q < d; ++q)
                if (p != q) off += A[(size_t)p * d + q] * A[(size_t)p * d + q];
        if (sqrt(off) <= 1e-14 * fro || fro == 0.0) { converged = 1; break; }
        for (int p = 0; p < d - 1; ++p) {
            for (int q = p + 1; q < d; ++q) {
                const double apq = A[(size_t)p * d + q];
                if (apq == 0.0) continue;
                const double app = A[(size_t)p * d + p], aqq = A[(size_t)q * d + q];
                const double theta = (aqq - app) / (2.0 * apq);
                const double t = (theta >= 0.0 ? 1.0 : -1.0) / (fabs(theta) + sqrt(theta * theta + 1.0));
                const double c = 1.0 / sqrt(t * t + 1.0), s = t * c;
                /* A <- J^T A J with J the rotation in the (p,q) plane */
                for (int k = 0; k < d; ++k) {
                    const double akp = A[(size_t)k * d + p], akq = A[(size_t)k * d + q];
                    A[(size_t)k * d + p] = c * akp - s * akq;
                    A[(size_t)k * d + q] = s * akp + c * akq;
                }
                for (int k = 0; k < d; ++k) {
                    const double apk = A[(size_t)p * d + k], aqk = A[(size_t)q * d + k];
                    A[(size_t)p * d + k] = c * apk - s * aqk;
                    A[(size_t)q * d + k] = s * apk + c * aqk;
                }
            }
        }
    }
    for (int i = 0; i < d; ++i) lam[i] = A[(size_t)i * d + i];
    qsort(lam, (size_t)d, sizeof(double), cmp_desc);
    return converged ? sweep : -1;
}

/* ------------------------------------------------------------------------------------------------
 * Truncated matrix entropy and truncated effective rank (Section 3.2):
 *     H_k = - sum_{i<=k} p_i ln p_i ,   erank_k = exp(H_k)
 * over the k largest eigenvalues.  lam must be sorted descending.  Negative eigenvalues (round-off of
 * a positive semi-definite matrix) count as 0 and 0 ln 0 = 0.  k is clipped to d.
 *   norm = 0: p_i = lam_i / sum_{j<=k} lam_j   (the spectrum of the leading sub-matrix is normalised
 *             to unit trace; the reading under which an isotropic matrix gives H_k = ln k, as the
 *             bound H_k <= ln k of the appendix requires equality for)
 *   norm = 1: p_i = lam_i / sum_{j<=d} lam_j   (the whole covariance has unit trace, as the appendix
 *             states literally; the top-k terms of the full entropy sum)
 * ---------------------------------------------------------------------------------------------- */
void oracle_truncated_entropy(const double *lam, int d, int k, int norm, double *H, double *erank)
{
    if (k > d) k = d;
    double total = 0.0;
    const int m = norm ? d : k;
    for (int i = 0; i < m; ++i) total += lam[i] > 0.0 ? lam[i] : 0.0;
    double h = 0.0;
    if (total > 0.0) {
        for (int i = 0; i < k; ++i) {
            const double p = (lam[i] > 0.0 ? lam[i] : 0.0) / total;
            if (p > 0.0) h -= p * log(p);
        }
    }
    *H = h;
    *erank = exp(h);
}

/* One unit: token matrix X [N, d] -> H_k, erank_k (and, if lam_out != NULL, all d eigenvalues). */
int oracle_entropy(const double *X, int N, int d, int k_trunc, int center, int norm,
                   double *H, double *erank, double *lam_out)
{
    double *C = (double *)malloc((size_t)d * d * sizeof(double));
    double *lam = (double *)malloc((size_t)d * sizeof(double));
    oracle_covariance(X, N, d, center, C);
    const int sweeps = oracle_jacobi_eigenvalues(C, d, lam);
    oracle_truncated_entropy(lam, d, k_trunc, norm, H, erank);
    if (lam_out) memcpy(lam_out, lam, (size_t)d * sizeof(double));
    free(C);
    free(lam);
    return sweeps;
}

/* ------------------------------------------------------------------------------------------------
 * Head-group budgets (Section 3.3.3).
 *
 * Within each ranking set (the H heads of one layer of one sequence for scope = 0, all L*H heads of a
 * sequence for scope = 1; n = its size) heads are ranked by truncated effective rank, largest first
 * (equal values: lower (layer, head) index first), cut into M contiguous groups (ranks
 * [floor(g n / M), floor((g+1) n / M)) form group g, so sizes are equal when M divides n), and group g
 * receives the target
 *        t_g = n_max - g * step,      step = n (n_max - avg) / sum_g (n_g * g),
 * the paper's N_{i,g+1} = N_{i,g} - dn_g with the step chosen so that the budgets of the set add up to
 * n * avg (the paper fixes the average cache size per head; for equal groups step = 2 (n_max - avg)/(M-1)).
 * M = 1 gives every head avg.
 *
 * Integer budgets: every head first gets floor(t_g); the n*avg - sum floor(t_g) tokens still missing go,
 * one each, to the heads with the largest fractional part of t_g (equal fractions: better rank first).
 * t_g = num_g / S with num_g = n_max * S - g * n * (n_max - avg) and S = sum_g n_g * g, so floors and
 * fractional parts are exact integer quotients and remainders: no rounding error can move a budget.
 * (The paper prints integer schedules only; for non-integer steps its printed rows follow no single
 * rule, so this rounding rule is this implementation's own.)
 *
 * offsets = exclusive prefix sum of the budgets over units in (b, l, h) order, length units + 1.
 *
 * Layer-group partition (Section 3.3.2): e_l = mean over the layer's heads of erank; a group boundary
 * lies after layer l iff e_l - e_{l+1} > eps (the indicator of the paper's equation for C);
 * layer_group[l] = number of boundaries before l.  The first group keeps the full context N; with C_b
 * boundaries, group c >= 1 has context min(N, n_last + (C_b - c) * dn): the recurrence
 * N_{i+1} = N_i + dn read from the last (smallest) group backwards.  dn = 0 switches the partition
 * off: every layer is in group 0 with context N.
 *
 * Returns 0, or -1 if a precondition fails (M < 1, M > n, smallest target below w, n_max > N,
 * n_max < avg).
 * ---------------------------------------------------------------------------------------------- */
typedef struct { double key; int idx; } keyed_t;

static int cmp_key_desc_idx_asc(const void *a, const void *b)
{
    const keyed_t *x = (const keyed_t *)a, *y = (const keyed_t *)b;
    if (x->key > y->key) return -1;
    if (x->key < y->key) return 1;
    return (x->idx > y->idx) - (x->idx < y->idx);
}

typedef struct { int64_t rem; int rank; int idx; } frac_t;

static int cmp_rem_desc_rank_asc(const void *a, const void *b)
{
    const frac_t *x = (const frac_t *)a, *y = (const frac_t *)b;
    if (x->rem > y->rem) return -1;
    if (x->rem < y->rem) return 1;
    return (x->rank > y->rank) - (x->rank < y->rank);
}

int oracle_budgets(const double *erank, int B, int L, int H, int N, int w,
                   int avg, int M, int n_max, int scope, double eps, int dn, int n_last,
                   int32_t *budgets, int64_t *offsets, int32_t *layer_group, int32_t *layer_ctx)
{
    const int n = scope ? L * H : H;
    const int sets_per_seq = scope ? 1 : L;
    if (M < 1 || M > n || n_max > N || n_max < avg || avg < w) return -1;

    /* group sizes and the common denominator S */
    int64_t S = 0;
    for (int g = 0; g < M; ++g) {
        const int lo = (int)((int64_t)g * n / M), hi = (int)((int64_t)(g + 1) * n / M);
        S += (int64_t)(hi - lo) * g;
    }
    if (M > 1) {
        const int64_t num_last = (int64_t)n_max * S - (int64_t)(M - 1) * n * (n_max - avg);
        if (num_last < (int64_t)w * S) return -1;
    }

    keyed_t *order = (keyed_t *)malloc((size_t)n * sizeof(keyed_t));
    frac_t *fr = (frac_t *)malloc((size_t)n * sizeof(frac_t));
    for (int b = 0; b < B; ++b) {
        for (int s = 0; s < sets_per_seq; ++s) {
            const size_t base = ((size_t)b * L + (scope ? 0 : s)) * H;
            for (int i = 0; i < n; ++i) { order[i].key = erank[base + i]; order[i].idx = i; }
            qsort(order, (size_t)n, sizeof(keyed_t), cmp_key_desc_idx_asc);
            int64_t given = 0;
            for (int g = 0; g < M; ++g) {
                const int lo = (int)((int64_t)g * n / M), hi = (int)((int64_t)(g + 1) * n / M);
                int64_t fl, rem;
                if (M == 1) { fl = avg; rem = 0; }
                else {
                    const int64_t num = (int64_t)n_max * S - (int64_t)g * n * (n_max - avg);
                    fl = num / S;
                    rem = num % S;
                }
                for (int r = lo; r < hi; ++r) {
                    budgets[base + order[r].idx] = (int32_t)fl;
                    fr[r].rem = rem; fr[r].rank = r; fr[r].idx = order[r].idx;
                    given += fl;
                }
            }
            int64_t missing = (int64_t)n * avg - given;
            qsort(fr, (size_t)n, sizeof(frac_t), cmp_rem_desc_rank_asc);
            for (int i = 0; i < n && missing > 0; ++i, --missing) budgets[base + fr[i].idx] += 1;
        }
    }
    free(order);
    free(fr);

    const size_t units = (size_t)B * L * H;
    offsets[0] = 0;
    for (size_t u = 0; u < units; ++u) offsets[u + 1] = offsets[u] + budgets[u];

    if (layer_group && layer_ctx) {
        for (int b = 0; b < B; ++b) {
            int32_t *lg = layer_group + (size_t)b * L, *lc = layer_ctx + (size_t)b * L;
            if (dn <= 0) {
                for (int l = 0; l < L; ++l) { lg[l] = 0; lc[l] = N; }
                continue;
            }
            int boundaries = 0;
            lg[0] = 0;
            for (int l = 0; l + 1 < L; ++l) {
                double e0 = 0.0, e1 = 0.0;
                for (int h = 0; h < H; ++h) e0 += erank[((size_t)b * L + l) * H + h];
                for (int h = 0; h < H; ++h) e1 += erank[((size_t)b * L + l + 1) * H + h];
                e0 /= (double)H;
                e1 /= (double)H;
                if (e0 - e1 > eps) ++boundaries;
                lg[l + 1] = boundaries;
            }
            for (int l = 0; l < L; ++l) {
                if (lg[l] == 0) lc[l] = N;
                else {
                    const int64_t c = (int64_t)n_last + (int64_t)(boundaries - lg[l]) * dn;
                    lc[l] = (int32_t)(c < N ? c : N);
                }
            }
        }
    }
    return 0;
}

/* ------------------------------------------------------------------------------------------------
 * Observation-window scores of one unit (Section 3.3.3, "Dynamic KV Cache Eviction").
 *
 * Q is [G, w, d]: the last w query positions of the G query heads that attend to this KV head; row i
 * sits at position N - w + i.  K is [N, d].  Each row attends causally to keys j <= N - w + i with
 * logits scale * (q . k_j) and a softmax over all keys it sees (prefix and window alike).  The raw
 * score of prefix key j < N - w is the sum of its attention probabilities over the w rows and the G
 * query heads.  raw has N - w entries.
 * Readings: scale 1/sqrt(d) by the caller, sum over grouped query heads, causal inside the window.
 * ---------------------------------------------------------------------------------------------- */
void oracle_window_scores(const double *Q, const double *K, int N, int d, int w, int G, double scale,
                          double *raw)
{
    const int P = N - w;
    double *s = (double *)malloc((size_t)N * sizeof(double));
    for (int j = 0; j < P; ++j) raw[j] = 0.0;
    for (int g = 0; g < G; ++g) {
        for (int i = 0; i < w; ++i) {
            const double *q = Q + ((size_t)g * w + i) * d;
            const int last = P + i; /* inclusive */
            double mx = -INFINITY;
            for (int j = 0; j <= last; ++j) {
                double acc = 0.0;
                const double *k = K + (size_t)j * d;
                for (int a = 0; a < d; ++a) acc += q[a] * k[a];
                s[j] = scale * acc;
                if (s[j] > mx) mx = s[j];
            }
            double denom = 0.0;
            for (int j = 0; j <= last; ++j) denom += exp(s[j] - mx);
            for (int j = 0; j < P; ++j) raw[j] += exp(s[j] - mx) / denom;
        }
    }
    free(s);
}

/* ------------------------------------------------------------------------------------------------
 * Log-sum-exp of every window row (the row normaliser of the softmax above, Section 3.3.3): for query
 * head g and window row i, lse[g * w + i] = ln sum_{j <= N - w + i} exp(scale * (q . k_j)), natural
 * logarithm, over the same causally visible keys as oracle_window_scores.  It is what a prefill
 * attention kernel keeps per row; with it, softmax(s)[j] = exp(s[j] - lse).  lse has G * w entries.
 * ---------------------------------------------------------------------------------------------- */
void oracle_window_lse(const double *Q, const double *K, int N, int d, int w, int G, double scale,
                       double *lse)
{
    const int P = N - w;
    double *s = (double *)malloc((size_t)N * sizeof(double));
    for (int g = 0; g < G; ++g) {
        for (int i = 0; i < w; ++i) {
            const double *q = Q + ((size_t)g * w + i) * d;
            const int last = P + i; /* inclusive */
            double mx = -INFINITY;
            for (int j = 0; j <= last; ++j) {
                double acc = 0.0;
                const double *k = K + (size_t)j * d;
                for (int a = 0; a < d; ++a) acc += q[a] * k[a];
                s[j] = scale * acc;
                if (s[j] > mx) mx = s[j];
            }
            double denom = 0.0;
            for (int j = 0; j <= last; ++j) denom += exp(s[j] - mx);
            lse[(size_t)g * w + i] = mx + log(denom);
        }
    }
    free(s);
}

/* 1-D pooling over the prefix scores: window of pool_kernel (odd) entries centred on j, clipped to
 * [0, P); mode 0 = max, 1 = mean over the entries inside the range.  pool_kernel = 1 copies.
 * (The paper is silent on pooling; the SnapKV-style scorer it cites pools, and 7/max is the default.) */
void oracle_pool(const double *raw, int P, int pool_kernel, int pool_mode, double *pooled)
{
    const int half = pool_kernel / 2;
    for (int j = 0; j < P; ++j) {
        const int lo = j - half < 0 ? 0 : j - half;
        const int hi = j + half > P - 1 ? P - 1 : j + half;
        double acc = pool_mode ? 0.0 : raw[lo];
        for (int t = lo; t <= hi; ++t) {
            if (pool_mode) acc += raw[t];
            else if (raw[t] > acc) acc = raw[t];
        }
        pooled[j] = pool_mode ? acc / (double)(hi - lo + 1) : acc;
    }
}

/* ------------------------------------------------------------------------------------------------
 * Selection: with budget b (window included) keep the k = b - w prefix positions with the largest
 * scores (equal scores: the lower position wins) and all w window positions.  idx receives b entries:
 * the kept prefix positions in ascending order, then N - w, ..., N - 1.
 * ---------------------------------------------------------------------------------------------- */
void oracle_select(const double *score, int P, int w, int budget, int32_t *idx)
{
    const int k = budget - w;
    keyed_t *order = (keyed_t *)malloc((size_t)(P > 0 ? P : 1) * sizeof(keyed_t));
    char *keep = (char *)calloc((size_t)(P > 0 ? P : 1), 1);
    for (int j = 0; j < P; ++j) { order[j].key = score[j]; order[j].idx = j; }
    qsort(order, (size_t)P, sizeof(keyed_t), cmp_key_desc_idx_asc);
    for (int r = 0; r < k && r < P; ++r) keep[order[r].idx] = 1;
    int o = 0;
    for (int j = 0; j < P; ++j) if (keep[j]) idx[o++] = j;
    for (int i = 0; i < w; ++i) idx[o++] = P + i;
    free(order);
    free(keep);
}

/* Compaction of one unit: dst row t = src row idx[t]; rows are row_bytes raw bytes. */
void oracle_compact(const unsigned char *src, size_t row_bytes, const int32_t *idx, int count,
                    unsigned char *dst)
{
    for (int t = 0; t < count; ++t)
        memcpy(dst + (size_t)t * row_bytes, src + (size_t)idx[t] * row_bytes, row_bytes);
}

/* ------------------------------------------------------------------------------------------------
 * Hidden-state eviction between layer groups (Section 3.3.2, "Hidden State Eviction"): the tokens kept
 * for the next layer are chosen by the attention scores of the LAST token of the current layer.
 *
 * q is [Hq, d] (the last position's query of every query head), K is [H, N, d] (the layer's keys; query
 * head h attends to KV head h / (Hq / H)).  Each head's logits scale * (q_h . k_j) over all N positions
 * go through a softmax; score[j] is the sum over the Hq heads.  score has N entries.
 * Readings (the paper gives one sentence): heads are summed, scale 1/sqrt(d) by the caller.  The caller
 * keeps the last position unconditionally and selects among the first N - 1 (oracle_select with w = 1).
 * ---------------------------------------------------------------------------------------------- */
void oracle_last_token_scores(const double *q, const double *K, int H, int Hq, int N, int d, double scale,
                              double *score)
{
    const int G = Hq / H;
    double *s = (double *)malloc((size_t)N * sizeof(double));
    for (int j = 0; j < N; ++j) score[j] = 0.0;
    for (int h = 0; h < Hq; ++h) {
        const double *qh = q + (size_t)h * d;
        const double *Kh = K + (size_t)(h / G) * N * d;
        double mx = -INFINITY;
        for (int j = 0; j < N; ++j) {
            double acc = 0.0;
            for (int a = 0; a < d; ++a) acc += qh[a] * Kh[(size_t)j * d + a];
            s[j] = scale * acc;
            if (s[j] > mx) mx = s[j];
        }
        double denom = 0.0;
        for (int j = 0; j < N; ++j) denom += exp(s[j] - mx);
        for (int j = 0; j < N; ++j) score[j] += exp(s[j] - mx) / denom;
    }
    free(s);
}

/* ----------------------------------------------------------------------------------------------
 * Decode-time cache update of one head (paper Section 3.3.3, "Dynamic KV Cache Eviction", last sentence;
 * Algorithm 2, decoding loop): the new token is concatenated with the head's cache, attention is computed
 * over the concatenation, and once the cache exceeds its budget the entry with the lowest cumulative
 * attention score is evicted.
 *
 * oracle_decode_probs: Kc is the head's cache [len, d], knew [d] the new token's key, q [G, d] the new
 * token's queries of the G query heads that share this KV head.  Each head's logits scale * (q_g . k_j)
 * over the len + 1 entries (entry len is the new token) go through a softmax; p[j] is the sum over the G
 * heads.  p has len + 1 entries.
 *
 * oracle_decode_evict: cum [len] are the cumulative scores of the cached entries AFTER this step's p has
 * been added, pos [len] their positions in the sequence.  Returns the entry to evict: the lowest
 * cumulative score among the entries with pos <= new_pos - protect (the newest `protect` positions,
 * the new token included, are not candidates); equal scores: the lower position.  If no entry is a
 * candidate, every cached entry is one.  len >= 1.
 * Readings: heads of a group are summed as in the prefill scorer; the new token starts with its own
 * probability as cumulative score; a cache below its budget appends without evicting (the caller decides).
 * ---------------------------------------------------------------------------------------------- */
void oracle_decode_probs(const double *q, const double *Kc, const double *knew, int G, int len, int d,
                         double scale, double *p)
{
    const int n = len + 1;
    double *s = (double *)malloc((size_t)n * sizeof(double));
    for (int j = 0; j < n; ++j) p[j] = 0.0;
    for (int g = 0; g < G; ++g) {
        const double *qg = q + (size_t)g * d;
        double mx = -INFINITY;
        for (int j = 0; j < n; ++j) {
            const double *k = j < len ? Kc + (size_t)j * d : knew;
            double acc = 0.0;
            for (int a = 0; a < d; ++a) acc += qg[a] * k[a];
            s[j] = scale * acc;
            if (s[j] > mx) mx = s[j];
        }
        double denom = 0.0;
        for (int j = 0; j < n; ++j) denom += exp(s[j] - mx);
        for (int j = 0; j < n; ++j) p[j] += exp(s[j] - mx) / denom;
    }
    free(s);
}

int oracle_decode_evict(const double *cum, const int32_t *pos, int len, int new_pos, int protect)
{
    int any = 0;
    for (int j = 0; j < len; ++j) any |= pos[j] <= new_pos - protect;
    int best = -1;
    for (int j = 0; j < len; ++j) {
        if (any && !(pos[j] <= new_pos - protect)) continue;
        if (best < 0 || cum[j] < cum[best] || (cum[j] == cum[best] && pos[j] < pos[best])) best = j;
    }
    return best;
}

/* ----------------------------------------------------------------------------------------------
 * Preparation stage (Section 3.3.1 "Preparation Stage", its equation for the averaged effective rank;
 * Algorithm 1, head group identification).
 *
 * erank is [S, L, H]: the truncated effective rank of every head for each of S samples.
 *   oracle_prepare_mean    mean[l,h] = (1/S) sum_i erank[i,l,h]                       (the equation)
 *   oracle_group_labels    heads of a ranking set (one layer: scope 0, n = H; the whole model: scope 1,
 *                          n = L*H) sorted by descending value, equal values by ascending index; the head
 *                          at rank r gets group g with floor(g n / M) <= r < floor((g+1) n / M): M groups
 *                          whose sizes differ by at most one, group 0 the highest values (the grouping
 *                          the budget rule uses).  values is [L, H], one label per head.
 *   oracle_majority_vote   Algorithm 1: every sample labels the heads by oracle_group_labels on its own
 *                          values; votes[l,h,g] counts the samples that put head (l,h) in group g; the
 *                          final label is the group with most votes, the lowest such group on a tie.
 * Readings: "one of 8 clusters based on E" is taken as the rank-based equal-size grouping above (the
 * paper names no clustering algorithm and the inference stage ranks heads the same way); M = 2 gives
 * the retrieval / streaming split of Section 3.3.3 "Retrieval Head" with label 0 the retrieval heads.
 * ---------------------------------------------------------------------------------------------- */
void oracle_prepare_mean(const double *erank, int S, int L, int H, double *mean)
{
    for (int i = 0; i < L * H; ++i) {
        double acc = 0.0;
        for (int s = 0; s < S; ++s) acc += erank[(size_t)s * L * H + i];
        mean[i] = acc / (double)S;
    }
}

int oracle_group_labels(const double *values, int L, int H, int M, int scope, int32_t *labels)
{
    const int n = scope ? L * H : H;
    const int sets = scope ? 1 : L;
    if (M < 1 || M > n) return -1;
    keyed_t *order = (keyed_t *)malloc((size_t)n * sizeof(keyed_t));
    for (int s = 0; s < sets; ++s) {
        const size_t base = (size_t)s * n;
        for (int i = 0; i < n; ++i) { order[i].key = values[base + i]; order[i].idx = i; }
        qsort(order, (size_t)n, sizeof(keyed_t), cmp_key_desc_idx_asc);
        for (int g = 0; g < M; ++g) {
            const int lo = (int)((int64_t)g * n / M), hi = (int)((int64_t)(g + 1) * n / M);
            for (int r = lo; r < hi; ++r) labels[base + order[r].idx] = g;
        }
    }
    free(order);
    return 0;
}

int oracle_majority_vote(const double *erank, int S, int L, int H, int M, int scope, int32_t *votes,
                         int32_t *labels)
{
    const int LH = L * H;
    int32_t *one = (int32_t *)malloc((size_t)LH * sizeof(int32_t));
    for (int i = 0; i < LH * M; ++i) votes[i] = 0;
    for (int s = 0; s < S; ++s) {
        if (oracle_group_labels(erank + (size_t)s * LH, L, H, M, scope, one) != 0) { free(one); return -1; }
        for (int i = 0; i < LH; ++i) votes[(size_t)i * M + one[i]] += 1;
    }
    for (int i = 0; i < LH; ++i) {
        int best = 0;
        for (int g = 1; g < M; ++g)
            if (votes[(size_t)i * M + g] > votes[(size_t)i * M + best]) best = g;
        labels[i] = best;
    }
    free(one);
    return 0;
}


/* ----------------------------------------------------------------------------------------------
 * Cumulative scores of a head's cache right after prefill (Section 3.3.3, "Dynamic KV Cache Eviction":
 * the cumulative attention score window is what decides evictions during decoding).
 * score is the head's prefill score of every prefix position [P]; idx [n] the kept positions (prefix
 * positions < P and the w window positions >= P).  A kept prefix position starts with its prefill score.
 * Reading: the paper does not score the window positions themselves (they are kept unconditionally at
 * prefill); each starts with the largest score among the kept prefix positions of its head (0 if none
 * is kept), so a window token never leaves before a prefix token merely for lack of a score.
 * ---------------------------------------------------------------------------------------------- */
void oracle_decode_seed(const double *score, int P, const int32_t *idx, int n, double *cum)
{
    double top = 0.0;
    int any = 0;
    for (int t = 0; t < n; ++t)
        if (idx[t] < P && (!any || score[idx[t]] > top)) { top = score[idx[t]]; any = 1; }
    for (int t = 0; t < n; ++t) cum[t] = idx[t] < P ? score[idx[t]] : top;
}


/* ----------------------------------------------------------------------------------------------
 * Retrieval layer (Section 3.3.2, "Retrieval Layer": the layer with the maximum entropy increase).
 * values is [L, H] (the truncated entropy, or the effective rank, of every head; e.g. the averaged
 * values of the preparation stage).  With e_l the mean over the H heads of layer l, increase[l] =
 * e_{l+1} - e_l for l = 0 .. L-2 and the retrieval layer is l* + 1 for the first l* that attains the
 * largest increase: the layer whose token matrix gained the most over its predecessor.  L >= 2.
 * Reading: the paper names the criterion only; taking the layer AFTER the jump, the mean over heads as
 * the layer's value and the earliest layer on a tie are this implementation's choices.  The merging
 * of that layer's parameters with the last layer's is a change of model weights and not part of this.
 * ---------------------------------------------------------------------------------------------- */
int oracle_retrieval_layer(const double *values, int L, int H, double *increase)
{
    int best = 0;
    double prev = 0.0, best_inc = 0.0;
    for (int l = 0; l < L; ++l) {
        double e = 0.0;
        for (int h = 0; h < H; ++h) e += values[(size_t)l * H + h];
        e /= (double)H;
        if (l > 0) {
            const double inc = e - prev;
            if (increase) increase[l - 1] = inc;
            if (l == 1 || inc > best_inc) { best_inc = inc; best = l; }
        }
        prev = e;
    }
    return best;
}
