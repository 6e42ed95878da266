/*
 * uncomp.h -- C ABI of the prefill-end KV-cache compression pass of UNComp (arXiv 2410.03090),
 * implemented as hand-written CUDA for NVIDIA B200 (sm_100a).
 *
 * One pass, four calls, all asynchronous on the caller's stream and with no host synchronisation in
 * between (budgets and offsets stay on the device):
 *
 *   uncomp_entropy         truncated matrix entropy / effective rank of every (batch, layer, KV head)
 *                          key matrix                                     (paper Section 3.1 - 3.2)
 *   uncomp_assign_budgets  per-head token budgets from the effective ranks, and the layer-group
 *                          partition                                      (paper Section 3.3.2, 3.3.3)
 *   uncomp_score_select    observation-window attention scores of the prefix tokens and the top
 *                          tokens of every head within its budget         (Section 3.3.3, "Dynamic KV
 *                                                                          Cache Eviction")
 *   uncomp_compact         gather of the kept K / V rows into a ragged per-head cache
 *                                                                         (Section 3.3.3; Algorithm 2,
 *                                                                          prefill loop over heads)
 *
 * Conventions
 *   - "unit" = one (batch b, layer l, KV head h); units are numbered row-major over [B, L, H].
 *   - Pointers whose name starts with d_ are DEVICE pointers; everything else is host memory.
 *   - The library never allocates or frees device memory.  Inputs, outputs and the workspace belong to
 *     the caller and must stay valid until the stream work of the call has finished.
 *   - Every call returns an int: UNCOMP_OK or a negative UNCOMP_E_* code for a synchronous, host-side
 *     rejection (nothing was launched).  Conditions found on the device are OR-ed into a status word
 *     that uncomp_status() reads; kernels never trap, assert or spin without a limit.
 *   - A context is bound to one shape and one workspace and is not thread-safe; use one per stream.
 *   - `stream` is a cudaStream_t passed as void* (NULL = the default stream).
 */
#ifndef UNCOMP_H_
#define UNCOMP_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct uncomp_ctx uncomp_ctx; /* opaque */

typedef enum { UNCOMP_BF16 = 0, UNCOMP_FP32 = 1 } uncomp_dtype;

/* Shape of one pass.  B sequences, L layers, H KV heads, Hq query heads (a multiple of H; G = Hq / H
 * query heads share one KV head), N tokens, head dimension d (must be 128), observation window w
 * (1 <= w <= 64, w < N, G * w <= 512), storage type of K, V and the window queries. */
typedef struct {
    int32_t B, L, H, Hq, N, d, w;
    int32_t dtype; /* uncomp_dtype */
} uncomp_shape;

/* Element strides of a [B, L, H, N, d] tensor; the d stride is 1.  Every row must start on a 16-byte
 * boundary (base pointer 16-byte aligned, strides multiples of 16 bytes). */
typedef struct {
    int64_t sB, sL, sH, sN;
} uncomp_strides;

enum {
    UNCOMP_OK = 0,
    UNCOMP_E_NULL = -1,        /* a required pointer is NULL */
    UNCOMP_E_SHAPE = -2,       /* unsupported shape (d != 128, N <= w, Hq % H != 0, ...) */
    UNCOMP_E_ALIGN = -3,       /* pointer or stride not 16-byte aligned */
    UNCOMP_E_WORKSPACE = -4,   /* workspace smaller than uncomp_workspace_bytes() */
    UNCOMP_E_PARAM = -5,       /* invalid hyper-parameter */
    UNCOMP_E_CUDA = -6,        /* a CUDA runtime / driver call failed; see uncomp_last_cuda_error() */
    UNCOMP_E_LIMIT = -7        /* size beyond a documented maximum */
};

/* Bits of the device status word. */
enum {
    UNCOMP_STATUS_NOT_CONVERGED = 1u, /* eigenvalue multi-section hit max_iters before its tolerance */
    UNCOMP_STATUS_TIMEOUT = 2u,       /* a bounded device-side wait expired */
    UNCOMP_STATUS_BOUNDS = 4u,        /* an index, offset or budget check failed; the value was clamped / skipped */
    UNCOMP_STATUS_NONFINITE = 8u      /* a caller-supplied log-sum-exp was NaN or infinite; its row was left out */
};

/* Bytes of device workspace a context of this shape needs.  Pure host function.  0 on a bad shape. */
size_t uncomp_workspace_bytes(const uncomp_shape *shape);

/* Create a context over caller-owned device workspace (256-byte aligned, at least
 * uncomp_workspace_bytes(shape) bytes).  Clears the status word with a cudaMemset and waits for it.
 * The device current at creation must be current for every later call. */
int uncomp_create(uncomp_ctx **out, const uncomp_shape *shape, void *d_workspace, size_t workspace_bytes);
void uncomp_destroy(uncomp_ctx *ctx);

/* ---------------------------------------------------------------------------------------------------
 * uncomp_entropy -- Section 3.1 Eq. 1 (covariance), Lemma 2 (eigenvalue form of the matrix entropy),
 * Section 3.2 (truncated matrix entropy H_k and truncated effective rank erank_k = exp H_k).
 *
 * For every unit, with X = K[b, l, h] of shape [N, d]:
 *   C = sum_i (x_i - mean)(x_i - mean)^T            (center = 1; C = X^T X for center = 0; the factor
 *                                                    1/(N-1) of Eq. 1 cancels below)
 *   lambda_1 >= ... >= lambda_d  eigenvalues of C, negatives counted as 0
 *   p_i = lambda_i / sum_{j<=k} lambda_j  (norm = 0)   or   lambda_i / trace(C)  (norm = 1)
 *   H_k = - sum_{i<=k} p_i ln p_i ,  erank_k = exp(H_k),   k = min(k_trunc, d)
 *
 * bf16 input: Gram matrix on the tensor cores with fp32 accumulation, chunk partials added in fp64, then
 * an fp32 Householder tridiagonalisation held in registers and a Sturm-count multi-section for the k
 * largest eigenvalues (bracketed to 2e-8 of the spectral radius; the fp32 reduction is good to about
 * 1e-7).  fp32 input: Gram matrix and eigenvalues in fp64 throughout (Householder in shared memory,
 * brackets to 1e-13 of the spectral radius).  max_iters bounds the multi-section rounds (0 = the default
 * of the path, 10 or 14); a unit that has not reached its tolerance by then sets
 * UNCOMP_STATUS_NOT_CONVERGED and still writes its current estimate.
 *
 * Fusion with the scorer: the window scorer (uncomp_score_select) also sweeps over K and needs, before
 * anything else, the softmax statistics of its window rows.  If d_Qw is given (bf16 keys only; ignored
 * otherwise), those statistics are produced in the same sweep that forms the Gram matrices -- one read of
 * K instead of two -- and are kept in the workspace.  The next uncomp_score_select call on this context
 * skips its statistics pass if it sets reuse_stats = 1 and passes the same d_K, strides, d_Qw and scale;
 * by setting the flag the caller vouches that K and Qw have not changed in between (the library compares
 * pointers, it cannot see contents).  Any uncomp_score_select call consumes the statistics.
 * d_Qw = NULL runs the entropy stage on its own.
 *
 * d_K        in   [B, L, H, N, d] with strides sK, storage dtype of the shape
 * d_Qw       in   [B, L, Hq, w, d] window queries as for uncomp_score_select, or NULL
 * scale           logit scale of the scorer (0 means 1 / sqrt(d)); only used with d_Qw
 * d_entropy  out  [B, L, H] float, H_k
 * d_erank    out  [B, L, H] float, erank_k; may be NULL
 * d_spectrum out  [B, L, H, k] double, the k largest eigenvalues of C (unnormalised); may be NULL
 * ------------------------------------------------------------------------------------------------- */
typedef struct {
    int32_t k_trunc;   /* >= 1 */
    int32_t center;    /* 1 = Eq. 1 (centred), 0 = uncentred */
    int32_t norm;      /* 0 = normalise over the k kept eigenvalues, 1 = over the whole trace */
    int32_t max_iters; /* multi-section rounds, 0 = default */
} uncomp_entropy_params;

int uncomp_entropy(uncomp_ctx *ctx, const void *d_K, uncomp_strides sK, const uncomp_entropy_params *params,
                   const void *d_Qw, float scale, float *d_entropy, float *d_erank, double *d_spectrum,
                   void *stream);

/* uncomp_gram -- the building blocks of Eq. 1 on their own: for every unit the Gram matrix G = X^T X and
 * the column sums s = X^T 1 (the covariance of Eq. 1 is (G - s s^T / N) / (N - 1)), as produced by the
 * first stage of uncomp_entropy and summed over its token chunks in fp64.
 * d_gram  out  [B*L*H, d*d + d] double: G row-major, then s. */
int uncomp_gram(uncomp_ctx *ctx, const void *d_K, uncomp_strides sK, double *d_gram, void *stream);

/* uncomp_gram_static -- uncomp_gram for callers that cannot allocate device memory.  The paper has no
 * counterpart: this entry point exists for integration only.
 *
 * Who needs it: code that runs where cudaMalloc is off limits, and that therefore cannot create the
 * workspace every other call of this library lives in -- a custom-operator hook inside a serving framework
 * whose own caching allocator owns the device memory, or a latency-critical thread that must not take the
 * device-wide stall an allocation or a free causes.  It needs no context and no workspace: the per-chunk
 * partial sums go to a fixed array inside the library image (uncomp_gram_static_max_bytes() = 4,227,072
 * bytes, plus one status word), which every GPU that loads the library holds until the process exits.
 * The call itself allocates nothing, on the device or through any library.
 *
 * Limits and rules
 *   - The array holds 64 chunk partials for bf16 keys and 32 for fp32 keys, and every unit needs at least
 *     one: at most 64 (32) units per call, any number of tokens.  More units are refused with
 *     UNCOMP_E_LIMIT and nothing is launched.  When units x (token chunks uncomp_gram would use) exceeds
 *     the array, the call takes fewer, longer chunks (e.g. one layer of 8 heads x 32768 tokens in bf16 runs
 *     as 8 x 8 chunks of 4096 tokens instead of 8 x 32).  A chunk is accumulated in fp32 on the tensor
 *     cores, so longer chunks round more: about 1e-5 of the largest entry at 4096 tokens per chunk, against
 *     2e-6 at uncomp_gram's 1024; with the same chunking the two entry points agree bit for bit.
 *   - The first call on a device looks up the array's device address (the device must be current).  Make
 *     that first call outside any stream capture.
 *   - All calls share the one array and it keeps the previous call's contents; this call overwrites the
 *     part it reads and clears its status word itself.  Two calls whose GPU work overlaps (different
 *     streams, or threads) race on it: serialise them.
 *   - Device-side conditions (a bounded wait that expired) are not reported by this entry point.
 * Arguments as for uncomp_gram, with the shape passed directly. */
int uncomp_gram_static(const uncomp_shape *shape, const void *d_K, uncomp_strides sK, double *d_gram, void *stream);
size_t uncomp_gram_static_max_bytes(void);

/* ---------------------------------------------------------------------------------------------------
 * uncomp_assign_budgets -- Section 3.3.3 "Head-Group Compression": heads ranked by truncated effective
 * rank, split into M groups, group budgets N_{i,g+1} = N_{i,g} - step from n_max downwards; and
 * Section 3.3.2 "Layer-Group Compression": Delta c_i, the stage count C and N_{i+1} = N_i + dn.
 *
 * Ranking set: the H heads of a layer (scope = 0) or all L*H heads of a sequence (scope = 1); n = its
 * size.  Larger erank ranks first, ties go to the lower (layer, head) index.  Ranks
 * [floor(g n/M), floor((g+1) n/M)) form group g.  Group target t_g = n_max - g * step with
 * step = n (n_max - avg_budget) / sum_g(n_g g), so that the set's budgets sum to n * avg_budget
 * exactly: heads get floor(t_g) and the remaining tokens go one each to the largest fractional parts
 * (ties: better rank first).  All of it in exact integer arithmetic.  The window is part of a budget.
 * d_offsets is the exclusive prefix sum of the budgets over units; d_offsets[units] = units * avg_budget.
 *
 * Layer partition (dn > 0): e_l = mean erank of layer l; a boundary follows layer l iff
 * e_l - e_{l+1} > eps; d_layer_group[l] = boundaries before l; d_layer_ctx = N for group 0, else
 * min(N, n_last + (boundaries_total - group) * dn).  dn = 0: group 0 and N everywhere.
 *
 * Rejected with UNCOMP_E_PARAM: M < 1, M > n, avg_budget < w, n_max < avg_budget, n_max > N, smallest
 * group target below w.
 *
 * d_erank        in   [B, L, H] float
 * d_budgets      out  [B, L, H] int32
 * d_offsets      out  [B*L*H + 1] int64
 * d_layer_group  out  [B, L] int32, may be NULL
 * d_layer_ctx    out  [B, L] int32, may be NULL
 * ------------------------------------------------------------------------------------------------- */
typedef struct {
    int32_t avg_budget; /* average tokens kept per head, window included */
    int32_t M;          /* head groups */
    int32_t n_max;      /* budget of the group with the largest erank (paper: N_{i,1}) */
    int32_t scope;      /* 0 = rank within each layer, 1 = rank over all heads of a sequence */
    float eps;          /* layer partition threshold (paper: epsilon) */
    int32_t dn;         /* context step between layer groups (paper: Delta n); 0 disables */
    int32_t n_last;     /* context of the last layer group */
} uncomp_budget_params;

int uncomp_assign_budgets(uncomp_ctx *ctx, const float *d_erank, const uncomp_budget_params *params,
                          int32_t *d_budgets, int64_t *d_offsets, int32_t *d_layer_group,
                          int32_t *d_layer_ctx, void *stream);

/* ---------------------------------------------------------------------------------------------------
 * uncomp_score_select -- Section 3.3.3 "Dynamic KV Cache Eviction": the attention of the last w query
 * positions is summed per key position and the highest-scored tokens are kept within the head's budget.
 *
 * For every unit and every prefix position j < N - w:
 *   raw[j] = sum over the G query heads q of the unit and window rows i < w of softmax_j'(s_{q,i})[j],
 *   s_{q,i}[j'] = scale * <Qw[b,l,q,i,:], K[b,l,h,j',:]>  over the causally visible j' <= N - w + i.
 *   score[j] = max (pool_mode 0) or mean (pool_mode 1) of raw over [j - pool_kernel/2, j + pool_kernel/2]
 *              clipped to the prefix.
 * The budget[u] - w prefix positions with the largest score (ties: lower position) are written in
 * ascending order to d_indices[offsets[u] ...], followed by the window positions N-w .. N-1.
 *
 * Softmax needs every row's normaliser before any column can be summed, so the window logits are formed
 * twice (a statistics sweep over K, then the column sums) unless the normalisers are already known:
 *   - reuse_stats = 1: a preceding uncomp_entropy call with d_Qw left them in the workspace (see there);
 *   - d_lse given: the caller supplies them.  A prefill attention kernel that has just processed the same
 *     window rows owns, per row, lse = ln sum_{j' visible} exp(s_{q,i}[j']) (natural logarithm, of the
 *     SCALED logits, over all causally visible keys, prefix and window alike).  Then
 *     softmax(s)[j] = exp(s[j] - lse) and one sweep over K suffices.  The values are trusted: an lse that
 *     does not belong to these queries and keys gives scores that are wrong by the same factor.  A NaN or
 *     infinite entry sets UNCOMP_STATUS_NONFINITE and its row contributes nothing.
 *
 * Every slab offsets[u] .. offsets[u+1] is filled completely and nothing is written outside it: a budget
 * that differs from the slab length or lies outside [w, N], or offsets that are not ascending inside
 * [0, offsets[units]], set UNCOMP_STATUS_BOUNDS; the unit then keeps as many top positions as the slab and
 * the budget allow, the window positions as far as they fit, and fills what remains with position N - 1
 * (a unit whose offsets are unusable writes nothing).
 *
 * d_Qw       in   [B, L, Hq, w, d] contiguous, storage dtype; query head q belongs to KV head q / G
 * d_K        in   as in uncomp_entropy
 * d_lse      in   [B, L, Hq, w] float, or NULL
 * d_budgets  in   [B, L, H] int32, each in [w, N] and equal to offsets[u+1] - offsets[u]
 * d_offsets  in   [B*L*H + 1] int64
 * d_scores   out  [B, L, H, N - w] float, the pooled scores; may be NULL (workspace is used then)
 * d_indices  out  [offsets[units]] int32
 * ------------------------------------------------------------------------------------------------- */
typedef struct {
    int32_t pool_kernel; /* odd, 1 = no pooling, at most 63 */
    int32_t pool_mode;   /* 0 = max, 1 = mean */
    float scale;         /* 0 means 1 / sqrt(d) */
    int32_t reuse_stats; /* 1 = take the row statistics the preceding uncomp_entropy (with d_Qw) left for these
                            d_K, strides, d_Qw and scale; when there are none (another tensor, fp32 keys) the
                            statistics sweep runs as with 0.  0 = never reuse.  Ignored when d_lse is given. */
} uncomp_score_params;

int uncomp_score_select(uncomp_ctx *ctx, const void *d_Qw, const void *d_K, uncomp_strides sK, const float *d_lse,
                        const int32_t *d_budgets, const int64_t *d_offsets, const uncomp_score_params *params,
                        float *d_scores, int32_t *d_indices, void *stream);

/* ---------------------------------------------------------------------------------------------------
 * uncomp_compact -- the per-head ragged cache of Section 3.3.3 ("each head maintains its context
 * window"); keys and values share one selection (caption of the paper's main table).
 *   Kc[offsets[u] + t, :] = K[unit u, indices[offsets[u] + t], :]   for t < offsets[u+1] - offsets[u]
 * and the same for V.  Rows are copied bit for bit.  An index outside [0, N) is replaced by the nearest
 * valid position and sets UNCOMP_STATUS_BOUNDS (no address outside the unit's rows is ever formed).
 *
 * d_K, d_V    in   [B, L, H, N, d] with strides sK, sV
 * d_indices   in   [offsets[units]] int32
 * d_offsets   in   [B*L*H + 1] int64
 * d_Kc, d_Vc  out  [offsets[units], d] contiguous, storage dtype, 16-byte aligned
 * ------------------------------------------------------------------------------------------------- */
int uncomp_compact(uncomp_ctx *ctx, const void *d_K, const void *d_V, uncomp_strides sK, uncomp_strides sV,
                   const int32_t *d_indices, const int64_t *d_offsets, void *d_Kc, void *d_Vc, void *stream);

/* ---------------------------------------------------------------------------------------------------
 * uncomp_evict_hidden -- Section 3.3.2 "Hidden State Eviction" (Algorithm 2: "compress hidden states"):
 * between layer groups the hidden states of the tokens with the highest attention scores of the LAST token
 * of the current layer are kept, n_keep of them (the context size d_layer_ctx gives for the next group).
 *
 * One layer per call, for every sequence b of the context's shape (L and w of the shape are not used):
 *   score[j] = sum over the Hq query heads h of softmax_j(scale * <qlast[b,h,:], K[b, h/G, j, :]>), all N positions
 *   kept = the last position and the n_keep - 1 highest-scored of the first N - 1 (ties: lower position),
 *          written in ascending order;  Xout[b, t, :] = X[b, kept[t], :]  bit for bit.
 * Readings where the paper is silent: heads are summed; the last position always survives (it is the
 * position the next layers continue from).
 *
 * d_qlast    in   [B, Hq, d] contiguous, the last position's queries of this layer, storage dtype
 * d_K        in   this layer's keys [B, H, N, d]; strides sK.sB, sK.sH, sK.sN (sK.sL is ignored)
 * d_X        in   [B, N, D] contiguous hidden states, storage dtype, D * element size a multiple of 16
 * n_keep          1 <= n_keep <= N
 * scale           0 means 1 / sqrt(d)
 * d_scores   out  [B, N - 1] float scores of the prefix positions; may be NULL
 * d_indices  out  [B, n_keep] int32
 * d_Xout     out  [B, n_keep, D]
 * Rejected: G = Hq / H not in {1, 2, 4, 8, 16} (UNCOMP_E_SHAPE), misaligned rows, n_keep out of range.
 * ------------------------------------------------------------------------------------------------- */
int uncomp_evict_hidden(uncomp_ctx *ctx, const void *d_qlast, const void *d_K, uncomp_strides sK, const void *d_X,
                        int32_t D, int32_t n_keep, float scale, float *d_scores, int32_t *d_indices, void *d_Xout,
                        void *stream);

/* ---------------------------------------------------------------------------------------------------
 * uncomp_decode_seed -- Section 3.3.3 "Dynamic KV Cache Eviction": the cumulative attention scores that
 * decide evictions during decoding start from the prefill's window scores.  For every unit, row t of its
 * slab of the ragged cache (position indices[offsets[u] + t]) gets
 *   cum = scores[u, position]                               for a kept prefix position (< N - w)
 *   cum = max over the unit's kept prefix positions of scores[u, .]   for a window position (0 if the unit
 *         keeps no prefix position)
 * Reading: the prefill does not score the window positions (they are kept unconditionally); giving them
 * the head's largest kept score means a window token is never evicted before a prefix token merely for
 * lack of a score.  d_pos of uncomp_decode_update is d_indices itself (copy it: the update changes it).
 *
 * d_scores   in   [B, L, H, N - w] float, the d_scores output of uncomp_score_select
 * d_indices  in   [offsets[units]] int32;  d_offsets in [B*L*H + 1] int64 (outputs of the same call)
 * d_cum      out  [offsets[units]] float
 * ------------------------------------------------------------------------------------------------- */
int uncomp_decode_seed(uncomp_ctx *ctx, const float *d_scores, const int32_t *d_indices, const int64_t *d_offsets,
                       float *d_cum, void *stream);

/* ---------------------------------------------------------------------------------------------------
 * uncomp_decode_update -- Section 3.3.3 "Dynamic KV Cache Eviction", last sentence (as new tokens are
 * generated, the token with the lowest cumulative attention score is evicted) and Algorithm 2, decoding
 * loop (the new token is concatenated with each head's cache and attends over the concatenation).
 *
 * One decode step for every unit u = (b, l, h) of the context's shape (N and w of the shape are not used
 * beyond sizing).  Unit u owns rows offsets[u] .. offsets[u+1] - 1 of the ragged cache (the layout
 * uncomp_compact writes: its capacity is the head's token budget) of which the first lens[u] are filled.
 *   p[j]   = sum over the G query heads g of softmax_j(scale * <qnew[u*G+g, :], k_j>), j over the lens[u]
 *            cached keys and, as entry lens[u], the new token's own key
 *   cum[j] += p[j] for the cached entries; the new token's cumulative score starts at p[lens[u]]
 *   lens[u] <  capacity: the new token is appended, lens[u] += 1, evicted[u] = -1
 *   lens[u] == capacity: the cached entry with the lowest cum among those with pos <= new_pos[b] - protect
 *            leaves (equal scores: the lower position; no such entry: all cached entries are candidates),
 *            evicted[u] = its position, and the new token takes its ROW: rows of a unit are not kept in
 *            position order, d_pos names the position of each row.
 * Readings where the paper is silent: grouped query heads are summed as in the prefill scorer; the new
 * token cannot leave in the step that adds it (protect >= 1 newest positions are never candidates).
 *
 * d_qnew     in      [B, L, Hq, d] contiguous, storage dtype: the new token's queries
 * d_knew     in      [B, L, H, d] contiguous; d_vnew likewise: the new token's key and value rows
 * d_new_pos  in      [B] int32, the new token's position in its sequence (larger than every cached pos)
 * d_offsets  in      [B*L*H + 1] int64
 * d_lens     in/out  [B*L*H] int32
 * max_cap            host: an upper bound of every unit's capacity, 1 <= max_cap <= N (sizes the grid)
 * total_cap          host: offsets[B*L*H]
 * protect            >= 1
 * scale              0 means 1 / sqrt(d)
 * d_Kc, d_Vc in/out  [total_cap, d] storage dtype, 16-byte aligned
 * d_pos      in/out  [total_cap] int32
 * d_cum      in/out  [total_cap] float
 * d_p        out     [total_cap + B*L*H] float, entry j of unit u at offsets[u] + u + j; may be NULL
 * d_evicted  out     [B*L*H] int32; may be NULL
 * Rejected: G not in {1, 2, 4, 8, 16} (UNCOMP_E_SHAPE); (total_cap + units) * G floats beyond the
 * workspace region that holds the logits, 2 * units * (N - w) floats (UNCOMP_E_LIMIT).  A unit whose
 * capacity is 0 or above max_cap, or whose length is outside [0, capacity], is left untouched and raises
 * UNCOMP_STATUS_BOUNDS.
 * ------------------------------------------------------------------------------------------------- */
int uncomp_decode_update(uncomp_ctx *ctx, const void *d_qnew, const void *d_knew, const void *d_vnew,
                         const int32_t *d_new_pos, const int64_t *d_offsets, int32_t *d_lens, int32_t max_cap,
                         int64_t total_cap, int32_t protect, float scale, void *d_Kc, void *d_Vc, int32_t *d_pos,
                         float *d_cum, float *d_p, int32_t *d_evicted, void *stream);

/* ---------------------------------------------------------------------------------------------------
 * uncomp_prepare_groups -- Section 3.3.1 "Preparation Stage" (the effective rank of each head averaged
 * over the d sampled data points) and Algorithm 1 (each sample assigns every head to one of M clusters by
 * its truncated entropy; the final label of a head is the majority vote).  With M = 2 the labels are the
 * retrieval / streaming split of Section 3.3.3 "Retrieval Head" (label 0: the high-rank group).
 *
 * L and H come from the context's shape.  A ranking set is one layer (scope 0, n = H) or the whole model
 * (scope 1, n = L*H); inside a set heads are ranked by descending value, equal values by ascending index,
 * and rank r belongs to group g with floor(g n / M) <= r < floor((g+1) n / M), the grouping
 * uncomp_assign_budgets uses.  Reading: the paper names no clustering algorithm; this equal-size
 * rank-based grouping is used for the per-sample clusters too.
 *   mean[l,h]       = (1/S) sum_i erank[i,l,h]  (fp64 accumulation in a fixed order, rounded to float)
 *   group_mean[l,h] = group of head (l,h) when the set is ranked by mean
 *   votes[l,h,g]    = number of samples whose own ranking puts head (l,h) in group g
 *   group_vote[l,h] = arg max_g votes[l,h,g], the lowest g on a tie
 *
 * d_erank       in   [S, L, H] float, e.g. the d_erank output of uncomp_entropy for a batch of S samples
 * S                  1 <= S <= 65535;  M: 1 <= M <= n;  n <= 8192 (UNCOMP_E_LIMIT beyond)
 * d_mean        out  [L, H] float
 * d_group_mean  out  [L, H] int32
 * d_votes       out  [L, H, M] int32 (cleared by the call)
 * d_group_vote  out  [L, H] int32
 * ------------------------------------------------------------------------------------------------- */
int uncomp_prepare_groups(uncomp_ctx *ctx, const float *d_erank, int32_t S, int32_t M, int32_t scope, float *d_mean,
                          int32_t *d_group_mean, int32_t *d_votes, int32_t *d_group_vote, void *stream);

/* ---------------------------------------------------------------------------------------------------
 * uncomp_entropy_wide -- Section 3.1 Eq. 1 for token vectors x_i in R^D with D beyond a head (the hidden
 * states of a layer, D = 4096, or the heads of a layer side by side), Lemma 2 and Section 3.2: the same
 * H_k and erank_k as uncomp_entropy, of `count` matrices X_i [N, D] (bf16; the context must be a bf16
 * one).  The D x D scatter matrix is formed on the tensor cores, tridiagonalised in fp32 by one
 * cooperative kernel that spans the GPU and its k largest eigenvalues are found in fp64 (Sturm counts).
 *
 * d_X            in   matrix i starts at element i * stride_matrix; token rows stride_row elements apart
 *                     (stride_row >= D, both strides multiples of 8 elements), features contiguous
 * N, D                N >= 2; 128 <= D <= 4096 (UNCOMP_E_LIMIT beyond), D a multiple of 64
 * params              as for uncomp_entropy, k_trunc <= 256
 * d_scratch           caller-owned device memory, 256-byte aligned, at least
 *                     uncomp_entropy_wide_scratch_bytes(N, D) bytes (0 for an unsupported shape); the
 *                     matrices are processed one after the other and share it
 * d_entropy      out  [count] float;  d_erank out [count] float, may be NULL
 * d_spectrum     out  [count, min(k_trunc, D)] double, the largest eigenvalues, descending; may be NULL
 * The cooperative kernel needs the GPU to itself while it runs: launching it on a device whose SMs are
 * held by another long-running kernel delays it, it never deadlocks (its grid barrier gives up after a
 * bounded number of polls and raises UNCOMP_STATUS_TIMEOUT).
 * ------------------------------------------------------------------------------------------------- */
size_t uncomp_entropy_wide_scratch_bytes(int32_t N, int32_t D);
int uncomp_entropy_wide(uncomp_ctx *ctx, const void *d_X, int32_t count, int64_t stride_matrix, int64_t stride_row,
                        int32_t N, int32_t D, const uncomp_entropy_params *params, void *d_scratch, size_t scratch_bytes,
                        float *d_entropy, float *d_erank, double *d_spectrum, void *stream);

/* uncomp_measure_l2_sweep -- measurement aid, no counterpart in the paper: the memory pattern of the
 * tridiagonalisation sweep of uncomp_entropy_wide on its own (a warp per row, every element read, changed by
 * one fused multiply-add and written back, `passes` times).  Timed by the caller with events on `stream`, a
 * matrix that fits in L2 gives the bandwidth that sweep can be held against.  d_A [rows, cols] float, device,
 * 16-byte aligned, cols a multiple of 4; its contents are overwritten. */
int uncomp_measure_l2_sweep(float *d_A, int32_t rows, int32_t cols, int32_t passes, void *stream);

/* ---------------------------------------------------------------------------------------------------
 * uncomp_compress -- the whole pass in one call: Section 3.1 - 3.2 (entropy), Section 3.3.3 (budgets, window
 * scores, selection, per-head cache), in the order that needs the fewest sweeps over K.  Results are those of
 * uncomp_entropy, uncomp_assign_budgets, uncomp_score_select and uncomp_compact called one after the other
 * with the same arguments; what changes is the schedule:
 *   - d_lse given (bf16 keys): ONE sweep over K produces the window scores and the Gram partials of the entropy
 *     stage together; eigenvalues and budgets follow, then selection and gather.  The staged calls need two
 *     sweeps for the same result (uncomp_entropy cannot know the normalisers).  The Gram partials are then
 *     summed per scorer chunk, so entropies can differ from the staged calls in the last bits.
 *   - d_lse NULL (bf16 keys): the Gram + statistics sweep of uncomp_entropy, then eigenvalues and budgets on a
 *     second stream beside the merge and the column sums (only the selection needs both), joined again before
 *     the selection.  The second stream is a host object the context creates in the first such call; all work
 *     is ordered after what `stream` held at the call and `stream` waits for it: same results as the staged
 *     calls, bit for bit.
 *   - fp32 keys: the four staged calls.
 * sparams->reuse_stats is ignored.  Arguments, ownership and errors as for the four calls; d_erank is required
 * here (the budget rule reads it), d_scores may be NULL (scores stay in the workspace), d_layer_group /
 * d_layer_ctx both NULL or both given. */
int uncomp_compress(uncomp_ctx *ctx, const void *d_K, const void *d_V, uncomp_strides sK, uncomp_strides sV,
                    const void *d_Qw, const float *d_lse, const uncomp_entropy_params *eparams,
                    const uncomp_budget_params *bparams, const uncomp_score_params *sparams, float *d_entropy,
                    float *d_erank, int32_t *d_budgets, int64_t *d_offsets, int32_t *d_layer_group, int32_t *d_layer_ctx,
                    float *d_scores, int32_t *d_indices, void *d_Kc, void *d_Vc, void *stream);

/* ---------------------------------------------------------------------------------------------------
 * uncomp_eviction_plan -- Section 3.3.2 "Hidden State Eviction"; Algorithm 2, "compress hidden states":
 * where the prefill cuts the hidden states, read off the layer partition of ONE sequence as
 * uncomp_assign_budgets writes it.  Host function on HOST arrays (copy the L entries of the sequence back
 * first); launches nothing.  Before layer l, the first layer of a new layer group whose context is
 * smaller than what is still there, the hidden states are cut to layer_ctx[l] positions
 * (uncomp_evict_hidden with n_keep = layer_ctx[l], scored by layer l - 1).  A group whose context is not
 * smaller needs no call and is left out.
 *
 * layer_group, layer_ctx  in   [L] int32, host
 * out_layer, out_keep     out  [L] int32, host: the first `return value` entries are the calls to make
 * Returns the number of entries, or a negative error code (UNCOMP_E_NULL, UNCOMP_E_PARAM for L < 0).
 * ------------------------------------------------------------------------------------------------- */
int uncomp_eviction_plan(const int32_t *layer_group, const int32_t *layer_ctx, int32_t L, int32_t *out_layer,
                         int32_t *out_keep);

/* ---------------------------------------------------------------------------------------------------
 * uncomp_retrieval_layer -- Section 3.3.2 "Retrieval Layer": the retrieval layer is chosen as the layer of
 * maximum entropy increase.  d_values [L, H] holds a per-head value (the truncated entropy or the
 * effective rank, of one input or averaged by uncomp_prepare_groups); with e_l its mean over the heads of
 * layer l (fp64, head order), increase[l] = e_{l+1} - e_l and *d_layer = l* + 1 for the first l* with the
 * largest increase.  Readings: the layer AFTER the jump is reported, a tie goes to the earliest layer.
 * The paper then merges that layer's parameters with the last layer's by averaging; that is a change of
 * model weights and outside this library.
 *
 * d_values    in   [L, H] float (L, H of the context's shape; L >= 2, L <= 4096)
 * d_layer     out  [1] int32
 * d_increase  out  [L - 1] float; may be NULL
 * ------------------------------------------------------------------------------------------------- */
int uncomp_retrieval_layer(uncomp_ctx *ctx, const float *d_values, int32_t *d_layer, float *d_increase, void *stream);

/* Synchronise `stream`, copy the status word to *host_bits and clear it on the device.  The only call
 * that waits for the device. */
int uncomp_status(uncomp_ctx *ctx, void *stream, uint32_t *host_bits);

/* Options of a context (no counterpart in the paper).  UNCOMP_OPT_CUDA_CORES = 1 makes bf16 inputs take
 * the plain CUDA-core kernels that fp32 inputs always use instead of the tensor-core kernels: a
 * debugging aid for comparing the two. */
enum { UNCOMP_OPT_CUDA_CORES = 1 };
int uncomp_set_option(uncomp_ctx *ctx, int option, int value);

/* ---------------------------------------------------------------------------------------------------
 * Per-kernel timing (no counterpart in the paper; it serves measurement).  While enabled, every kernel
 * the four calls launch is bracketed by a pair of CUDA events on the caller's stream.
 * uncomp_profile_read waits for the recorded events, adds the elapsed milliseconds and the launch
 * counts per kernel slot into ms_sum / launches (host arrays of max_slots entries) and forgets the
 * records.  Events are host-side driver objects; no device memory is allocated.
 * ------------------------------------------------------------------------------------------------- */
int uncomp_profile_enable(uncomp_ctx *ctx, int on);
int uncomp_profile_slots(void);
const char *uncomp_profile_slot_name(int slot);
int uncomp_profile_read(uncomp_ctx *ctx, int max_slots, float *ms_sum, int32_t *launches);

/* Text for a return code; never NULL. */
const char *uncomp_strerror(int code);

/* The cudaError_t (as int) behind the most recent UNCOMP_E_CUDA of this context, else 0. */
int uncomp_last_cuda_error(const uncomp_ctx *ctx);

/* Library version: major * 10000 + minor * 100 + patch. */
int uncomp_version(void);

#ifdef __cplusplus
}
#endif
#endif /* UNCOMP_H_ */
