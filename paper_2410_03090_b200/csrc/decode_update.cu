// Decode-time update of the ragged per-head cache (paper Section 3.3.3, "Dynamic KV Cache Eviction", last
// sentence: as new tokens are generated, the token with the lowest cumulative attention score leaves;
// Algorithm 2, decoding loop: the new token is concatenated with the head's cache and attends over it).
//
// Per unit (batch, layer, KV head) with a cache of len entries inside a slab of cap rows:
//   p[j]   = sum over the G query heads of softmax_j(scale * q_g . k_j), j over the len cached keys and the
//            new token's own key (entry len);
//   cum[j] += p[j] for the cached entries; the new token starts with p[len];
//   len < cap : the new token is appended;
//   len == cap: the entry with the lowest cum among those with pos <= new_pos - protect leaves (equal
//               scores: the lower position; no such entry: every cached entry is a candidate) and the new
//               token takes its row, so the slab is not kept in position order: `pos` names each row.
//
// The step is bound by reading the cached keys once.  Three launches:
//   1. logits      grid (chunks of 1024 entries, units): the G logits of every entry (log2 domain) to scratch,
//                  per chunk the softmax statistics (max, sum of 2^(x - max)) per query head;
//   2. accumulate  same grid: merges the chunk statistics, forms p, updates cum, and leaves per chunk the
//                  lexicographic minimum of (cum, pos) over the candidates and over all entries;
//   3. commit      one small CTA per unit: picks the row, copies the new key / value rows, updates pos, cum, len.
// Positions are unique inside a unit, so every minimum is unique and no result depends on thread order.
#include "common.cuh"

namespace uncomp {

namespace {
constexpr int kDecThreads = 256;
constexpr int kDecWarps = kDecThreads / 32;
constexpr int kDecChunk = 1024;

__device__ __forceinline__ float ex2f(float x) {
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}

struct MinRec {          // candidate for eviction: (cum, pos) ordered lexicographically; pos < 0 means none
    float c;
    int32_t pos, j;
};
struct MinPair {
    MinRec el, any;      // among the entries old enough / among all cached entries
};

__device__ __forceinline__ bool rec_less(float c, int32_t pos, const MinRec &b) {
    return b.pos < 0 || c < b.c || (c == b.c && pos < b.pos);
}
__device__ __forceinline__ void rec_take(MinRec &a, const MinRec &b) {
    if (b.pos >= 0 && rec_less(b.c, b.pos, a)) a = b;
}

__device__ __forceinline__ void mma_bf16_16816(float (&c)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3,
                                               uint32_t b0, uint32_t b1) {
    asm volatile(
        "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0, %1, %2, %3}, {%4, %5, %6, %7}, {%8, %9}, "
        "{%0, %1, %2, %3};"
        : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
        : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}

struct DecArgs {
    const void *q, *knew;            // [units * G, d], [units, d]
    const void *Kc;                  // [total_cap, d]
    const int64_t *offsets;          // [units + 1]
    const int32_t *lens;             // [units]
    int units, G, max_cap, chunks_max;
    float c_log2;
    float *logits;                   // [(total_cap + units) * G]
    float *stats;                    // [units, chunks_max, G, 2]
};

// Entry e of unit u sits at row offsets[u] + u + e of the scratch (and of the optional p output): every unit
// has one more entry than its slab has rows.
__device__ __forceinline__ bool unit_ok(const DecArgs &a, int u, int64_t &off, int &len) {
    off = a.offsets[u];
    const int64_t cap = a.offsets[u + 1] - off;
    len = a.lens[u];
    return cap >= 1 && cap <= a.max_cap && len >= 0 && len <= cap;
}

// bf16: the warp-level tensor-core instruction on 16 entries x 16 features times 16 features x 8 heads.  Both
// operands are loaded in the order that makes the loads contiguous (lane (gid, tig) reads bytes
// [64 j + 16 tig, +16) of key rows gid and gid + 8 and of query head gid); a dot product does not depend on the
// order in which the features are visited.  fp32 accumulation, scaled afterwards.
template <int G>
__global__ void __launch_bounds__(kDecThreads) decode_logits_mma_kernel(DecArgs a) {
    constexpr int NB = (G + 7) / 8;
    __shared__ float red_m[kDecWarps][32][NB * 2], red_l[kDecWarps][32][NB * 2];
    const int c = blockIdx.x, u = blockIdx.y;
    int64_t off;
    int len;
    if (!unit_ok(a, u, off, len)) return;
    const int n = len + 1;
    const int t0 = c * kDecChunk, t1 = min(n, t0 + kDecChunk);
    if (t0 >= n) return;
    const int tid = threadIdx.x, lane = tid & 31, wid = tid >> 5, gid = lane >> 2, tig = lane & 3;
    const __nv_bfloat16 *qb = (const __nv_bfloat16 *)a.q + (size_t)u * G * kD;
    const __nv_bfloat16 *Kb = (const __nv_bfloat16 *)a.Kc + off * kD;
    const __nv_bfloat16 *kn = (const __nv_bfloat16 *)a.knew + (size_t)u * kD;
    uint32_t bq[NB][16];
#pragma unroll
    for (int nb = 0; nb < NB; ++nb) {
        const int h = nb * 8 + gid;
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            uint4 x = make_uint4(0u, 0u, 0u, 0u);
            if (h < G) x = reinterpret_cast<const uint4 *>(qb + (size_t)h * kD)[4 * j + tig];
            bq[nb][4 * j] = x.x; bq[nb][4 * j + 1] = x.y; bq[nb][4 * j + 2] = x.z; bq[nb][4 * j + 3] = x.w;
        }
    }
    float m_run[NB][2], l_run[NB][2];
#pragma unroll
    for (int nb = 0; nb < NB; ++nb)
#pragma unroll
        for (int i = 0; i < 2; ++i) { m_run[nb][i] = -1e30f; l_run[nb][i] = 0.f; }
    float *lg = a.logits + (off + u) * G;
    for (int base = t0 + wid * 32; base < t1; base += kDecWarps * 32) {
        uint4 ka[2][2][4];
#pragma unroll
        for (int tile = 0; tile < 2; ++tile)
#pragma unroll
            for (int half = 0; half < 2; ++half) {
                const int row = base + tile * 16 + half * 8 + gid;
                const uint4 *src = reinterpret_cast<const uint4 *>(row < len ? Kb + (int64_t)row * kD : kn);
#pragma unroll
                for (int j = 0; j < 4; ++j) ka[tile][half][j] = row < t1 ? src[4 * j + tig] : make_uint4(0u, 0u, 0u, 0u);
            }
#pragma unroll
        for (int tile = 0; tile < 2; ++tile)
#pragma unroll
            for (int nb = 0; nb < NB; ++nb) {
                float acc[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
                for (int j = 0; j < 4; ++j) {
                    const uint4 lo = ka[tile][0][j], hi = ka[tile][1][j];
                    mma_bf16_16816(acc, lo.x, hi.x, lo.y, hi.y, bq[nb][4 * j], bq[nb][4 * j + 1]);
                    mma_bf16_16816(acc, lo.z, hi.z, lo.w, hi.w, bq[nb][4 * j + 2], bq[nb][4 * j + 3]);
                }
                // acc[0], acc[1]: entry gid, heads 2 tig and 2 tig + 1;  acc[2], acc[3]: entry gid + 8
#pragma unroll
                for (int i = 0; i < 2; ++i) {
                    const int h = nb * 8 + 2 * tig + i;
                    if (h < G) {
#pragma unroll
                        for (int half = 0; half < 2; ++half) {
                            const int t = base + tile * 16 + half * 8 + gid;
                            if (t < t1) {
                                const float v = acc[2 * half + i] * a.c_log2;
                                lg[(int64_t)t * G + h] = v;
                                const float m_new = fmaxf(m_run[nb][i], v);
                                l_run[nb][i] = fmaf(l_run[nb][i], ex2f(m_run[nb][i] - m_new), ex2f(v - m_new));
                                m_run[nb][i] = m_new;
                            }
                        }
                    }
                }
            }
    }
#pragma unroll
    for (int nb = 0; nb < NB; ++nb)
#pragma unroll
        for (int i = 0; i < 2; ++i) { red_m[wid][lane][nb * 2 + i] = m_run[nb][i]; red_l[wid][lane][nb * 2 + i] = l_run[nb][i]; }
    __syncthreads();
    if (tid < G) {   // fixed order: warps 0.., then the 8 row lanes that hold this head
        const int nb = tid >> 3, tg = (tid & 7) >> 1, i = tid & 1;
        float m = -1e30f;
        for (int x = 0; x < kDecWarps; ++x)
            for (int g8 = 0; g8 < 8; ++g8) m = fmaxf(m, red_m[x][g8 * 4 + tg][nb * 2 + i]);
        float l_sum = 0.f;
        for (int x = 0; x < kDecWarps; ++x)
            for (int g8 = 0; g8 < 8; ++g8)
                l_sum += red_l[x][g8 * 4 + tg][nb * 2 + i] * ex2f(red_m[x][g8 * 4 + tg][nb * 2 + i] - m);
        float *o = a.stats + (((size_t)u * a.chunks_max + c) * G + tid) * 2;
        o[0] = m;
        o[1] = l_sum;
    }
}

// fp32 keys: a warp per entry, a lane holds 4 features, the G dot products are reduced by shuffles.
__global__ void __launch_bounds__(kDecThreads) decode_logits_f32_kernel(DecArgs a) {
    __shared__ __align__(16) float qs[16][kD];
    __shared__ float red_m[kDecWarps][16], red_l[kDecWarps][16];
    const int c = blockIdx.x, u = blockIdx.y, G = a.G;
    int64_t off;
    int len;
    if (!unit_ok(a, u, off, len)) return;
    const int n = len + 1;
    const int t0 = c * kDecChunk, t1 = min(n, t0 + kDecChunk);
    if (t0 >= n) return;
    const int tid = threadIdx.x, lane = tid & 31, wid = tid >> 5;
    const float *qb = (const float *)a.q + (size_t)u * G * kD;
    for (int e = tid; e < G * kD; e += kDecThreads) qs[e / kD][e % kD] = qb[e];
    __syncthreads();
    const float *Kb = (const float *)a.Kc + off * kD;
    const float *kn = (const float *)a.knew + (size_t)u * kD;
    float *lg = a.logits + (off + u) * G;
    float m_run = -1e30f, l_run = 0.f;   // lane g < G keeps the statistics of head g
    for (int t = t0 + wid; t < t1; t += kDecWarps) {
        const float4 k4 = *reinterpret_cast<const float4 *>((t < len ? Kb + (int64_t)t * kD : kn) + lane * 4);
        float mine = 0.f;
        for (int g = 0; g < G; ++g) {
            const float4 q4 = *reinterpret_cast<const float4 *>(&qs[g][lane * 4]);
            float v = fmaf(k4.x, q4.x, fmaf(k4.y, q4.y, fmaf(k4.z, q4.z, k4.w * q4.w)));
            v = warp_sum(v) * a.c_log2;
            if (lane == g) mine = v;
        }
        if (lane < G) {
            lg[(int64_t)t * G + lane] = mine;
            const float m_new = fmaxf(m_run, mine);
            l_run = fmaf(l_run, ex2f(m_run - m_new), ex2f(mine - m_new));
            m_run = m_new;
        }
    }
    if (lane < G) { red_m[wid][lane] = m_run; red_l[wid][lane] = l_run; }
    __syncthreads();
    if (tid < G) {
        float m = -1e30f;
        for (int x = 0; x < kDecWarps; ++x) m = fmaxf(m, red_m[x][tid]);
        float l_sum = 0.f;
        for (int x = 0; x < kDecWarps; ++x) l_sum += red_l[x][tid] * ex2f(red_m[x][tid] - m);
        float *o = a.stats + (((size_t)u * a.chunks_max + c) * G + tid) * 2;
        o[0] = m;
        o[1] = l_sum;
    }
}

__global__ void __launch_bounds__(kDecThreads) decode_accumulate_kernel(DecArgs a, int H_per_seq, const int32_t *new_pos,
                                                                       int protect, const int32_t *pos, float *cum,
                                                                       float *p_out, MinPair *partial, float *new_cum) {
    __shared__ float mprime[16];
    __shared__ MinPair red[kDecWarps];
    const int c = blockIdx.x, u = blockIdx.y, G = a.G, tid = threadIdx.x, lane = tid & 31, wid = tid >> 5;
    int64_t off;
    int len;
    if (!unit_ok(a, u, off, len)) return;
    const int n = len + 1, chunks = (n + kDecChunk - 1) / kDecChunk;
    if (c >= chunks) return;
    if (tid < G) {
        const float *s = a.stats + ((size_t)u * a.chunks_max * G + tid) * 2;
        float m = -1e30f;
        for (int x = 0; x < chunks; ++x) m = fmaxf(m, s[(size_t)x * G * 2]);
        float l = 0.f;
        for (int x = 0; x < chunks; ++x) l += s[(size_t)x * G * 2 + 1] * exp2f(s[(size_t)x * G * 2] - m);
        mprime[tid] = m + log2f(l);
    }
    __syncthreads();
    const int limit = new_pos[u / H_per_seq] - protect;   // candidates have pos <= limit
    const float *lg = a.logits + (off + u) * G;
    MinPair best;
    best.el.c = best.any.c = 0.f;
    best.el.pos = best.any.pos = -1;
    best.el.j = best.any.j = -1;
    const int t1 = min(n, (c + 1) * kDecChunk);
    for (int j = c * kDecChunk + tid; j < t1; j += kDecThreads) {
        float p = 0.f;   // heads in ascending order, whichever load width is used
        if ((G & 3) == 0) {
            const float4 *l4 = reinterpret_cast<const float4 *>(lg + (int64_t)j * G);
            for (int g = 0; g < G; g += 4) {
                const float4 x = l4[g >> 2];
                p += ex2f(x.x - mprime[g]);
                p += ex2f(x.y - mprime[g + 1]);
                p += ex2f(x.z - mprime[g + 2]);
                p += ex2f(x.w - mprime[g + 3]);
            }
        } else {
            for (int g = 0; g < G; ++g) p += ex2f(lg[(int64_t)j * G + g] - mprime[g]);
        }
        if (p_out) p_out[off + u + j] = p;
        if (j < len) {
            const float cn = cum[off + j] + p;
            cum[off + j] = cn;
            const int32_t ps = pos[off + j];
            if (rec_less(cn, ps, best.any)) { best.any.c = cn; best.any.pos = ps; best.any.j = j; }
            if (ps <= limit && rec_less(cn, ps, best.el)) { best.el.c = cn; best.el.pos = ps; best.el.j = j; }
        } else {
            new_cum[u] = p;
        }
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        MinPair other;
        other.el.c = __shfl_xor_sync(0xffffffffu, best.el.c, o);
        other.el.pos = __shfl_xor_sync(0xffffffffu, best.el.pos, o);
        other.el.j = __shfl_xor_sync(0xffffffffu, best.el.j, o);
        other.any.c = __shfl_xor_sync(0xffffffffu, best.any.c, o);
        other.any.pos = __shfl_xor_sync(0xffffffffu, best.any.pos, o);
        other.any.j = __shfl_xor_sync(0xffffffffu, best.any.j, o);
        rec_take(best.el, other.el);
        rec_take(best.any, other.any);
    }
    if (lane == 0) red[wid] = best;
    __syncthreads();
    if (tid == 0) {
        for (int x = 1; x < kDecWarps; ++x) { rec_take(best.el, red[x].el); rec_take(best.any, red[x].any); }
        partial[(size_t)u * a.chunks_max + c] = best;
    }
}

__global__ void __launch_bounds__(64) decode_commit_kernel(DecArgs a, int H_per_seq, const int32_t *new_pos,
                                                          const void *vnew, int row_bytes, void *Kc, void *Vc,
                                                          int32_t *pos, float *cum, int32_t *lens, int32_t *evicted,
                                                          const MinPair *partial, const float *new_cum,
                                                          uint32_t *status) {
    __shared__ int slot_s;
    const int u = blockIdx.x, tid = threadIdx.x;
    int64_t off;
    int len;
    if (!unit_ok(a, u, off, len)) {
        if (tid == 0) {
            atomicOr(status, (uint32_t)UNCOMP_STATUS_BOUNDS);
            if (evicted) evicted[u] = -1;
        }
        return;
    }
    const int64_t cap = a.offsets[u + 1] - off;
    if (tid == 0) {
        int slot = len, gone = -1;
        if (len >= cap) {
            const int chunks = (len + 1 + kDecChunk - 1) / kDecChunk;
            MinPair best = partial[(size_t)u * a.chunks_max];
            for (int x = 1; x < chunks; ++x) {
                const MinPair o = partial[(size_t)u * a.chunks_max + x];
                rec_take(best.el, o.el);
                rec_take(best.any, o.any);
            }
            const MinRec &r = best.el.pos >= 0 ? best.el : best.any;
            slot = r.j;
            gone = r.pos;
        } else {
            lens[u] = len + 1;
        }
        if (!UNCOMP_INDEX_OK(slot, cap, status)) slot = -1;       // debug library: the row must lie in the unit's slab
        if (slot >= 0) {
            pos[off + slot] = new_pos[u / H_per_seq];
            cum[off + slot] = new_cum[u];
        }
        if (evicted) evicted[u] = gone;
        slot_s = slot;
    }
    __syncthreads();
    const int slot = slot_s, vecs = row_bytes >> 4;      // 16-byte vectors per row: 16 (bf16) or 32 (fp32)
    if (slot < 0) return;                                // only the debug library can get here
    const int4 *srcK = reinterpret_cast<const int4 *>((const char *)a.knew + (size_t)u * row_bytes);
    const int4 *srcV = reinterpret_cast<const int4 *>((const char *)vnew + (size_t)u * row_bytes);
    int4 *dstK = reinterpret_cast<int4 *>((char *)Kc + (off + slot) * row_bytes);
    int4 *dstV = reinterpret_cast<int4 *>((char *)Vc + (off + slot) * row_bytes);
    if (tid < 32) { if (tid < vecs) dstK[tid] = srcK[tid]; }
    else if (tid - 32 < vecs) dstV[tid - 32] = srcV[tid - 32];
}
// Cumulative scores right after prefill: a kept prefix position takes its prefill score, a window position the
// largest score among the kept prefix positions of its head (0 if there is none).  One CTA per unit.
__global__ void __launch_bounds__(256) decode_seed_kernel(const float *__restrict__ scores, int P,
                                                         const int32_t *__restrict__ indices,
                                                         const int64_t *__restrict__ offsets, float *__restrict__ cum) {
    __shared__ float red[8];
    const int u = blockIdx.x, tid = threadIdx.x, lane = tid & 31, wid = tid >> 5;
    const int64_t off = offsets[u];
    const int n = (int)(offsets[u + 1] - off);
    const float *s = scores + (size_t)u * P;
    float top = -INFINITY;
    for (int t = tid; t < n; t += 256) {
        const int j = indices[off + t];
        if (j < P) top = fmaxf(top, s[j]);
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) top = fmaxf(top, __shfl_xor_sync(0xffffffffu, top, o));
    if (lane == 0) red[wid] = top;
    __syncthreads();
    top = red[0];
#pragma unroll
    for (int i = 1; i < 8; ++i) top = fmaxf(top, red[i]);
    if (top == -INFINITY) top = 0.f;
    for (int t = tid; t < n; t += 256) {
        const int j = indices[off + t];
        cum[off + t] = j < P ? s[j] : top;
    }
}
}  // namespace

cudaError_t launch_decode_seed(const Plan &p, const float *d_scores, const int32_t *d_indices, const int64_t *d_offsets,
                               float *d_cum, cudaStream_t st) {
    decode_seed_kernel<<<p.units, 256, 0, st>>>(d_scores, p.prefix, d_indices, d_offsets, d_cum);
    return cudaGetLastError();
}

int decode_chunks(int max_cap) { return (max_cap + 1 + kDecChunk - 1) / kDecChunk; }
size_t decode_partial_bytes() { return sizeof(MinPair); }

cudaError_t launch_decode_update(const Plan &p, const void *d_q, const void *d_knew, const void *d_vnew,
                                 const int32_t *d_new_pos, const int64_t *d_offsets, int32_t *d_lens, int max_cap,
                                 int protect, float scale, void *d_Kc, void *d_Vc, int32_t *d_pos, float *d_cum,
                                 float *d_p, int32_t *d_evicted, float *d_logits, float *d_stats, void *d_partial,
                                 float *d_new_cum, uint32_t *d_status, Profiler *prof, cudaStream_t st) {
    const uncomp_shape &s = p.shape;
    DecArgs a;
    a.q = d_q; a.knew = d_knew; a.Kc = d_Kc; a.offsets = d_offsets; a.lens = d_lens;
    a.units = p.units; a.G = p.G; a.max_cap = max_cap; a.chunks_max = decode_chunks(max_cap);
    a.c_log2 = scale * 1.4426950408889634f;
    a.logits = d_logits; a.stats = d_stats;
    const dim3 grid(a.chunks_max, p.units);
    const int row_bytes = kD * (s.dtype == UNCOMP_FP32 ? 4 : 2);
    {
        ProfScope ps(prof, kSlotDecodeLogits, st);
        if (s.dtype == UNCOMP_FP32) decode_logits_f32_kernel<<<grid, kDecThreads, 0, st>>>(a);
        else switch (p.G) {
            case 1: decode_logits_mma_kernel<1><<<grid, kDecThreads, 0, st>>>(a); break;
            case 2: decode_logits_mma_kernel<2><<<grid, kDecThreads, 0, st>>>(a); break;
            case 4: decode_logits_mma_kernel<4><<<grid, kDecThreads, 0, st>>>(a); break;
            case 8: decode_logits_mma_kernel<8><<<grid, kDecThreads, 0, st>>>(a); break;
            case 16: decode_logits_mma_kernel<16><<<grid, kDecThreads, 0, st>>>(a); break;
            default: return cudaErrorInvalidValue;
        }
    }
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return e;
    {
        ProfScope ps(prof, kSlotDecodeAccumulate, st);
        decode_accumulate_kernel<<<grid, kDecThreads, 0, st>>>(a, s.L * s.H, d_new_pos, protect, d_pos, d_cum, d_p,
                                                               (MinPair *)d_partial, d_new_cum);
    }
    {
        ProfScope ps(prof, kSlotDecodeCommit, st);
        decode_commit_kernel<<<p.units, 64, 0, st>>>(a, s.L * s.H, d_new_pos, d_vnew, row_bytes, d_Kc, d_Vc, d_pos, d_cum,
                                                     d_lens, d_evicted, (const MinPair *)d_partial, d_new_cum, d_status);
    }
    return cudaGetLastError();
}

}  // namespace uncomp
