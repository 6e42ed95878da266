// Hidden-state eviction between layer groups (paper Section 3.3.2, "Hidden State Eviction"; Algorithm 2,
// "compress hidden states"): the tokens whose hidden states go on to the next layer group are those with
// the highest attention scores of the LAST token of the current layer.
//
// Per sequence: score[j] = sum over the Hq query heads of softmax_j(scale * q_h . k_j), j over all N
// positions; the last position is always kept, the n_keep - 1 best of the first N - 1 join it (ties to
// the lower position), indices ascending; rows of the hidden-state matrix X [N, D] are gathered.
//
// The last token has one query row per head, so this is matrix-vector work bound by reading K once:
//   1. logits kernel   grid (token chunks, B*H): half a warp owns a token and reads its 128-feature key row
//                      as one coalesced line; the G dot products of its KV head against the query vectors
//                      (pre-scaled to the log2 domain) are summed over the lanes by a transposing butterfly;
//                      logits go to scratch, each chunk leaves (max, sum of 2^(x - max)) per query head;
//   2. scores kernel   merges the chunk statistics per head (fixed order) and adds 2^(x - m'_h) over heads;
//   3. selection       the radix select of select.cu with one unit per sequence;
//   4. row gather      a warp per kept row, 16-byte vectors, any row width that is a multiple of 16 bytes.
#include "common.cuh"

namespace uncomp {

namespace {
constexpr int kEvThreads = 256;

__device__ __forceinline__ float ex2f(float x) {
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}

template <typename T> struct Vec8;   // 8 consecutive features of a key row as floats
template <> struct Vec8<__nv_bfloat16> {
    __device__ static void load(const __nv_bfloat16 *p, float (&f)[8]) {
        const uint4 v = *reinterpret_cast<const uint4 *>(p);
        const uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            f[2 * i] = __uint_as_float(w[i] << 16);
            f[2 * i + 1] = __uint_as_float(w[i] & 0xffff0000u);
        }
    }
};
template <> struct Vec8<float> {
    __device__ static void load(const float *p, float (&f)[8]) {
        const float4 a = *reinterpret_cast<const float4 *>(p), b = *reinterpret_cast<const float4 *>(p + 4);
        f[0] = a.x; f[1] = a.y; f[2] = a.z; f[3] = a.w; f[4] = b.x; f[5] = b.y; f[6] = b.z; f[7] = b.w;
    }
};

// grid (chunks, B * H).  Half a warp owns a key row: its 16 lanes read the row's 256 bytes (bf16) as one
// coalesced 16-byte load each and hold their 8 features of the G query vectors in registers.  A warp takes
// 2 * R rows per round, R = 32 / G, which leaves G * R = 32 partial dot products per lane; a transposing
// butterfly (send one half of the values, keep the other, 16 + 8 + 4 + 2 shuffles) sums them over the 16
// lanes and leaves every lane two finished logits of ONE query head, the same head in every round, so the
// running (max, sum) of the softmax statistics stays private to the lane until the end of the chunk.
template <typename T, int G>
__global__ void __launch_bounds__(kEvThreads) last_token_logits_kernel(
    const T *__restrict__ qlast, const T *__restrict__ K, int H, int64_t sB, int64_t sH, int64_t sN, int N, int chunk,
    int chunks, float c_log2, float *__restrict__ logits, float *__restrict__ stats_part) {
    constexpr int R = 32 / G;                 // rows per half-warp and round
    constexpr bool kQReg = G <= 4;            // query features in registers; wider groups read them from smem
    constexpr int kWarps = kEvThreads / 32;
    __shared__ __align__(16) float qs[G][kD];
    __shared__ float red_m[kWarps][32], red_l[kWarps][32];
    const int c = blockIdx.x, bh = blockIdx.y, b = bh / H, h = bh % H;
    const int tid = threadIdx.x, lane = tid & 31, wid = tid >> 5, hw = lane >> 4, sub = lane & 15;
    const int Hq = H * G;
    for (int e = tid; e < G * kD; e += kEvThreads)
        qs[e / kD][e % kD] = to_float(qlast[((size_t)b * Hq + (size_t)h * G) * kD + e]) * c_log2;
    __syncthreads();
    float qr[kQReg ? G : 1][8];
    if (kQReg) {
#pragma unroll
        for (int g = 0; g < G; ++g)
#pragma unroll
            for (int i = 0; i < 8; ++i) qr[g][i] = qs[g][sub * 8 + i];
    }
    const T *Kb = K + b * sB + h * sH + sub * 8;
    // after the butterfly this lane holds values 2 * sub and 2 * sub + 1 of the index g * R + r
    const int my_g = (2 * sub) / R, my_r = (2 * sub) % R;
    float m_run = -1e30f, l_run = 0.f;
    float *my_logits = logits + ((size_t)b * Hq + (size_t)h * G + my_g) * N;
    const int t0 = c * chunk, t1 = min(N, t0 + chunk);
    for (int base = t0 + wid * 2 * R; base < t1; base += kWarps * 2 * R) {
        const int row0 = base + hw * R;       // this half-warp's R consecutive rows
        float v[32];
#pragma unroll
        for (int r = 0; r < R; ++r) {
            float kf[8];
            if (row0 + r < t1) Vec8<T>::load(Kb + (int64_t)(row0 + r) * sN, kf);
            else {
#pragma unroll
                for (int i = 0; i < 8; ++i) kf[i] = 0.f;
            }
#pragma unroll
            for (int g = 0; g < G; ++g) {
                float a = 0.f;
                if (kQReg) {
#pragma unroll
                    for (int i = 0; i < 8; ++i) a = fmaf(kf[i], qr[g][i], a);
                } else {
                    const float4 q0 = *reinterpret_cast<const float4 *>(&qs[g][sub * 8]);
                    const float4 q1 = *reinterpret_cast<const float4 *>(&qs[g][sub * 8 + 4]);
                    a = fmaf(kf[0], q0.x, a); a = fmaf(kf[1], q0.y, a); a = fmaf(kf[2], q0.z, a); a = fmaf(kf[3], q0.w, a);
                    a = fmaf(kf[4], q1.x, a); a = fmaf(kf[5], q1.y, a); a = fmaf(kf[6], q1.z, a); a = fmaf(kf[7], q1.w, a);
                }
                v[g * R + r] = a;
            }
        }
        // transposing butterfly over the 16 lanes of the half-warp: 32 -> 16 -> 8 -> 4 -> 2 values
#pragma unroll
        for (int o = 8, n = 32; o > 0; o >>= 1, n >>= 1) {
            const bool up = (lane & o) != 0;
#pragma unroll
            for (int i = 0; i < n / 2; ++i) {
                const float send = up ? v[i] : v[i + n / 2];
                const float keep = up ? v[i + n / 2] : v[i];
                v[i] = keep + __shfl_xor_sync(0xffffffffu, send, o);
            }
        }
#pragma unroll
        for (int i = 0; i < 2; ++i) {
            const int t = row0 + my_r + i;
            if (t < t1) {
                my_logits[t] = v[i];
                const float m_new = fmaxf(m_run, v[i]);
                l_run = fmaf(l_run, ex2f(m_run - m_new), ex2f(v[i] - m_new));
                m_run = m_new;
            }
        }
    }
    // block reduction of (m, l) per query head in a fixed order: warps 0.., lanes 0..31 of the head
    red_m[wid][lane] = m_run;
    red_l[wid][lane] = l_run;
    __syncthreads();
    if (tid < G) {
        float m = -1e30f;
        for (int x = 0; x < kWarps; ++x)
            for (int l = 0; l < 32; ++l)
                if ((2 * (l & 15)) / R == tid) m = fmaxf(m, red_m[x][l]);
        float l_sum = 0.f;
        for (int x = 0; x < kWarps; ++x)
            for (int l = 0; l < 32; ++l)
                if ((2 * (l & 15)) / R == tid) l_sum += red_l[x][l] * ex2f(red_m[x][l] - m);
        float *o = stats_part + (((size_t)b * Hq + (size_t)h * G + tid) * chunks + c) * 2;
        o[0] = m;
        o[1] = l_sum;
    }
}

// The same step for bf16 keys with the warp-level tensor-core instruction (16 rows x 16 features times
// 16 features x 8 heads): with scalar arithmetic the kernel issues about 30 instructions per key row, two
// thirds of what the SM can issue in the time HBM delivers the row, and ends up issue-bound; here a round
// of 32 rows costs 16 loads and 16 (x NB) matrix instructions and the kernel waits on memory only.
// A dot product does not care in which order the features are visited, so both operands use the
// feature order that makes the loads contiguous: lane (gid, tig) reads bytes [64 j + 16 tig, +16) of key
// rows gid and gid + 8, j = 0..3 (the four lanes of a row cover 64 contiguous bytes per load), and the
// same bytes of query head gid for the right-hand operand; the two 32-bit halves of each 8-byte half of
// such a vector are the instruction's feature slots {2 tig, 2 tig + 1} and {2 tig + 8, 2 tig + 9}.
// The products are exact in fp32 and accumulate in fp32; the logit is scaled afterwards.
__device__ __forceinline__ void mma_bf16_16816(float (&c)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3,
                                               uint32_t b0, uint32_t b1) {
    asm volatile(
        "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0, %1, %2, %3}, {%4, %5, %6, %7}, {%8, %9}, "
        "{%0, %1, %2, %3};"
        : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
        : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}

template <int G>
__global__ void __launch_bounds__(kEvThreads) last_token_logits_mma_kernel(
    const __nv_bfloat16 *__restrict__ qlast, const __nv_bfloat16 *__restrict__ K, int H, int64_t sB, int64_t sH,
    int64_t sN, int N, int chunk, int chunks, float c_log2, float *__restrict__ logits,
    float *__restrict__ stats_part) {
    constexpr int NB = (G + 7) / 8;           // 8-head column blocks
    constexpr int kWarps = kEvThreads / 32;
    __shared__ float red_m[kWarps][32][NB * 2], red_l[kWarps][32][NB * 2];
    const int c = blockIdx.x, bh = blockIdx.y, b = bh / H, h = bh % H;
    const int tid = threadIdx.x, lane = tid & 31, wid = tid >> 5, gid = lane >> 2, tig = lane & 3;
    const int Hq = H * G;
    const __nv_bfloat16 *qb = qlast + ((size_t)b * Hq + (size_t)h * G) * kD;
    uint32_t bq[NB][16];
#pragma unroll
    for (int nb = 0; nb < NB; ++nb) {
        const int n = nb * 8 + gid;
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            uint4 x = make_uint4(0u, 0u, 0u, 0u);
            if (n < G) x = reinterpret_cast<const uint4 *>(qb + (size_t)n * kD)[4 * j + tig];
            bq[nb][4 * j] = x.x; bq[nb][4 * j + 1] = x.y; bq[nb][4 * j + 2] = x.z; bq[nb][4 * j + 3] = x.w;
        }
    }
    const __nv_bfloat16 *Kb = K + b * sB + h * sH;
    float m_run[NB][2], l_run[NB][2];
#pragma unroll
    for (int nb = 0; nb < NB; ++nb)
#pragma unroll
        for (int i = 0; i < 2; ++i) { m_run[nb][i] = -1e30f; l_run[nb][i] = 0.f; }
    const int t0 = c * chunk, t1 = min(N, t0 + chunk);
    for (int base = t0 + wid * 32; base < t1; base += kWarps * 32) {
        uint4 ka[2][2][4];                    // [16-row tile][rows gid / gid + 8][j]
#pragma unroll
        for (int tile = 0; tile < 2; ++tile)
#pragma unroll
            for (int half = 0; half < 2; ++half) {
                const int row = base + tile * 16 + half * 8 + gid;
                const uint4 *src = reinterpret_cast<const uint4 *>(Kb + (int64_t)row * sN);
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
                // acc[0], acc[1]: row gid, heads 2 tig and 2 tig + 1;  acc[2], acc[3]: row gid + 8
#pragma unroll
                for (int i = 0; i < 2; ++i) {
                    const int n = nb * 8 + 2 * tig + i;
                    if (n < G) {
                        float *dst = logits + ((size_t)b * Hq + (size_t)h * G + n) * N;
#pragma unroll
                        for (int half = 0; half < 2; ++half) {
                            const int t = base + tile * 16 + half * 8 + gid;
                            if (t < t1) {
                                const float v = acc[2 * half + i] * c_log2;
                                dst[t] = v;
                                const float m_new = fmaxf(m_run[nb][i], v);
                                l_run[nb][i] = fmaf(l_run[nb][i], ex2f(m_run[nb][i] - m_new), ex2f(v - m_new));
                                m_run[nb][i] = m_new;
                            }
                        }
                    }
                }
            }
    }
    // block reduction of (m, l) per query head in a fixed order: warps 0.., then the 8 row lanes of the head
#pragma unroll
    for (int nb = 0; nb < NB; ++nb)
#pragma unroll
        for (int i = 0; i < 2; ++i) { red_m[wid][lane][nb * 2 + i] = m_run[nb][i]; red_l[wid][lane][nb * 2 + i] = l_run[nb][i]; }
    __syncthreads();
    if (tid < G) {
        const int nb = tid >> 3, tg = (tid & 7) >> 1, i = tid & 1;
        float m = -1e30f;
        for (int x = 0; x < kWarps; ++x)
            for (int g8 = 0; g8 < 8; ++g8) m = fmaxf(m, red_m[x][g8 * 4 + tg][nb * 2 + i]);
        float l_sum = 0.f;
        for (int x = 0; x < kWarps; ++x)
            for (int g8 = 0; g8 < 8; ++g8)
                l_sum += red_l[x][g8 * 4 + tg][nb * 2 + i] * ex2f(red_m[x][g8 * 4 + tg][nb * 2 + i] - m);
        float *o = stats_part + (((size_t)b * Hq + (size_t)h * G + tid) * chunks + c) * 2;
        o[0] = m;
        o[1] = l_sum;
    }
}

// grid (ceil((N - 1) / 256), B): score of the prefix positions; also fills the per-sequence budget / offsets
__global__ void __launch_bounds__(kEvThreads) last_token_scores_kernel(
    const float *__restrict__ logits, const float *__restrict__ stats_part, int B, int Hq, int N, int chunks, int n_keep,
    float *__restrict__ raw, int32_t *__restrict__ budgets, int64_t *__restrict__ offsets) {
    extern __shared__ float mprime[];   // [Hq]
    const int b = blockIdx.y, tid = threadIdx.x;
    for (int h = tid; h < Hq; h += kEvThreads) {
        const float *p = stats_part + ((size_t)b * Hq + h) * chunks * 2;
        float m = -1e30f;
        for (int c = 0; c < chunks; ++c) m = fmaxf(m, p[2 * c]);
        float l = 0.f;
        for (int c = 0; c < chunks; ++c) l += p[2 * c + 1] * exp2f(p[2 * c] - m);
        mprime[h] = m + log2f(l);
    }
    if (blockIdx.x == 0 && blockIdx.y == 0) {
        for (int i = tid; i < B; i += kEvThreads) budgets[i] = n_keep;
        for (int i = tid; i <= B; i += kEvThreads) offsets[i] = (int64_t)i * n_keep;
    }
    __syncthreads();
    const int j = blockIdx.x * kEvThreads + tid;
    if (j >= N - 1) return;
    float acc[4] = {0.f, 0.f, 0.f, 0.f};
    for (int h = 0; h < Hq; ++h) acc[h & 3] += ex2f(logits[((size_t)b * Hq + h) * N + j] - mprime[h]);
    raw[(size_t)b * (N - 1) + j] = (acc[0] + acc[1]) + (acc[2] + acc[3]);
}

// one warp per kept row: Xout[b, t, :] = X[b, idx[b, t], :]
__global__ void __launch_bounds__(256) gather_rows_kernel(const unsigned char *__restrict__ X,
                                                         const int32_t *__restrict__ idx, int64_t rows_total, int n_keep,
                                                         int N, int64_t row_bytes, unsigned char *__restrict__ out,
                                                         uint32_t *__restrict__ status) {
    const int lane = threadIdx.x & 31;
    const int64_t warp = ((int64_t)blockIdx.x * blockDim.x + threadIdx.x) >> 5;
    const int64_t nwarps = ((int64_t)gridDim.x * blockDim.x) >> 5;
    for (int64_t t = warp; t < rows_total; t += nwarps) {
        const int64_t b = t / n_keep;
        if (!UNCOMP_INDEX_OK(idx[t], N, status)) continue;
        const int4 *src = reinterpret_cast<const int4 *>(X + (b * N + idx[t]) * row_bytes);
        int4 *dst = reinterpret_cast<int4 *>(out + t * row_bytes);
        const int nvec = (int)(row_bytes >> 4);
        for (int v = lane; v < nvec; v += 32) dst[v] = src[v];
    }
}

template <typename T>
cudaError_t launch_logits(int G, dim3 grid, cudaStream_t st, const T *q, const T *K, int H, int64_t sB, int64_t sH,
                          int64_t sN, int N, int chunk, int chunks, float c_log2, float *logits, float *stats) {
    switch (G) {
        case 1: last_token_logits_kernel<T, 1><<<grid, kEvThreads, 0, st>>>(q, K, H, sB, sH, sN, N, chunk, chunks, c_log2, logits, stats); break;
        case 2: last_token_logits_kernel<T, 2><<<grid, kEvThreads, 0, st>>>(q, K, H, sB, sH, sN, N, chunk, chunks, c_log2, logits, stats); break;
        case 4: last_token_logits_kernel<T, 4><<<grid, kEvThreads, 0, st>>>(q, K, H, sB, sH, sN, N, chunk, chunks, c_log2, logits, stats); break;
        case 8: last_token_logits_kernel<T, 8><<<grid, kEvThreads, 0, st>>>(q, K, H, sB, sH, sN, N, chunk, chunks, c_log2, logits, stats); break;
        case 16: last_token_logits_kernel<T, 16><<<grid, kEvThreads, 0, st>>>(q, K, H, sB, sH, sN, N, chunk, chunks, c_log2, logits, stats); break;
        default: return cudaErrorInvalidValue;
    }
    return cudaGetLastError();
}
cudaError_t launch_logits_mma(int G, dim3 grid, cudaStream_t st, const __nv_bfloat16 *q, const __nv_bfloat16 *K, int H,
                              int64_t sB, int64_t sH, int64_t sN, int N, int chunk, int chunks, float c_log2,
                              float *logits, float *stats) {
    switch (G) {
        case 1: last_token_logits_mma_kernel<1><<<grid, kEvThreads, 0, st>>>(q, K, H, sB, sH, sN, N, chunk, chunks, c_log2, logits, stats); break;
        case 2: last_token_logits_mma_kernel<2><<<grid, kEvThreads, 0, st>>>(q, K, H, sB, sH, sN, N, chunk, chunks, c_log2, logits, stats); break;
        case 4: last_token_logits_mma_kernel<4><<<grid, kEvThreads, 0, st>>>(q, K, H, sB, sH, sN, N, chunk, chunks, c_log2, logits, stats); break;
        case 8: last_token_logits_mma_kernel<8><<<grid, kEvThreads, 0, st>>>(q, K, H, sB, sH, sN, N, chunk, chunks, c_log2, logits, stats); break;
        case 16: last_token_logits_mma_kernel<16><<<grid, kEvThreads, 0, st>>>(q, K, H, sB, sH, sN, N, chunk, chunks, c_log2, logits, stats); break;
        default: return cudaErrorInvalidValue;
    }
    return cudaGetLastError();
}
}  // namespace

constexpr int kEvChunk = 1024;   // tokens per CTA of the logits kernel
int evict_chunks(const uncomp_shape &s) { return (s.N + kEvChunk - 1) / kEvChunk; }

cudaError_t launch_evict_hidden(const Plan &p, const void *d_qlast, const void *d_K, int64_t sB, int64_t sH, int64_t sN,
                                const void *d_X, int64_t row_bytes, int n_keep, float scale, float *d_logits,
                                float *d_stats, float *d_raw, int32_t *d_budgets, int64_t *d_offsets, float *d_scores,
                                int32_t *d_indices, void *d_Xout, uint32_t *d_status, Profiler *prof, cudaStream_t st) {
    const uncomp_shape &s = p.shape;
    const int chunk = kEvChunk, chunks = evict_chunks(s);
    const float c_log2 = scale * 1.4426950408889634f;
    cudaError_t e;
    {
        ProfScope ps(prof, kSlotEvictLogits, st);
        dim3 grid(chunks, s.B * s.H);
        if (s.dtype == UNCOMP_FP32)
            e = launch_logits<float>(p.G, grid, st, (const float *)d_qlast, (const float *)d_K, s.H, sB, sH, sN, s.N, chunk,
                                     chunks, c_log2, d_logits, d_stats);
        else
            e = launch_logits_mma(p.G, grid, st, (const __nv_bfloat16 *)d_qlast, (const __nv_bfloat16 *)d_K, s.H, sB, sH,
                                  sN, s.N, chunk, chunks, c_log2, d_logits, d_stats);
        if (e != cudaSuccess) return e;
    }
    {
        ProfScope ps(prof, kSlotEvictScores, st);
        dim3 grid((s.N - 1 + kEvThreads - 1) / kEvThreads, s.B);
        last_token_scores_kernel<<<grid, kEvThreads, s.Hq * sizeof(float), st>>>(d_logits, d_stats, s.B, s.Hq, s.N, chunks,
                                                                                n_keep, d_raw, d_budgets, d_offsets);
    }
    {
        // the selection kernel with one unit per sequence, a window of one (the last position), no pooling
        ProfScope ps(prof, kSlotPoolSelect, st);
        Plan q = p;
        q.units = s.B;
        q.prefix = s.N - 1;
        q.shape.w = 1;
        e = launch_pool_select(q, d_raw, d_scores, 1, 0, d_budgets, d_offsets, d_indices, d_status, st);
        if (e != cudaSuccess) return e;
    }
    {
        ProfScope ps(prof, kSlotEvictGather, st);
        int dev = 0, sms = 148;
        cudaGetDevice(&dev);
        cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
        gather_rows_kernel<<<sms * 8, 256, 0, st>>>((const unsigned char *)d_X, d_indices, (int64_t)s.B * n_keep, n_keep,
                                                    s.N, row_bytes, (unsigned char *)d_Xout, d_status);
    }
    return cudaGetLastError();
}

}  // namespace uncomp
