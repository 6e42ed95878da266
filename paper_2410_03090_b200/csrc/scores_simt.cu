// Observation-window scores on the CUDA cores (paper Section 3.3.3, "Dynamic KV Cache Eviction").
//
// This is the plain two-pass form, used for fp32 inputs and as the known-good path the tensor-core
// scorer is tested against:
//   pass A  row statistics: for every window row r (query head g, window position i) the maximum m_r and
//           the sum l_r = sum_j exp(s_rj - m_r) of its causally visible logits, per token chunk;
//   merge   chunk statistics combined in chunk order into (m_r, 1 / l_r);
//   pass B  raw[j] = sum_r exp(s_rj - m_r) / l_r for the prefix positions j < N - w.
// Every reduction has a fixed order, so repeated runs give identical bits.
#include "common.cuh"

namespace uncomp {

constexpr int kSB = 64;   // rows and tokens per block of logits
constexpr int kKPad = kD + 1;

template <typename T>
__device__ __forceinline__ void load_rows(float (*dst)[kKPad], const T *src, int64_t row_stride, int first, int limit,
                                          int tid) {
    for (int e = tid; e < kSB * kD; e += 256) {
        const int r = e >> 7, c = e & 127;
        const int row = first + r;
        dst[r][c] = row < limit ? to_float(src[(int64_t)row * row_stride + c]) : 0.f;
    }
}

// logits of a 64 x 64 block: thread (ty, tx) gets rows ty + 16 i, tokens tx + 16 j
__device__ __forceinline__ void block_logits(const float (*q)[kKPad], const float (*k)[kKPad], int tx, int ty,
                                             float s[4][4]) {
#pragma unroll
    for (int i = 0; i < 4; ++i)
#pragma unroll
        for (int j = 0; j < 4; ++j) s[i][j] = 0.f;
#pragma unroll 8
    for (int a = 0; a < kD; ++a) {
        float qa[4], ka[4];
#pragma unroll
        for (int i = 0; i < 4; ++i) { qa[i] = q[ty + 16 * i][a]; ka[i] = k[tx + 16 * i][a]; }
#pragma unroll
        for (int i = 0; i < 4; ++i)
#pragma unroll
            for (int j = 0; j < 4; ++j) s[i][j] = fmaf(qa[i], ka[j], s[i][j]);
    }
}

// grid (score_splits, row blocks, units)
template <typename T>
__global__ void __launch_bounds__(256) score_stats_simt_kernel(const T *__restrict__ Qw, const T *__restrict__ K,
                                                              UnitAddr addr, int N, int w, int G, int chunk,
                                                              int splits, float scale,
                                                              float *__restrict__ stats_part) {
    extern __shared__ __align__(16) unsigned char smem_raw[];
    float(*qs)[kKPad] = reinterpret_cast<float(*)[kKPad]>(smem_raw);
    float(*ks)[kKPad] = qs + kSB;
    const int c = blockIdx.x, rb = blockIdx.y, u = blockIdx.z;
    const int tid = threadIdx.x, tx = tid & 15, ty = tid >> 4;
    const int rows = G * w, P = N - w;
    const T *Qu = Qw + (size_t)u * rows * kD;   // [G, w, d] of this unit: its G query heads are adjacent
    const T *Ku = K + addr.base(u);
    load_rows(qs, Qu, kD, rb * kSB, rows, tid);

    float m_run[4], l_run[4];
#pragma unroll
    for (int i = 0; i < 4; ++i) { m_run[i] = -INFINITY; l_run[i] = 0.f; }
    const int t0 = c * chunk, t1 = min(N, t0 + chunk);
    for (int t = t0; t < t1; t += kSB) {
        __syncthreads();
        load_rows(ks, Ku, addr.sN, t, t1, tid);
        __syncthreads();
        float s[4][4];
        block_logits(qs, ks, tx, ty, s);
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            const int r = rb * kSB + ty + 16 * i;
            const int last = P + (r % w);           // last visible position of this row
            float mx = -INFINITY;
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                const int pos = t + tx + 16 * j;
                s[i][j] = (pos < t1 && pos <= last) ? s[i][j] * scale : -INFINITY;
                mx = fmaxf(mx, s[i][j]);
            }
#pragma unroll
            for (int o = 8; o > 0; o >>= 1) mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, o));
            const float m_new = fmaxf(m_run[i], mx);
            float sum = 0.f;
            if (m_new > -INFINITY) {
#pragma unroll
                for (int j = 0; j < 4; ++j) sum += expf(s[i][j] - m_new);
            }
#pragma unroll
            for (int o = 8; o > 0; o >>= 1) sum += __shfl_xor_sync(0xffffffffu, sum, o);
            const float corr = m_run[i] > -INFINITY ? expf(m_run[i] - m_new) : 0.f;
            l_run[i] = l_run[i] * corr + sum;
            m_run[i] = m_new;
        }
    }
    if (tx == 0) {
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            const int r = rb * kSB + ty + 16 * i;
            if (r < rows) {
                float *o = stats_part + (((size_t)u * splits + c) * kMaxRows + r) * 2;
                o[0] = m_run[i];
                o[1] = l_run[i];
            }
        }
    }
}

// one thread per (unit, row): combine the chunk statistics in chunk order -> (m, 1/l)
__global__ void score_stats_merge_kernel(const float *__restrict__ stats_part, int units, int rows, int splits,
                                         float *__restrict__ stats) {
    const int idx = blockIdx.x * blockDim.x + threadIdx.x;
    if (idx >= units * rows) return;
    const int u = idx / rows, r = idx % rows;
    float m = -INFINITY;
    for (int c = 0; c < splits; ++c) m = fmaxf(m, stats_part[(((size_t)u * splits + c) * kMaxRows + r) * 2]);
    float l = 0.f;
    for (int c = 0; c < splits; ++c) {
        const float *p = stats_part + (((size_t)u * splits + c) * kMaxRows + r) * 2;
        if (p[0] > -INFINITY) l += p[1] * expf(p[0] - m);
    }
    stats[((size_t)u * kMaxRows + r) * 2] = m;
    stats[((size_t)u * kMaxRows + r) * 2 + 1] = 1.f / l;
}

// grid (prefix tiles of 64 tokens, units)
template <typename T>
__global__ void __launch_bounds__(256) score_colsum_simt_kernel(const T *__restrict__ Qw, const T *__restrict__ K,
                                                               UnitAddr addr, int N, int w, int G, float scale,
                                                               const float *__restrict__ stats,
                                                               float *__restrict__ raw) {
    extern __shared__ __align__(16) unsigned char smem_raw[];
    float(*qs)[kKPad] = reinterpret_cast<float(*)[kKPad]>(smem_raw);
    float(*ks)[kKPad] = qs + kSB;
    float(*red)[kSB] = reinterpret_cast<float(*)[kSB]>(ks + kSB);   // [16][64]
    const int tile = blockIdx.x, u = blockIdx.y;
    const int tid = threadIdx.x, tx = tid & 15, ty = tid >> 4;
    const int rows = G * w, P = N - w;
    const T *Qu = Qw + (size_t)u * rows * kD;
    const T *Ku = K + addr.base(u);
    const int t = tile * kSB;
    load_rows(ks, Ku, addr.sN, t, P, tid);
    float col[4] = {0.f, 0.f, 0.f, 0.f};
    for (int rb = 0; rb * kSB < rows; ++rb) {
        __syncthreads();
        load_rows(qs, Qu, kD, rb * kSB, rows, tid);
        __syncthreads();
        float s[4][4];
        block_logits(qs, ks, tx, ty, s);
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            const int r = rb * kSB + ty + 16 * i;
            if (r < rows) {
                const float m = stats[((size_t)u * kMaxRows + r) * 2];
                const float inv_l = stats[((size_t)u * kMaxRows + r) * 2 + 1];
#pragma unroll
                for (int j = 0; j < 4; ++j) col[j] += expf(s[i][j] * scale - m) * inv_l;
            }
        }
    }
#pragma unroll
    for (int j = 0; j < 4; ++j) red[ty][tx + 16 * j] = col[j];
    __syncthreads();
    if (tid < kSB && t + tid < P) {
        float acc = 0.f;
#pragma unroll
        for (int y = 0; y < 16; ++y) acc += red[y][tid];
        raw[(size_t)u * P + t + tid] = acc;
    }
}

// one thread per (unit, row): the caller's natural-log sum of exponentials in place of pass A and the merge
__global__ void lse_import_kernel(const float *__restrict__ lse, int units, int rows, int log2_domain,
                                  float *__restrict__ stats, uint32_t *__restrict__ status) {
    const int idx = blockIdx.x * blockDim.x + threadIdx.x;
    if (idx >= units * rows) return;
    const int u = idx / rows, r = idx % rows;
    float v = lse[idx];
    if (!isfinite(v)) {
        atomicOr(status, (uint32_t)UNCOMP_STATUS_NONFINITE);
        v = INFINITY;                        // exp(s - inf) = 0: the row drops out of every column sum
    }
    if (log2_domain) {
        stats[(size_t)u * kMaxRows + r] = v * 1.4426950408889634f;
    } else {
        stats[((size_t)u * kMaxRows + r) * 2] = v;
        stats[((size_t)u * kMaxRows + r) * 2 + 1] = 1.f;
    }
}

cudaError_t launch_lse_import(const Plan &p, const float *d_lse, float *d_stats, bool log2_domain, uint32_t *d_status,
                              cudaStream_t st) {
    const int total = p.units * p.rows;
    lse_import_kernel<<<(total + 255) / 256, 256, 0, st>>>(d_lse, p.units, p.rows, log2_domain ? 1 : 0, d_stats,
                                                           d_status);
    return cudaGetLastError();
}

template <typename T>
static cudaError_t launch_scores_simt_t(const Plan &p, const T *dQw, const T *dK, const UnitAddr &addr, float scale,
                                        const float *d_lse, float *d_stats_part, float *d_stats, float *d_raw,
                                        uint32_t *d_status, Profiler *prof, cudaStream_t st) {
    const size_t smemA = 2 * kSB * kKPad * sizeof(float);
    const size_t smemB = smemA + 16 * kSB * sizeof(float);
    cudaError_t e = cudaFuncSetAttribute(score_stats_simt_kernel<T>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                         (int)smemA);
    if (e != cudaSuccess) return e;
    e = cudaFuncSetAttribute(score_colsum_simt_kernel<T>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smemB);
    if (e != cudaSuccess) return e;
    if (d_lse) {
        ProfScope ps(prof, kSlotStatsMerge, st);
        e = launch_lse_import(p, d_lse, d_stats, false, d_status, st);
        if (e != cudaSuccess) return e;
    } else {
        const int row_blocks = (p.rows + kSB - 1) / kSB;
        dim3 gA(p.score_splits, row_blocks, p.units);
        {
            ProfScope ps(prof, kSlotScoreStats, st);
            score_stats_simt_kernel<T><<<gA, 256, smemA, st>>>(dQw, dK, addr, p.shape.N, p.shape.w, p.G, p.score_chunk,
                                                               p.score_splits, scale, d_stats_part);
        }
        const int total = p.units * p.rows;
        ProfScope ps(prof, kSlotStatsMerge, st);
        score_stats_merge_kernel<<<(total + 255) / 256, 256, 0, st>>>(d_stats_part, p.units, p.rows, p.score_splits,
                                                                      d_stats);
    }
    dim3 gB((p.prefix + kSB - 1) / kSB, p.units);
    {
        ProfScope ps(prof, kSlotScoreColsum, st);
        score_colsum_simt_kernel<T><<<gB, 256, smemB, st>>>(dQw, dK, addr, p.shape.N, p.shape.w, p.G, scale, d_stats,
                                                            d_raw);
    }
    return cudaGetLastError();
}

cudaError_t launch_scores_simt(const Plan &p, const void *dQw, const void *dK, const UnitAddr &addr, float scale,
                               const float *d_lse, float *d_stats_part, float *d_stats, float *d_raw,
                               uint32_t *d_status, Profiler *prof, cudaStream_t st) {
    if (p.shape.dtype == UNCOMP_FP32)
        return launch_scores_simt_t<float>(p, (const float *)dQw, (const float *)dK, addr, scale, d_lse, d_stats_part,
                                           d_stats, d_raw, d_status, prof, st);
    return launch_scores_simt_t<__nv_bfloat16>(p, (const __nv_bfloat16 *)dQw, (const __nv_bfloat16 *)dK, addr, scale,
                                               d_lse, d_stats_part, d_stats, d_raw, d_status, prof, st);
}

}  // namespace uncomp
