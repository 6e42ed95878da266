// Truncated matrix entropy of WIDE token matrices X [N, D], D up to 4096: hidden states, or the heads of a
// layer side by side (paper Section 3.1 Eq. 1 with x_i in R^D, Lemma 2, Section 3.2; the appendix section on
// the truncated effective rank of hidden states).  The D x D scatter matrix does not fit an SM, so the stage
// is split differently from the per-head path:
//   1. column sums       s = X^T 1, fp64, token chunks summed in a fixed order;
//   2. Gram              G = X^T X on tcgen05: a CTA owns a 256 x 256 block pair (I <= J) of G and a token
//                        chunk; per 64-token stage TMA brings the 256 features of block I and of block J
//                        (64-feature boxes, 128B swizzle); both MMA operands are read MN-major, two
//                        M = 128, N = 256 accumulators fill the 512 TMEM columns; partial blocks to scratch;
//   3. assemble          C = G - s s^T / N (fp64 subtraction), stored as a full symmetric fp32 matrix;
//   4. tridiagonalise    Householder on the whole GPU: one cooperative launch, rows of the trailing matrix
//                        spread over all warps, ONE grid barrier per column.  The rank-2 update of column k
//                        is applied while the matrix is swept for the matrix-vector product of column k + 1,
//                        so the matrix (64 MB at D = 4096, resident in L2) is read and written once per column;
//   5. eigenvalues       Sturm-count 256-section (fp64), one CTA per wanted eigenvalue of the tridiagonal
//                        matrix, then H_k and erank_k.
// When the matrix has fewer tokens than features (N < D) the same non-zero eigenvalues are taken from the N x N
// matrix of the centred rows' inner products, (x_i - mean) . (x_j - mean) = G'_ij - g_i - g_j + mean . mean with
// G' = X X^T and g = X mean: the Gram kernel then contracts over features (both operands K-major, a CTA owns a
// 256 x 256 block pair of tokens and a chunk of 64-feature slices) and everything after it runs at size N.
// Every wait is bounded: the TMA / MMA barriers as in the other tensor-core kernels, the grid barrier by a
// poll limit after which the kernel raises UNCOMP_STATUS_TIMEOUT and all CTAs leave.
#include <math.h>

#include "tc_common.cuh"

namespace uncomp {

namespace {
// ------------------------------------------------------------------------------------------ 1. column sums
constexpr int kColChunks = 64;

// grid (D / 128 feature groups, token chunks), 8 warps: a lane owns 4 adjacent features (one 8-byte load per token
// row, a warp reads 256 contiguous bytes), warp w takes the tokens t0 + w, t0 + w + 8, ...; the 8 warps are added
// in warp order
__global__ void __launch_bounds__(256) wide_colsum_kernel(const __nv_bfloat16 *__restrict__ X, int64_t sN, int N, int D,
                                                         double *__restrict__ part) {
    __shared__ double red[8][128];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int f = blockIdx.x * 128 + lane * 4, c = blockIdx.y;
    const int per = (N + kColChunks - 1) / kColChunks;
    const int t0 = c * per, t1 = min(N, t0 + per);
    double acc[4] = {0.0, 0.0, 0.0, 0.0};
    if (f < D) {
        for (int t = t0 + warp; t < t1; t += 32) {
            uint2 x[4];
#pragma unroll
            for (int u = 0; u < 4; ++u)
                x[u] = t + 8 * u < t1 ? *reinterpret_cast<const uint2 *>(X + (int64_t)(t + 8 * u) * sN + f) : make_uint2(0u, 0u);
#pragma unroll
            for (int u = 0; u < 4; ++u) {
                acc[0] += (double)__uint_as_float(x[u].x << 16);
                acc[1] += (double)__uint_as_float(x[u].x & 0xffff0000u);
                acc[2] += (double)__uint_as_float(x[u].y << 16);
                acc[3] += (double)__uint_as_float(x[u].y & 0xffff0000u);
            }
        }
    }
#pragma unroll
    for (int i = 0; i < 4; ++i) red[warp][lane * 4 + i] = acc[i];
    __syncthreads();
    if (threadIdx.x < 128 && blockIdx.x * 128 + threadIdx.x < D) {
        double sum = 0.0;
#pragma unroll
        for (int wv = 0; wv < 8; ++wv) sum += red[wv][threadIdx.x];
        part[(size_t)c * D + blockIdx.x * 128 + threadIdx.x] = sum;
    }
}

__global__ void __launch_bounds__(256) wide_colsum_reduce_kernel(const double *__restrict__ part, int D,
                                                                double *__restrict__ s) {
    const int f = blockIdx.x * 256 + threadIdx.x;
    if (f >= D) return;
    double acc = 0.0;
    for (int c = 0; c < kColChunks; ++c) acc += part[(size_t)c * D + f];
    s[f] = acc;
}

// ------------------------------------------------------------------------------------------------ 2. Gram
constexpr int kWTok = 64;                        // tokens per stage
constexpr int kWRegion = 64 * 128;               // 8 KB: 64 tokens x 64 features (128 B rows)
constexpr int kWHalf = 4 * kWRegion;             // 32 KB: the 256 features of one block
constexpr int kWStage = 2 * kWHalf;              // 64 KB: block I then block J
constexpr int kWStages = 3;
constexpr int kWThreads = 192;
constexpr int kWBlock = 256;                     // features per block of G

struct WideTail {
    uint64_t full[kWStages];
    uint64_t empty[kWStages];
    uint64_t accum;
    uint32_t tmem_base;
    uint32_t abort;
};
constexpr int kWSmem = 1024 + kWStages * kWStage + (int)sizeof(WideTail);

// grid (block pairs, chunks of the contracted dimension).  DUAL = false: blocks of 256 features, contraction over
// tokens in stages of 64 (operands MN-major); DUAL = true: blocks of 256 tokens, contraction over features in slices
// of 64 (operands K-major: rows 128 B apart, 8-row groups 1024 B apart, 16 features further = 32 B).
// N here is the extent of the contracted dimension, chunk its share per CTA (a multiple of 64).
template <bool DUAL>
__global__ void __launch_bounds__(kWThreads, 1)
gram_wide_kernel(const __grid_constant__ CUtensorMap tmap, int N, int nblk, int chunk, float *__restrict__ partials,
                 uint32_t *__restrict__ status) {
    extern __shared__ unsigned char smem_raw[];
    const uint32_t raw_addr = tc::smem_u32(smem_raw);
    const uint32_t pad = (1024u - (raw_addr & 1023u)) & 1023u;
    unsigned char *smem = smem_raw + pad;
    const uint32_t tiles_addr = raw_addr + pad;
    WideTail &T = *reinterpret_cast<WideTail *>(smem + kWStages * kWStage);

    int I = 0, J = 0;
    {
        int rem = blockIdx.x;
        for (I = 0; I < nblk; ++I) {
            const int cnt = nblk - I;
            if (rem < cnt) { J = I + rem; break; }
            rem -= cnt;
        }
    }
    const bool diag = I == J;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int t0 = blockIdx.y * chunk, t1 = min(N, t0 + chunk);
    const int ntiles = (t1 - t0 + kWTok - 1) / kWTok;

    if (threadIdx.x == 0) {
        for (int s = 0; s < kWStages; ++s) {
            tc::mbar_init(tc::smem_u32(&T.full[s]), 1);
            tc::mbar_init(tc::smem_u32(&T.empty[s]), 1);
        }
        tc::mbar_init(tc::smem_u32(&T.accum), 1);
        T.abort = 0;
        tc::fence_mbar_init();
    }
    if (warp == 5) {
        tc::tmem_alloc(tc::smem_u32(&T.tmem_base), 512);
        tc::tmem_relinquish();
    }
    if (warp == 4 && lane == 0) tc::prefetch_tmap(&tmap);
    tc::tc_fence_before();
    __syncthreads();
    tc::tc_fence_after();
    const uint32_t tmem = T.tmem_base;

    if (warp == 4) {
        if (lane == 0) {
            int issued = 0;
            for (int i = 0; i < ntiles; ++i, ++issued) {
                const int s = i % kWStages;
                if (i >= kWStages && !tc::mbar_wait(tc::smem_u32(&T.empty[s]), ((i / kWStages) - 1) & 1, status)) {
                    T.abort = 1;
                    break;
                }
                const uint32_t bar = tc::smem_u32(&T.full[s]);
                const uint32_t dst = tiles_addr + s * kWStage;
                tc::mbar_expect_tx(bar, diag ? kWHalf : kWStage);
                if (DUAL) {      // one box of 64 features x 256 tokens per block
                    tc::tma_load_3d(dst, &tmap, bar, t0 + i * kWTok, I * kWBlock, 0);
                    if (!diag) tc::tma_load_3d(dst + kWHalf, &tmap, bar, t0 + i * kWTok, J * kWBlock, 0);
                } else {
#pragma unroll
                    for (int r = 0; r < 4; ++r)
                        tc::tma_load_3d(dst + r * kWRegion, &tmap, bar, I * kWBlock + r * 64, t0 + i * kWTok, 0);
                    if (!diag) {
#pragma unroll
                        for (int r = 0; r < 4; ++r)
                            tc::tma_load_3d(dst + kWHalf + r * kWRegion, &tmap, bar, J * kWBlock + r * 64, t0 + i * kWTok, 0);
                    }
                }
            }
            if (T.abort) {
                for (int i = max(0, issued - kWStages); i < issued; ++i)
                    tc::mbar_wait(tc::smem_u32(&T.full[i % kWStages]), (i / kWStages) & 1, status);
            }
        }
    } else if (warp == 5) {
        if (lane == 0) {
            constexpr uint32_t idesc = DUAL ? tc::idesc_bf16_f32(128, 256, 0, 0) : tc::idesc_bf16_f32(128, 256, 1, 1);
            // MN-major, 128-byte swizzle: 64-feature regions kWRegion apart (LBO), 8-token groups 1024 B apart
            // (SBO); 16 tokens further = 2048 B = +128 in the 16-byte address field.  K-major: 8-row groups 1024 B
            // apart, 16 features further = 32 B = +2; the second 128 rows of a block start 16 KB further.
            constexpr uint32_t kStep = DUAL ? 2u : 128u;
            constexpr uint32_t kSecondHalf = DUAL ? (uint32_t)((128 * 128) >> 4) : (uint32_t)((2 * kWRegion) >> 4);
            const uint64_t base_desc = tc::smem_desc_sw128(tiles_addr, DUAL ? 16 : kWRegion, 1024);
            const uint32_t dhi = tc::desc_hi(base_desc);
            bool ok = true;
            for (int i = 0; i < ntiles && ok; ++i) {
                const int s = i % kWStages;
                ok = tc::mbar_wait(tc::smem_u32(&T.full[s]), (i / kWStages) & 1, status);
                if (!ok) { T.abort = 1; break; }
                tc::tc_fence_after();
                const uint32_t lo = tc::desc_lo(base_desc) + (uint32_t)(s * (kWStage >> 4));
                const uint32_t b_lo = lo + (diag ? 0u : (uint32_t)(kWHalf >> 4));
#pragma unroll
                for (int k = 0; k < kWTok / 16; ++k) {
                    const uint32_t acc = (i > 0 || k > 0) ? 1u : 0u;
                    tc::mma_f16_ss_lohi(tmem, lo + k * kStep, b_lo + k * kStep, dhi, idesc, acc);
                    tc::mma_f16_ss_lohi(tmem + 256, lo + kSecondHalf + k * kStep, b_lo + k * kStep, dhi, idesc, acc);
                }
                tc::mma_commit(tc::smem_u32(&T.empty[s]));
            }
            tc::mma_commit(tc::smem_u32(&T.accum));
        }
    } else {
        const bool ok = tc::mbar_wait(tc::smem_u32(&T.accum), 0, status);
        tc::tc_fence_after();
        if (ok && !T.abort) {
            const int m = warp * 32 + lane;
            uint32_t r[32];
#pragma unroll 1
            for (int mi = 0; mi < 2; ++mi) {
                float *out = partials + (((size_t)blockIdx.y * gridDim.x + blockIdx.x) * 2 + mi) * (128 * kWBlock) +
                             (size_t)m * kWBlock;
#pragma unroll 1
                for (int c0 = 0; c0 < kWBlock; c0 += 32) {
                    tc::tmem_ld32(tmem + ((uint32_t)(warp * 32) << 16) + mi * 256 + c0, r);
                    tc::tmem_ld_wait();
                    float4 *dst = reinterpret_cast<float4 *>(out + c0);
#pragma unroll
                    for (int q = 0; q < 8; ++q)
                        dst[q] = make_float4(__uint_as_float(r[4 * q]), __uint_as_float(r[4 * q + 1]),
                                             __uint_as_float(r[4 * q + 2]), __uint_as_float(r[4 * q + 3]));
                }
            }
        }
    }
    tc::tc_fence_before();
    __syncthreads();
    if (warp == 5) tc::tmem_dealloc(tmem, 512);
}

// -------------------------------------------------------------------------------------------- 3. assemble
// grid (block pairs, 256 rows of the pair's block), thread = column.  Only the upper triangle of a diagonal
// block is taken from the MMA result and mirrored, so C is symmetric bit for bit.
__global__ void __launch_bounds__(256) wide_assemble_kernel(const float *__restrict__ partials, int pairs, int chunks,
                                                           int nblk, int D, int N, int center,
                                                           const double *__restrict__ s, float *__restrict__ C) {
    int I = 0, J = 0;
    {
        int rem = blockIdx.x;
        for (I = 0; I < nblk; ++I) {
            const int cnt = nblk - I;
            if (rem < cnt) { J = I + rem; break; }
            rem -= cnt;
        }
    }
    const int r = blockIdx.y, c = threadIdx.x;
    const int gi = I * kWBlock + r, gj = J * kWBlock + c;
    if (gi >= D || gj >= D || (I == J && r > c)) return;
    const int mi = r >> 7, m = r & 127;
    double acc = 0.0;
    for (int ch = 0; ch < chunks; ++ch)
        acc += (double)partials[(((size_t)ch * pairs + blockIdx.x) * 2 + mi) * (128 * kWBlock) + (size_t)m * kWBlock + c];
    if (center) acc -= s[gi] * s[gj] / (double)N;
    const float v = (float)acc;
    C[(size_t)gi * D + gj] = v;
    C[(size_t)gj * D + gi] = v;
}

// Token-space variant: C'_ij = G'_ij - g_i - g_j + mm for i, j < N (g = X mean, mm = mean . mean, stored at g[Dt]);
// rows and columns N .. Dt - 1 only pad the matrix to a multiple of 64 and are zero.
__global__ void __launch_bounds__(256) wide_assemble_dual_kernel(const float *__restrict__ partials, int pairs, int chunks,
                                                                int nblk, int Dt, int N, int center,
                                                                const double *__restrict__ g, float *__restrict__ C) {
    int I = 0, J = 0;
    {
        int rem = blockIdx.x;
        for (I = 0; I < nblk; ++I) {
            const int cnt = nblk - I;
            if (rem < cnt) { J = I + rem; break; }
            rem -= cnt;
        }
    }
    const int r = blockIdx.y, c = threadIdx.x;
    const int gi = I * kWBlock + r, gj = J * kWBlock + c;
    if (gi >= Dt || gj >= Dt || (I == J && r > c)) return;
    const int mi = r >> 7, m = r & 127;
    double acc = 0.0;
    if (gi < N && gj < N) {
        for (int ch = 0; ch < chunks; ++ch)
            acc += (double)partials[(((size_t)ch * pairs + blockIdx.x) * 2 + mi) * (128 * kWBlock) + (size_t)m * kWBlock + c];
        if (center) acc += g[Dt] - g[gi] - g[gj];
    }
    const float v = (float)acc;
    C[(size_t)gi * Dt + gj] = v;
    C[(size_t)gj * Dt + gi] = v;
}

// g_i = x_i . mean (a warp per token, fp64) and mean . mean at g[Dt]
__global__ void __launch_bounds__(256) wide_rowdot_kernel(const __nv_bfloat16 *__restrict__ X, int64_t sN, int N, int D, int Dt,
                                                         const double *__restrict__ s, double *__restrict__ g) {
    const int lane = threadIdx.x & 31, row = blockIdx.x * 8 + (threadIdx.x >> 5);
    if (row > N) return;                                  // warp N computes mean . mean
    double acc = 0.0;
    for (int f = lane; f < D; f += 32) {
        const double m = s[f] / (double)N;
        acc += (row < N ? (double)__bfloat162float(X[(int64_t)row * sN + f]) : m) * m;
    }
    acc = warp_sum(acc);
    if (lane == 0) g[row < N ? row : Dt] = acc;
}

// ------------------------------------------------------------------------------------- 4. tridiagonalisation
constexpr int kTriThreads = 1024;
constexpr int kTriWarps = kTriThreads / 32;
constexpr unsigned kBarrierSpin = 1u << 22;

// Three block-wide sums at once; every thread gets the totals.  Warp 0 adds the per-warp sums (a butterfly: a fixed
// order) and publishes them.  `red` must not be the array of the previous call: the calls alternate between two
// arrays, which saves the barrier that would otherwise protect the array's reuse.
__device__ __forceinline__ void tri_block_sum3(float &x, float &y, float &z, float (*red)[kTriWarps + 1]) {
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    x = warp_sum(x);
    y = warp_sum(y);
    z = warp_sum(z);
    if (lane == 0) { red[0][warp] = x; red[1][warp] = y; red[2][warp] = z; }
    __syncthreads();
    if (warp == 0) {
        float tx = warp_sum(red[0][lane]), ty = warp_sum(red[1][lane]), tz = warp_sum(red[2][lane]);
        if (lane == 0) { red[0][kTriWarps] = tx; red[1][kTriWarps] = ty; red[2][kTriWarps] = tz; }
    }
    __syncthreads();
    x = red[0][kTriWarps];
    y = red[1][kTriWarps];
    z = red[2][kTriWarps];
}

// All CTAs of a cooperative launch meet here.  `bar` counts arrivals monotonically.
__device__ __forceinline__ bool tri_grid_barrier(unsigned *bar, unsigned &phase, uint32_t *status, int *flag) {
    __syncthreads();
    if (threadIdx.x == 0) {
        __threadfence();
        atomicAdd(bar, 1u);
        const unsigned target = (phase + 1u) * gridDim.x;
        bool ok = false;
        for (unsigned it = 0; it < kBarrierSpin; ++it) {
            unsigned cur;
            asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(cur) : "l"(bar) : "memory");
            if (cur >= target) { ok = true; break; }
        }
        if (!ok) atomicOr(status, (uint32_t)UNCOMP_STATUS_TIMEOUT);
        *flag = ok ? 1 : 0;
    }
    __syncthreads();
    ++phase;
    return *flag != 0;
}

// A: full symmetric fp32 matrix [D, D], destroyed.  Output: diagonal a[D] and off-diagonal e[D - 1].
// State at the top of iteration k: rows >= k of A hold the matrix after the reflections of columns 0 .. k - 2;
// the rank-2 update of column k - 1, A -= 2 (v w^T + w v^T) on rows and columns >= k, is still pending: its
// vector v is in shared memory (vn), the product p = A v it needs is in global memory (written by the last sweep).
// Every CTA repeats the O(D) vector work of a column (a thread owns up to four columns in registers), so one
// column costs one grid barrier, two block-wide sums and one sweep over the trailing matrix.
constexpr int kTriQ = 4;   // columns per thread: D <= kTriQ * kTriThreads

__global__ void __launch_bounds__(kTriThreads, 1) tridiag_wide_kernel(float *__restrict__ A, int D, double *__restrict__ a_out,
                                                                     double *__restrict__ e_out, float *__restrict__ pbuf,
                                                                     unsigned *bar, uint32_t *__restrict__ status) {
    extern __shared__ float sm[];
    float *v = sm, *w = sm + D, *vn = sm + 2 * D;
    __shared__ float redA[3][kTriWarps + 1], redB[3][kTriWarps + 1];
    __shared__ int flag;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    // rows go round-robin over the CTAs first, so that a short trailing matrix still keeps every SM busy
    const int total_warps = gridDim.x * kTriWarps, gw = warp * gridDim.x + blockIdx.x;
    for (int i = tid; i < D; i += kTriThreads) { v[i] = 0.f; w[i] = 0.f; vn[i] = 0.f; }
    __syncthreads();
    unsigned phase = 0;
    for (int k = 0; k + 2 < D; ++k) {
        // ---- vector work: finish the pending update (w = p - (v . p) v), apply it to row k, next reflection ----
        const float *pprev = pbuf + (size_t)((k + 1) & 1) * D;
        float pj[kTriQ], rj[kTriQ];
#pragma unroll
        for (int q = 0; q < kTriQ; ++q) {
            const int j = tid + q * kTriThreads;
            const bool own = j < D && j >= k;
            pj[q] = (own && k > 0) ? __ldcg(pprev + j) : 0.f;
            rj[q] = own ? __ldcg(A + (size_t)k * D + j) : 0.f;
        }
        float Kdot = 0.f, pk = 0.f, unused = 0.f;
#pragma unroll
        for (int q = 0; q < kTriQ; ++q) {
            const int j = tid + q * kTriThreads;
            if (j < D && j >= k) {
                Kdot = fmaf(vn[j], pj[q], Kdot);
                if (j == k) pk = pj[q];
            }
        }
        tri_block_sum3(Kdot, pk, unused, redA);
        const float vk = vn[k], wk = pk - Kdot * vk;
        float sigma = 0.f, akk = 0.f, x0 = 0.f;
#pragma unroll
        for (int q = 0; q < kTriQ; ++q) {
            const int j = tid + q * kTriThreads;
            if (j < D && j >= k) {
                const float vj = vn[j], wj = pj[q] - Kdot * vj;
                v[j] = vj;
                w[j] = wj;
                const float r = rj[q] - 2.f * (vk * wj + wk * vj);
                rj[q] = r;
                if (j > k) sigma = fmaf(r, r, sigma);
                if (j == k) akk = r;
                if (j == k + 1) x0 = r;
            }
        }
        tri_block_sum3(sigma, akk, x0, redB);     // every thread has read vn[k] before this barrier
        float alpha = 0.f, inv = 0.f;
        if (sigma > 0.f) {
            alpha = -copysignf(sqrtf(sigma), x0);
            inv = 1.f / sqrtf(2.f * (sigma - alpha * x0));     // 1 / |x - alpha e_1|
        }
        // the sweep starts at a multiple of four columns: up to three dead columns left of k + 1 ride along
        // (nobody reads them again) and must not enter the dot product, hence the zeros
#pragma unroll
        for (int q = 0; q < kTriQ; ++q) {
            const int j = tid + q * kTriThreads;
            if (j < D && j + 3 >= k) vn[j] = j > k ? (rj[q] - (j == k + 1 ? alpha : 0.f)) * inv : 0.f;
        }
        if (blockIdx.x == 0 && tid == 0) { a_out[k] = (double)akk; e_out[k] = (double)alpha; }
        __syncthreads();
        // ---- sweep: apply the pending update to rows >= k + 1 and form p = A' vn on the fly, 16 bytes per lane ----
        float *pw = pbuf + (size_t)(k & 1) * D;
        const int j0 = (k + 1) & ~3;
        for (int i = k + 1 + gw; i < D; i += total_warps) {
            const float vi = -2.f * v[i], wi = -2.f * w[i];
            float *row = A + (size_t)i * D;
            float acc = 0.f;
            for (int jb = j0 + 4 * lane; jb < D; jb += 512) {      // batches of four loads in flight per lane
                float4 x[4];
#pragma unroll
                for (int u = 0; u < 4; ++u)
                    x[u] = jb + u * 128 < D ? __ldcg(reinterpret_cast<const float4 *>(row + jb + u * 128))
                                            : make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
                for (int u = 0; u < 4; ++u) {
                    const int j = jb + u * 128;
                    if (j < D) {
                        const float4 v4 = *reinterpret_cast<const float4 *>(v + j), w4 = *reinterpret_cast<const float4 *>(w + j);
                        const float4 n4 = *reinterpret_cast<const float4 *>(vn + j);
                        float4 y = x[u];
                        y.x = fmaf(vi, w4.x, fmaf(wi, v4.x, y.x));
                        y.y = fmaf(vi, w4.y, fmaf(wi, v4.y, y.y));
                        y.z = fmaf(vi, w4.z, fmaf(wi, v4.z, y.z));
                        y.w = fmaf(vi, w4.w, fmaf(wi, v4.w, y.w));
                        __stcg(reinterpret_cast<float4 *>(row + j), y);
                        acc = fmaf(y.x, n4.x, fmaf(y.y, n4.y, fmaf(y.z, n4.z, fmaf(y.w, n4.w, acc))));
                    }
                }
            }
            acc = warp_sum(acc);
            if (lane == 0) __stcg(pw + i, acc);
        }
        if (!tri_grid_barrier(bar, phase, status, &flag)) return;
    }
    // the last 2 x 2 block: its pending update comes from column D - 3
    if (blockIdx.x == 0 && tid == 0) {
        const int i = D - 2, j = D - 1;
        const float *pprev = pbuf + (size_t)((D - 3) & 1) * D;
        const float pi = __ldcg(pprev + i), pjv = __ldcg(pprev + j);
        const float Kdot = vn[i] * pi + vn[j] * pjv;
        const float wi = pi - Kdot * vn[i], wj = pjv - Kdot * vn[j];
        a_out[i] = (double)(__ldcg(A + (size_t)i * D + i) - 4.f * vn[i] * wi);
        e_out[i] = (double)(__ldcg(A + (size_t)i * D + j) - 2.f * (vn[i] * wj + wi * vn[j]));
        a_out[j] = (double)(__ldcg(A + (size_t)j * D + j) - 4.f * vn[j] * wj);
    }
}

// Measurement aid: the memory pattern of the sweep above on its own, so that the tridiagonalisation can be held
// against a bandwidth measured on the same GPU.  A matrix of rows x cols floats that fits in L2 is read and written
// once per pass, a warp per row, four 16-byte loads in flight per lane, one fused multiply-add per element.
__global__ void __launch_bounds__(kTriThreads, 1) l2_sweep_kernel(float *__restrict__ A, int rows, int cols, int passes) {
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int total_warps = gridDim.x * kTriWarps, gw = warp * gridDim.x + blockIdx.x;
    for (int p = 0; p < passes; ++p) {
        for (int i = gw; i < rows; i += total_warps) {
            float *row = A + (size_t)i * cols;
            for (int jb = 4 * lane; jb < cols; jb += 512) {
                float4 x[4];
#pragma unroll
                for (int u = 0; u < 4; ++u)
                    x[u] = jb + u * 128 < cols ? __ldcg(reinterpret_cast<const float4 *>(row + jb + u * 128))
                                               : make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
                for (int u = 0; u < 4; ++u) {
                    if (jb + u * 128 < cols) {
                        float4 y = x[u];
                        y.x = fmaf(y.x, 0.999f, 1e-6f); y.y = fmaf(y.y, 0.999f, 1e-6f);
                        y.z = fmaf(y.z, 0.999f, 1e-6f); y.w = fmaf(y.w, 0.999f, 1e-6f);
                        __stcg(reinterpret_cast<float4 *>(row + jb + u * 128), y);
                    }
                }
            }
        }
    }
}

// --------------------------------------------------------------------------------- 5. eigenvalues, entropy
constexpr int kSturmThreads = 256;
constexpr int kSturmMaxK = 256;

// number of eigenvalues of the tridiagonal matrix (a, e) below x
__device__ int sturm_count_wide(const double *__restrict__ a, const double *__restrict__ e, int D, double x, double tiny) {
    double q = a[0] - x;
    if (fabs(q) < tiny) q = -tiny;
    int cnt = q < 0.0;
    for (int i = 1; i < D; ++i) {
        const double ei = e[i - 1];
        q = (a[i] - x) - ei * ei / q;
        if (fabs(q) < tiny) q = -tiny;
        cnt += q < 0.0;
    }
    return cnt;
}

// grid (k): CTA t finds the t-th largest eigenvalue by 256-section (every CTA repeats the cheap set-up);
// lam_out[t] and, from CTA 0, the trace in lam_out[k]
__global__ void __launch_bounds__(kSturmThreads) sturm_wide_kernel(const double *__restrict__ a, const double *__restrict__ e,
                                                                  int D, int k, int max_iters, double *__restrict__ lam_out,
                                                                  uint32_t *__restrict__ status) {
    __shared__ double redlo[kSturmThreads / 32], redhi[kSturmThreads / 32], redtr[kSturmThreads / 32];
    __shared__ int redc[kSturmThreads / 32];
    __shared__ double bounds[3];
    __shared__ int nb_s;
    const int tid = threadIdx.x, lane = tid & 31, wid = tid >> 5, t = blockIdx.x;
    // Gershgorin interval and trace
    double lo = 1e300, hi = -1e300, tr = 0.0;
    for (int i = tid; i < D; i += kSturmThreads) {
        const double r = (i > 0 ? fabs(e[i - 1]) : 0.0) + (i + 1 < D ? fabs(e[i]) : 0.0);
        lo = fmin(lo, a[i] - r);
        hi = fmax(hi, a[i] + r);
        tr += a[i];
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        lo = fmin(lo, __shfl_xor_sync(0xffffffffu, lo, o));
        hi = fmax(hi, __shfl_xor_sync(0xffffffffu, hi, o));
        tr += __shfl_xor_sync(0xffffffffu, tr, o);
    }
    if (lane == 0) { redlo[wid] = lo; redhi[wid] = hi; redtr[wid] = tr; }
    __syncthreads();
    if (tid == 0) {
        double l = redlo[0], h = redhi[0], sum = 0.0;
        for (int i = 0; i < kSturmThreads / 32; ++i) { l = fmin(l, redlo[i]); h = fmax(h, redhi[i]); sum += redtr[i]; }
        const double span = fmax(h - l, 1e-300);
        bounds[0] = l - 1e-9 * span;
        bounds[1] = h + 1e-9 * span;
        bounds[2] = sum;
    }
    __syncthreads();
    double xl = bounds[0], xh = bounds[1];
    const double radius = fmax(fabs(xl), fabs(xh));
    const double tiny = fmax(radius, 1e-280) * 1e-19;      // floor of a pivot of the Sturm recurrence
    const double tol = radius * 1e-13;
    const int m = D - 1 - t;                               // ascending index of the wanted eigenvalue
    // invariant: count(xl) <= m < count(xh).  Each round cuts the bracket into 257 parts.
    const int rounds = max_iters > 0 ? max_iters : 8;
    int it = 0;
    for (; it < rounds && (xh - xl) > tol; ++it) {
        const double step = (xh - xl) / (double)(kSturmThreads + 1);
        const int c = sturm_count_wide(a, e, D, xl + step * (double)(tid + 1), tiny);
        // the points whose count is still <= m form a prefix
        int below = __popc(__ballot_sync(0xffffffffu, c <= m));
        if (lane == 0) redc[wid] = below;
        __syncthreads();
        if (tid == 0) {
            int nb = 0;
            for (int i = 0; i < kSturmThreads / 32; ++i) nb += redc[i];
            nb_s = nb;
        }
        __syncthreads();
        const int nb = nb_s;
        const double nl = xl + step * (double)nb, nh = nb < kSturmThreads ? xl + step * (double)(nb + 1) : xh;
        xl = nl;
        xh = nh;
    }
    if (tid == 0) {
        lam_out[t] = 0.5 * (xl + xh);
        if ((xh - xl) > tol) atomicOr(status, (uint32_t)UNCOMP_STATUS_NOT_CONVERGED);
        if (t == 0) lam_out[k] = bounds[2];
    }
}

// H_k and erank_k from the kf largest eigenvalues (descending; eigenvalues kf .. k - 1 are zero) and the trace at
// lam[kf]
__global__ void wide_entropy_kernel(const double *__restrict__ lam, int k, int kf, int norm, float *__restrict__ H_out,
                                    float *__restrict__ erank_out, double *__restrict__ spectrum) {
    if (threadIdx.x != 0) return;
    double denom = 0.0;
    if (norm == 0) {
        for (int i = 0; i < kf; ++i) denom += fmax(lam[i], 0.0);
    } else {
        denom = lam[kf];
    }
    double h = 0.0;
    for (int i = 0; i < kf; ++i) {
        const double pi = denom > 0.0 ? fmax(lam[i], 0.0) / denom : 0.0;
        if (pi > 0.0) h -= pi * log(pi);
    }
    *H_out = (float)h;
    if (erank_out) *erank_out = (float)exp(h);
    if (spectrum)
        for (int i = 0; i < k; ++i) spectrum[i] = i < kf ? lam[i] : 0.0;
}

size_t align256(size_t x) { return (x + 255) & ~(size_t)255; }

struct WideLayout {
    bool dual;          // token-space path (N < D)
    int Dt;             // size of the symmetric matrix that is tridiagonalised
    int nblk, pairs, chunk, chunks;
    size_t off_bar, off_s, off_colpart, off_a, off_e, off_lam, off_g, off_p, off_C, off_part, bytes;
};

WideLayout wide_layout(int N, int D) {
    WideLayout w;
    w.dual = N < D;
    w.Dt = w.dual ? (N + 63) / 64 * 64 : D;
    if (w.Dt < 128) w.Dt = 128;
    const int contract = w.dual ? D : N;                     // extent of the contracted dimension
    w.nblk = (w.Dt + kWBlock - 1) / kWBlock;
    w.pairs = w.nblk * (w.nblk + 1) / 2;
    int chunks = (2 * 148 + w.pairs - 1) / w.pairs;          // about two CTAs' worth of work per SM
    const int max_chunks = (contract + 511) / 512;
    if (chunks > max_chunks) chunks = max_chunks;
    if (chunks < 1) chunks = 1;
    w.chunk = (((contract + chunks - 1) / chunks) + kWTok - 1) / kWTok * kWTok;
    w.chunks = (contract + w.chunk - 1) / w.chunk;
    size_t o = 0;
    w.off_bar = o;      o = align256(o + 256);
    w.off_s = o;        o = align256(o + (size_t)D * sizeof(double));
    w.off_colpart = o;  o = align256(o + (size_t)kColChunks * D * sizeof(double));
    w.off_a = o;        o = align256(o + (size_t)w.Dt * sizeof(double));
    w.off_e = o;        o = align256(o + (size_t)w.Dt * sizeof(double));
    w.off_lam = o;      o = align256(o + (size_t)(kSturmMaxK + 1) * sizeof(double));
    w.off_g = o;        o = align256(o + (size_t)(w.Dt + 1) * sizeof(double));
    w.off_p = o;        o = align256(o + (size_t)2 * w.Dt * sizeof(float));
    w.off_C = o;        o = align256(o + (size_t)w.Dt * w.Dt * sizeof(float));
    w.off_part = o;     o = align256(o + (size_t)w.chunks * w.pairs * 2 * 128 * kWBlock * sizeof(float));
    w.bytes = o;
    return w;
}
}  // namespace

cudaError_t launch_l2_sweep(float *d_A, int rows, int cols, int passes, cudaStream_t st) {
    int dev = 0, sms = 0;
    cudaError_t err = cudaGetDevice(&dev);
    if (err != cudaSuccess) return err;
    err = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
    if (err != cudaSuccess) return err;
    l2_sweep_kernel<<<sms, kTriThreads, 0, st>>>(d_A, rows, cols, passes);
    return cudaGetLastError();
}

size_t entropy_wide_scratch_bytes(int N, int D) { return wide_layout(N, D).bytes; }

cudaError_t launch_entropy_wide(const void *d_X, int64_t sN, int N, int D, const uncomp_entropy_params &ep,
                                unsigned char *scratch, float *d_entropy, float *d_erank, double *d_spectrum,
                                uint32_t *d_status, Profiler *prof, cudaStream_t st) {
    const WideLayout w = wide_layout(N, D);
    const __nv_bfloat16 *X = (const __nv_bfloat16 *)d_X;
    double *s = (double *)(scratch + w.off_s), *colpart = (double *)(scratch + w.off_colpart);
    double *a = (double *)(scratch + w.off_a), *e = (double *)(scratch + w.off_e);
    float *pbuf = (float *)(scratch + w.off_p), *C = (float *)(scratch + w.off_C), *part = (float *)(scratch + w.off_part);
    double *g = (double *)(scratch + w.off_g);
    unsigned *bar = (unsigned *)(scratch + w.off_bar);
    cudaError_t err = cudaMemsetAsync(bar, 0, 256, st);
    if (err != cudaSuccess) return err;
    {
        ProfScope ps(prof, kSlotWideGram, st);
        wide_colsum_kernel<<<dim3((D + 127) / 128, kColChunks), 256, 0, st>>>(X, sN, N, D, colpart);
        wide_colsum_reduce_kernel<<<(D + 255) / 256, 256, 0, st>>>(colpart, D, s);
        CUtensorMap tmap;
        uint64_t dims[3] = {(uint64_t)D, (uint64_t)N, 1};
        uint64_t str[2] = {(uint64_t)sN * 2, (uint64_t)sN * 2 * (uint64_t)N};
        uint32_t box[3] = {64, w.dual ? (uint32_t)kWBlock : (uint32_t)kWTok, 1};
        err = encode_tensor_map(&tmap, d_X, 3, dims, str, box, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, CU_TENSOR_MAP_SWIZZLE_128B);
        if (err != cudaSuccess) return err;
        if (w.dual) {
            err = cudaFuncSetAttribute(gram_wide_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, kWSmem);
            if (err != cudaSuccess) return err;
            gram_wide_kernel<true><<<dim3(w.pairs, w.chunks), kWThreads, kWSmem, st>>>(tmap, D, w.nblk, w.chunk, part, d_status);
            wide_rowdot_kernel<<<(N + 1 + 7) / 8, 256, 0, st>>>(X, sN, N, D, w.Dt, s, g);
        } else {
            err = cudaFuncSetAttribute(gram_wide_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, kWSmem);
            if (err != cudaSuccess) return err;
            gram_wide_kernel<false><<<dim3(w.pairs, w.chunks), kWThreads, kWSmem, st>>>(tmap, N, w.nblk, w.chunk, part, d_status);
        }
    }
    {
        ProfScope ps(prof, kSlotWideAssemble, st);
        if (w.dual)
            wide_assemble_dual_kernel<<<dim3(w.pairs, kWBlock), 256, 0, st>>>(part, w.pairs, w.chunks, w.nblk, w.Dt, N, ep.center, g, C);
        else
            wide_assemble_kernel<<<dim3(w.pairs, kWBlock), 256, 0, st>>>(part, w.pairs, w.chunks, w.nblk, D, N, ep.center, s, C);
    }
    err = cudaGetLastError();
    if (err != cudaSuccess) return err;
    {
        ProfScope ps(prof, kSlotWideTridiag, st);
        int dev = 0, sms = 0, per_sm = 0;
        cudaGetDevice(&dev);
        cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
        const int Dt = w.Dt;
        const size_t smem = (size_t)3 * Dt * sizeof(float);
        err = cudaFuncSetAttribute(tridiag_wide_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
        if (err != cudaSuccess) return err;
        err = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, tridiag_wide_kernel, kTriThreads, smem);
        if (err != cudaSuccess) return err;
        if (per_sm < 1) return cudaErrorLaunchOutOfResources;
        int grid = sms;                                          // one CTA per SM: all of them are resident
        if (grid > Dt / 8) grid = Dt / 8;                         // small matrices: fewer CTAs, cheaper barrier
        int Di = Dt;
        void *args[] = {(void *)&C, (void *)&Di, (void *)&a, (void *)&e, (void *)&pbuf, (void *)&bar, (void *)&d_status};
        err = cudaLaunchCooperativeKernel((const void *)tridiag_wide_kernel, dim3(grid), dim3(kTriThreads), args, smem, st);
        if (err != cudaSuccess) return err;
    }
    {
        ProfScope ps(prof, kSlotWideSturm, st);
        const int k = ep.k_trunc < D ? ep.k_trunc : D;            // entries of the outputs
        const int kf = k < w.Dt ? k : w.Dt;                       // eigenvalues the matrix can have; the rest are zero
        double *lam = (double *)(scratch + w.off_lam);
        err = cudaMemsetAsync(lam, 0, (size_t)(kSturmMaxK + 1) * sizeof(double), st);
        if (err != cudaSuccess) return err;
        sturm_wide_kernel<<<kf, kSturmThreads, 0, st>>>(a, e, w.Dt, kf, ep.max_iters, lam, d_status);
        wide_entropy_kernel<<<1, 32, 0, st>>>(lam, k, kf, ep.norm, d_entropy, d_erank, d_spectrum);
    }
    return cudaGetLastError();
}

}  // namespace uncomp
