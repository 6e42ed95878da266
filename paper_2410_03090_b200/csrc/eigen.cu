// Truncated matrix entropy of every unit from its partial Gram matrices (paper Section 3.1 - 3.2).
//
// One CTA of 512 threads per unit, everything in fp64 and in shared memory:
//   1. C = sum_p G_p - s s^T / N with s = sum_p s_p (partials added in index order; the centring term is
//      dropped for the uncentred variant).  Eq. 1 without its 1/(N-1), which cancels in step 4.
//   2. Householder reduction of the 128 x 128 symmetric C to tridiagonal form (both triangles are kept
//      up to date, so every access runs along a row and is free of bank conflicts).
//   3. The k largest eigenvalues by Sturm-count multi-section: 16 lanes per eigenvalue evaluate the
//      division-free three-term recurrence of the characteristic polynomials at 16 interior points, so
//      the bracket shrinks 17-fold per round.  The recurrence is rescaled against underflow.
//   4. p_i = lambda_i / sum (over the k kept, or the whole trace), H_k = -sum p_i ln p_i, erank_k = exp H_k.
#include "common.cuh"

namespace uncomp {

constexpr int kEigThreads = 512;
constexpr int kEigWarps = kEigThreads / 32;

struct EigenSmem {
    double A[kD * kD];
    double v[kD];
    double pv[kD];
    double dd[kD];
    double ee[kD];    // ee[i] couples i and i+1
    double e2[kD];    // e2[i] = (ee[i-1] / scale)^2, e2[0] = 0
    double lam[kD];
    double scal[8];   // 0: beta, 2: skip flag, 3: scale, 4: trace
    int flags[4];
};

// number of eigenvalues of the normalised tridiagonal matrix that are < x
__device__ __forceinline__ int sturm_count(const double *dd, const double *e2, double inv_scale, double x) {
    const double tiny = 0x1p-400, big = 0x1p+400;
    double p0 = 0.0, p1 = 1.0;
    bool neg1 = false;
    int count = 0;
#pragma unroll 4
    for (int i = 0; i < kD; ++i) {
        double pn = (dd[i] * inv_scale - x) * p1 - e2[i] * p0;
        bool negn = pn < 0.0;
        if (pn == 0.0) {            // a zero takes the sign opposite to its predecessor
            negn = !neg1;
            pn = (negn ? -1.0 : 1.0) * fabs(p1) * 0x1p-100;
        }
        count += (negn != neg1);
        p0 = p1;
        p1 = pn;
        neg1 = negn;
        if (fabs(p1) < tiny) { p1 *= big; p0 *= big; }
    }
    return count;
}

template <typename PartialT>
__global__ void __launch_bounds__(kEigThreads, 1)
eigen_entropy_kernel(const PartialT *__restrict__ partials, int P, int N, int k_trunc, int center, int norm,
                     int max_iters, float *__restrict__ entropy, float *__restrict__ erank,
                     double *__restrict__ spectrum, uint32_t *__restrict__ status) {
    extern __shared__ __align__(16) unsigned char smem_raw[];
    EigenSmem &S = *reinterpret_cast<EigenSmem *>(smem_raw);
    const int u = blockIdx.x, tid = threadIdx.x, lane = tid & 31, wid = tid >> 5;
    constexpr int n = kD;
    const PartialT *base = partials + (size_t)u * P * (n * n + n);

    // ---- 1. assemble C ---------------------------------------------------------------------------
    if (tid < n) {
        double s = 0.0;
        for (int p = 0; p < P; ++p) s += (double)base[(size_t)p * (n * n + n) + n * n + tid];
        S.v[tid] = s;
    }
    __syncthreads();
    const double invN = 1.0 / (double)N;
    for (int e = tid; e < n * n; e += kEigThreads) {
        double g = 0.0;
        for (int p = 0; p < P; ++p) g += (double)base[(size_t)p * (n * n + n) + e];
        if (center) g -= S.v[e >> 7] * S.v[e & 127] * invN;
        S.A[e] = g;
    }
    __syncthreads();
    // symmetrise (the two triangles may come from different accumulation orders) and take the trace
    for (int e = tid; e < n * n; e += kEigThreads) {
        const int i = e >> 7, j = e & 127;
        if (i < j) {
            const double m = 0.5 * (S.A[i * n + j] + S.A[j * n + i]);
            S.A[i * n + j] = m;
            S.A[j * n + i] = m;
        }
    }
    __syncthreads();
    if (wid == 0) {
        double t = 0.0;
        for (int i = lane; i < n; i += 32) t += S.A[i * n + i];
        t = warp_sum(t);
        if (lane == 0) S.scal[4] = t;
    }

    // ---- 2. Householder tridiagonalisation -------------------------------------------------------
    for (int k = 0; k < n - 2; ++k) {
        const int m = n - k - 1;            // order of the trailing block
        double *Ak = S.A + (size_t)k * n + (k + 1);   // row k right of the diagonal == column k below it
        if (wid == 0) {
            double rest = 0.0;   // sum of squares below the sub-diagonal entry, free of cancellation
            for (int i = lane; i < m; i += 32) {
                const double x = Ak[i];
                if (i > 0) rest += x * x;
                S.v[i] = x;
            }
            rest = warp_sum(rest);
            if (lane == 0) {
                const double x0 = Ak[0];
                const double sig = rest + x0 * x0;
                S.dd[k] = S.A[(size_t)k * n + k];
                if (rest == 0.0) {                   // nothing to annihilate
                    S.ee[k] = x0;
                    S.scal[2] = 1.0;
                } else {
                    const double alpha = x0 >= 0.0 ? -sqrt(sig) : sqrt(sig);
                    S.ee[k] = alpha;
                    S.v[0] = x0 - alpha;
                    S.scal[0] = 1.0 / (sig - x0 * alpha);   // beta = 2 / (v^T v)
                    S.scal[2] = 0.0;
                }
            }
        }
        __syncthreads();
        if (S.scal[2] != 0.0) { __syncthreads(); continue; }
        const double beta = S.scal[0];
        double *A2 = S.A + (size_t)(k + 1) * n + (k + 1);
        // pv = beta * A2 v
        for (int i = wid; i < m; i += kEigWarps) {
            const double *row = A2 + (size_t)i * n;
            double acc = 0.0;
            for (int j = lane; j < m; j += 32) acc += row[j] * S.v[j];
            acc = warp_sum(acc);
            if (lane == 0) S.pv[i] = beta * acc;
        }
        __syncthreads();
        // kk = beta/2 * v^T pv (every warp computes it); w = pv - kk v; A2 -= v w^T + w v^T
        double kk = 0.0;
        for (int j = lane; j < m; j += 32) kk += S.v[j] * S.pv[j];
        kk = 0.5 * beta * warp_sum(kk);
        double vj[4], wj[4];
#pragma unroll
        for (int c = 0; c < 4; ++c) {
            const int j = lane + 32 * c;
            vj[c] = j < m ? S.v[j] : 0.0;
            wj[c] = j < m ? S.pv[j] - kk * vj[c] : 0.0;
        }
        for (int i = wid; i < m; i += kEigWarps) {
            const double vi = S.v[i];
            const double wi = S.pv[i] - kk * vi;
            double *row = A2 + (size_t)i * n;
#pragma unroll
            for (int c = 0; c < 4; ++c) {
                const int j = lane + 32 * c;
                if (j < m) row[j] -= vi * wj[c] + wi * vj[c];
            }
        }
        __syncthreads();
    }
    if (tid == 0) {
        S.dd[n - 2] = S.A[(size_t)(n - 2) * n + (n - 2)];
        S.ee[n - 2] = S.A[(size_t)(n - 2) * n + (n - 1)];
        S.dd[n - 1] = S.A[(size_t)(n - 1) * n + (n - 1)];
        S.ee[n - 1] = 0.0;
    }
    __syncthreads();

    // ---- 3. k largest eigenvalues by multi-section ----------------------------------------------
    if (wid == 0) {
        double r = 0.0;   // Gershgorin radius as the scale
        for (int i = lane; i < n; i += 32) {
            const double left = i > 0 ? fabs(S.ee[i - 1]) : 0.0;
            const double right = i < n - 1 ? fabs(S.ee[i]) : 0.0;
            r = fmax(r, fabs(S.dd[i]) + left + right);
        }
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) r = fmax(r, __shfl_xor_sync(0xffffffffu, r, o));
        if (lane == 0) S.scal[3] = r > 0.0 ? r : 1.0;
    }
    __syncthreads();
    const double scale = S.scal[3], inv_scale = 1.0 / scale;
    if (tid < n) {
        const double e = tid > 0 ? S.ee[tid - 1] * inv_scale : 0.0;
        S.e2[tid] = e * e;
    }
    if (tid == 0) S.flags[0] = 0;
    __syncthreads();

    const int k = min(k_trunc, n);
    const int iters = max_iters > 0 ? max_iters : 14;
    const double tol = 1e-13;
    const int sub = tid & 15;              // lane within the 16-lane team
    const unsigned team_mask = 0xffffu << (lane & 16);
    for (int j0 = 0; j0 < k; j0 += kEigThreads / 16) {
        const int j = j0 + (tid >> 4);      // this team looks for the j-th largest eigenvalue
        const bool active = j < k;
        const int idx = n - 1 - (active ? j : 0);   // its 0-based rank from below
        double lo = -1.0, hi = 1.0 + 0x1p-40;      // invariant: count(lo) <= idx < count(hi)
        for (int it = 0; it < iters; ++it) {
            const double width = hi - lo;
            const bool done = width <= tol;
            if (__all_sync(0xffffffffu, done)) break;     // warp-uniform exit
            int c = 0;
            if (!done) c = sturm_count(S.dd, S.e2, inv_scale, lo + width * (double)(sub + 1) * (1.0 / 17.0));
            const unsigned above = __ballot_sync(0xffffffffu, c > idx) & team_mask;   // interior points above lambda
            if (!done) {
                const int first = above ? (__ffs(above) - 1) - (lane & 16) : 16;
                const double new_hi = first < 16 ? lo + width * (double)(first + 1) * (1.0 / 17.0) : hi;
                const double new_lo = first > 0 ? lo + width * (double)first * (1.0 / 17.0) : lo;
                lo = new_lo;
                hi = new_hi;
            }
        }
        if (active && sub == 0) {
            S.lam[j] = 0.5 * (lo + hi) * scale;
            if (hi - lo > tol) atomicOr(&S.flags[0], 1);
        }
    }
    __syncthreads();

    // ---- 4. entropy -----------------------------------------------------------------------------
    if (tid == 0) {
        double total = 0.0;
        if (norm) total = S.scal[4];
        else for (int i = 0; i < k; ++i) total += S.lam[i] > 0.0 ? S.lam[i] : 0.0;
        double h = 0.0;
        if (total > 0.0) {
            for (int i = 0; i < k; ++i) {
                const double p = (S.lam[i] > 0.0 ? S.lam[i] : 0.0) / total;
                if (p > 0.0) h -= p * log(p);
            }
        }
        entropy[u] = (float)h;
        if (erank) erank[u] = (float)exp(h);
        if (S.flags[0]) atomicOr(status, UNCOMP_STATUS_NOT_CONVERGED);
    }
    if (spectrum && tid < k) spectrum[(size_t)u * k + tid] = S.lam[tid];
}

// Sum of the chunk partials of every unit in chunk order: out[u] = [G (d*d) | s (d)] in fp64.
template <typename PartialT>
__global__ void gram_reduce_kernel(const PartialT *__restrict__ partials, int P, double *__restrict__ out) {
    constexpr int len = kD * kD + kD;
    const int u = blockIdx.y;
    const int e = blockIdx.x * blockDim.x + threadIdx.x;
    if (e >= len) return;
    double g = 0.0;
    for (int p = 0; p < P; ++p) g += (double)partials[((size_t)u * P + p) * len + e];
    out[(size_t)u * len + e] = g;
}

cudaError_t launch_gram_reduce(const Plan &p, const void *d_partials, double *d_out, cudaStream_t st) {
    dim3 grid((kD * kD + kD + 255) / 256, p.units);
    if (p.shape.dtype == UNCOMP_FP32)
        gram_reduce_kernel<double><<<grid, 256, 0, st>>>((const double *)d_partials, p.gram_splits, d_out);
    else
        gram_reduce_kernel<float><<<grid, 256, 0, st>>>((const float *)d_partials, p.gram_splits, d_out);
    return cudaGetLastError();
}

cudaError_t launch_eigen_entropy(const Plan &p, const void *d_partials, const uncomp_entropy_params &ep,
                                 float *d_entropy, float *d_erank, double *d_spectrum, uint32_t *d_status,
                                 cudaStream_t st) {
    const size_t smem = sizeof(EigenSmem);
    cudaError_t e;
    if (p.shape.dtype == UNCOMP_FP32) {
        e = cudaFuncSetAttribute(eigen_entropy_kernel<double>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
        if (e != cudaSuccess) return e;
        eigen_entropy_kernel<double><<<p.units, kEigThreads, smem, st>>>(
            (const double *)d_partials, p.gram_splits, p.shape.N, ep.k_trunc, ep.center, ep.norm, ep.max_iters,
            d_entropy, d_erank, d_spectrum, d_status);
    } else {
        e = cudaFuncSetAttribute(eigen_entropy_kernel<float>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
        if (e != cudaSuccess) return e;
        eigen_entropy_kernel<float><<<p.units, kEigThreads, smem, st>>>(
            (const float *)d_partials, p.gram_splits, p.shape.N, ep.k_trunc, ep.center, ep.norm, ep.max_iters,
            d_entropy, d_erank, d_spectrum, d_status);
    }
    return cudaGetLastError();
}

}  // namespace uncomp
