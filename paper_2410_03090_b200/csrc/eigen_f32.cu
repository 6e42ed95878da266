// Truncated matrix entropy for bf16 keys: the same four steps as eigen.cu, with the 128 x 128 covariance
// held entirely in REGISTERS in fp32 (paper Section 3.1 - 3.2).
//
// The Gram partials of bf16 keys carry fp32 accumulation error already, and the entropy is a smooth
// function of the spectrum: an fp32 Householder reduction moves H_k by about 1e-8, four orders below the
// 1e-4 tolerance, while fp32 keys (whose small eigenvalues sit at 2e-8 of the largest) keep the fp64
// kernel of eigen.cu.
//
// 256 threads per unit, two CTAs per SM.  Thread (ty, tx) owns the 64 entries A[ty + 16 a][tx + 16 b],
// a, b < 8, so the rank-2 update A -= v w^T + w v^T is pure register arithmetic and the matrix never
// touches shared memory.  Per Householder step: the owners publish row k, every half-warp recomputes its
// norm, the matrix-vector product is reduced over the 16 lanes of a row group with an 8-shuffle
// transpose-reduction, and two __syncthreads order the two small shared vectors.  The step loop is
// unrolled over a = k / 16, so rows and columns that are already reduced drop out of the unrolled code.
// C is scaled to unit trace first (entries <= 1: no overflow in fp32).
//
// Eigenvalues: the Sturm-count recurrence of eigen.cu in fp64 on the tridiagonal result.  One coarse
// round evaluates 256 equally spaced points (one per thread) for all eigenvalues at once, then teams of
// 8 lanes refine one eigenvalue each, 9-fold per round.
#include "common.cuh"

namespace uncomp {

namespace {
constexpr int kT = 256;
constexpr int n = kD;

struct E32Smem {
    double sd[n];      // column sums
    double dn[n];      // diagonal / scale
    double e2[n];      // (off-diagonal / scale)^2, e2[0] = 0
    double lam[n];
    double red[8];
    float dnf[n];      // fp32 copies for the fast Sturm count
    float e2f[n];
    float xs[n];
    float ps[n];
    float dd[n];
    float ee[n];
    int cnt[kT + 2];
    int flags[2];
};

// Number of eigenvalues of the normalised tridiagonal matrix that are < x: sign changes of the three-term
// recurrence p_i = (d_i - x) p_{i-1} - e_{i-1}^2 p_{i-2}.  Robust form: a zero takes the sign opposite to
// its predecessor and the pair is rescaled whenever it gets small.
__device__ __noinline__ int sturm_count_robust(const double *dn, const double *e2, double x) {
    const double tiny = 0x1p-400, big = 0x1p+400;
    double p0 = 0.0, p1 = 1.0;
    bool neg1 = false;
    int count = 0;
    for (int i = 0; i < n; ++i) {
        double pn = (dn[i] - x) * p1 - e2[i] * p0;
        bool negn = pn < 0.0;
        if (pn == 0.0) {
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

// Fast form of the same count in fp32 (the tridiagonal matrix comes from an fp32 reduction, so its entries
// carry no more than fp32 accuracy anyway): one dependent fused multiply-add per step, signs compared on
// the raw bit patterns, the magnitude checked (and an exact zero looked for) every 4 steps.  With
// |d_i - x| <= 2 and e^2 <= 1 the pair grows by at most 2^6 in 4 steps and one step shrinks it by at most
// 2^-24, so re-centring into [2^-20, 2^20] every 4 steps keeps it inside the fp32 range.  An exact zero is
// rare; the robust fp64 form then recounts.
__device__ __forceinline__ int sturm_count_n(const double *dn, const double *e2, const float *dnf, const float *e2f,
                                             float x) {
    float p0 = 1.f, p1 = dnf[0] - x;
    int count = __float_as_int(p1) < 0 ? 1 : 0;      // sign change against p_0 = 1
    bool zero = p1 == 0.f;
#pragma unroll 1
    for (int i0 = 1; i0 < n; i0 += 4) {
#pragma unroll
        for (int i = i0; i < i0 + 4; ++i) {
            if (i < n) {
                const float pn = fmaf(dnf[i] - x, p1, -(e2f[i] * p0));
                count += (unsigned)(__float_as_int(pn) ^ __float_as_int(p1)) >> 31;
                zero |= pn == 0.f;
                p0 = p1;
                p1 = pn;
            }
        }
        const float a = fabsf(p1);
        if (a < 0x1p-20f) { p1 *= 0x1p+40f; p0 *= 0x1p+40f; }
        else if (a > 0x1p+20f) { p1 *= 0x1p-40f; p0 *= 0x1p-40f; }
    }
    if (zero) return sturm_count_robust(dn, e2, (double)x);
    return count;
}

__device__ __forceinline__ float half_warp_sum(float v) {   // over the 16 lanes that share ty
#pragma unroll
    for (int o = 8; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    return v;
}

// Householder steps k = 16 KA .. 16 KA + 15 (stopping at n - 3): rows / columns with a, b < KA are done.
template <int KA>
__device__ __forceinline__ void householder_block(float (&A)[8][8], E32Smem &S, int tx, int ty, int tid) {
#pragma unroll 1
    for (int kt = 0; kt < 16; ++kt) {
        const int k = 16 * KA + kt;
        if (k > n - 3) break;
        if (ty == kt) {
#pragma unroll
            for (int b = KA; b < 8; ++b) S.xs[tx + 16 * b] = A[KA][b];
            if (tx == kt) S.dd[k] = A[KA][KA];
        }
        __syncthreads();
        const float x0 = S.xs[k + 1];
        float vc[8], vr[8];
        float rest = 0.f;
#pragma unroll
        for (int b = KA; b < 8; ++b) {
            const int c = tx + 16 * b;
            const float x = S.xs[c];
            vc[b] = c > k + 1 ? x : 0.f;
            rest = fmaf(vc[b], vc[b], rest);
        }
        rest = half_warp_sum(rest);
        if (rest == 0.f) {                       // nothing to annihilate; uniform over the CTA
            if (tid == 0) S.ee[k] = x0;
            __syncthreads();
            continue;
        }
        const float sig = fmaf(x0, x0, rest);
        const float alpha = x0 >= 0.f ? -sqrtf(sig) : sqrtf(sig);
        const float beta = 1.f / (sig - x0 * alpha);       // 2 / (v^T v)
        if (tid == 0) S.ee[k] = alpha;
#pragma unroll
        for (int b = KA; b < 8; ++b)
            if (tx + 16 * b == k + 1) vc[b] = x0 - alpha;
#pragma unroll
        for (int a = KA; a < 8; ++a) {
            const int r = ty + 16 * a;
            vr[a] = r > k + 1 ? S.xs[r] : (r == k + 1 ? x0 - alpha : 0.f);
        }
        // p = beta * A v : partial sums over this thread's columns, reduced over the 16 lanes of the row group
        float part[8];
#pragma unroll
        for (int a = 0; a < 8; ++a) {
            part[a] = 0.f;
            if (a >= KA) {
#pragma unroll
                for (int b = KA; b < 8; ++b) part[a] = fmaf(A[a][b], vc[b], part[a]);
            }
        }
        float k4[4], k2[2];
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            const float send = (tx & 8) ? part[i] : part[i + 4];
            const float mine = (tx & 8) ? part[i + 4] : part[i];
            k4[i] = mine + __shfl_xor_sync(0xffffffffu, send, 8);
        }
#pragma unroll
        for (int i = 0; i < 2; ++i) {
            const float send = (tx & 4) ? k4[i] : k4[i + 2];
            const float mine = (tx & 4) ? k4[i + 2] : k4[i];
            k2[i] = mine + __shfl_xor_sync(0xffffffffu, send, 4);
        }
        float k1;
        {
            const float send = (tx & 2) ? k2[0] : k2[1];
            const float mine = (tx & 2) ? k2[1] : k2[0];
            k1 = mine + __shfl_xor_sync(0xffffffffu, send, 2);
        }
        k1 += __shfl_xor_sync(0xffffffffu, k1, 1);
        if ((tx & 1) == 0) S.ps[ty + 16 * (tx >> 1)] = beta * k1;     // row index a = tx >> 1
        __syncthreads();
        // kk = beta/2 v^T p ; w = p - kk v ; A -= v w^T + w v^T on the rows and columns beyond k
        float pc[8], kk = 0.f;
#pragma unroll
        for (int b = KA; b < 8; ++b) {
            pc[b] = S.ps[tx + 16 * b];
            kk = fmaf(vc[b], pc[b], kk);
        }
        kk = 0.5f * beta * half_warp_sum(kk);
        float wc[8], wr[8];
#pragma unroll
        for (int b = KA; b < 8; ++b) wc[b] = (tx + 16 * b > k) ? fmaf(-kk, vc[b], pc[b]) : 0.f;
#pragma unroll
        for (int a = KA; a < 8; ++a) {
            const int r = ty + 16 * a;
            wr[a] = r > k ? fmaf(-kk, vr[a], S.ps[r]) : 0.f;
        }
#pragma unroll
        for (int a = KA; a < 8; ++a)
#pragma unroll
            for (int b = KA; b < 8; ++b) A[a][b] = fmaf(-wr[a], vc[b], fmaf(-vr[a], wc[b], A[a][b]));
    }
}
}  // namespace

__global__ void __launch_bounds__(kT, 2)
eigen_f32_kernel(const float *__restrict__ partials, int P, int N, int k_trunc, int center, int norm, int max_iters,
                 float *__restrict__ entropy, float *__restrict__ erank, double *__restrict__ spectrum,
                 uint32_t *__restrict__ status) {
    __shared__ E32Smem S;
    const int u = blockIdx.x, tid = threadIdx.x, lane = tid & 31, wid = tid >> 5;
    const int tx = tid & 15, ty = tid >> 4;
    constexpr int len = n * n + n;
    const float *base = partials + (size_t)u * P * len;

    // ---- 1. assemble C / trace(C) in registers --------------------------------------------------
    const double invN = 1.0 / (double)N;
    if (tid < n) {
        double s = 0.0;
        for (int p = 0; p < P; ++p) s += (double)base[(size_t)p * len + n * n + tid];
        S.sd[tid] = s;
        double g = 0.0;
        for (int p = 0; p < P; ++p) g += (double)base[(size_t)p * len + tid * (n + 1)];
        if (center) g -= s * s * invN;
        g = warp_sum(g);
        if (lane == 0) S.red[wid] = g;
    }
    if (tid == 0) S.flags[0] = 0;
    __syncthreads();
    const double trace = S.red[0] + S.red[1] + S.red[2] + S.red[3];
    const double inv_tr = trace > 0.0 ? 1.0 / trace : 0.0;
    // Coalesced 16-byte loads of the partials (many in flight), summed and centred in fp64, scaled to unit
    // trace and staged in shared memory; each thread then picks its 64 entries from there.
    extern __shared__ __align__(16) float stage[];        // [n * n]
    {
        const float4 *base4 = reinterpret_cast<const float4 *>(base);
        constexpr int len4 = len / 4;
#pragma unroll 4
        for (int i = 0; i < n * n / 4 / kT; ++i) {
            const int e4 = tid + kT * i;
            double g0 = 0.0, g1 = 0.0, g2 = 0.0, g3 = 0.0;
            for (int p = 0; p < P; ++p) {
                const float4 v = __ldg(base4 + (size_t)p * len4 + e4);
                g0 += (double)v.x; g1 += (double)v.y; g2 += (double)v.z; g3 += (double)v.w;
            }
            const int r = (4 * e4) >> 7, c0 = (4 * e4) & 127;
            if (center) {
                const double sr = S.sd[r] * invN;
                g0 -= sr * S.sd[c0]; g1 -= sr * S.sd[c0 + 1]; g2 -= sr * S.sd[c0 + 2]; g3 -= sr * S.sd[c0 + 3];
            }
            *reinterpret_cast<float4 *>(stage + 4 * e4) =
                make_float4((float)(g0 * inv_tr), (float)(g1 * inv_tr), (float)(g2 * inv_tr), (float)(g3 * inv_tr));
        }
    }
    __syncthreads();
    float A[8][8];
#pragma unroll
    for (int a = 0; a < 8; ++a)
#pragma unroll
        for (int b = 0; b < 8; ++b) A[a][b] = stage[(ty + 16 * a) * n + tx + 16 * b];

    // ---- 2. Householder tridiagonalisation in registers -----------------------------------------
    householder_block<0>(A, S, tx, ty, tid);
    householder_block<1>(A, S, tx, ty, tid);
    householder_block<2>(A, S, tx, ty, tid);
    householder_block<3>(A, S, tx, ty, tid);
    householder_block<4>(A, S, tx, ty, tid);
    householder_block<5>(A, S, tx, ty, tid);
    householder_block<6>(A, S, tx, ty, tid);
    householder_block<7>(A, S, tx, ty, tid);
    if (ty == 14 && tx == 14) S.dd[n - 2] = A[7][7];
    if (ty == 14 && tx == 15) S.ee[n - 2] = A[7][7];
    if (ty == 15 && tx == 15) { S.dd[n - 1] = A[7][7]; S.ee[n - 1] = 0.f; }
    __syncthreads();

    // ---- 3. the k largest eigenvalues ------------------------------------------------------------
    if (wid == 0) {
        double r = 0.0;   // Gershgorin radius as the scale
        for (int i = lane; i < n; i += 32) {
            const double left = i > 0 ? fabs((double)S.ee[i - 1]) : 0.0;
            const double right = i < n - 1 ? fabs((double)S.ee[i]) : 0.0;
            r = fmax(r, fabs((double)S.dd[i]) + left + right);
        }
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) r = fmax(r, __shfl_xor_sync(0xffffffffu, r, o));
        if (lane == 0) S.red[4] = r > 0.0 ? r : 1.0;
    }
    __syncthreads();
    const double scale = S.red[4], inv_scale = 1.0 / scale;
    if (tid < n) {
        S.dn[tid] = (double)S.dd[tid] * inv_scale;
        const double e = tid > 0 ? (double)S.ee[tid - 1] * inv_scale : 0.0;
        S.e2[tid] = e * e;
        S.dnf[tid] = (float)S.dn[tid];
        S.e2f[tid] = (float)(e * e);
    }
    __syncthreads();
    // coarse round: counts at 256 interior points of [lo0, hi0], shared by all eigenvalues
    const double lo0 = -1.0, hi0 = 1.0 + 0x1p-40, step0 = (hi0 - lo0) / (double)(kT + 1);
    S.cnt[tid + 1] = sturm_count_n(S.dn, S.e2, S.dnf, S.e2f, (float)(lo0 + step0 * (double)(tid + 1)));
    if (tid == 0) { S.cnt[0] = 0; S.cnt[kT + 1] = n; }
    __syncthreads();

    const int k = min(k_trunc, n);
    const int iters = max_iters > 0 ? max_iters : 10;
    const double tol = 2e-8;    // of the spectral radius; the fp32 reduction itself is good to about 1e-7
    const int sub = tid & 7;
    const unsigned team_mask = 0xffu << (lane & 24);
    for (int j0 = 0; j0 < k; j0 += kT / 8) {
        const int j = j0 + (tid >> 3);              // this team of 8 lanes looks for the j-th largest
        const bool active = j < k;
        const int idx = n - 1 - (active ? j : 0);   // its 0-based rank from below
        // bracket from the coarse counts: first grid point whose count exceeds idx
        int first = kT + 1;
        {
            int lo_i = 0, hi_i = kT + 1;            // cnt[lo_i] <= idx < cnt[hi_i]
            while (hi_i - lo_i > 1) {
                const int mid = (lo_i + hi_i) >> 1;
                if (S.cnt[mid] > idx) hi_i = mid; else lo_i = mid;
            }
            first = hi_i;
        }
        double lo = lo0 + step0 * (double)(first - 1), hi = lo0 + step0 * (double)first;
        for (int it = 0; it < iters; ++it) {
            const double width = hi - lo;
            const bool done = width <= tol;
            if (__all_sync(0xffffffffu, done)) break;
            int c = 0;
            if (!done) c = sturm_count_n(S.dn, S.e2, S.dnf, S.e2f, (float)(lo + width * (double)(sub + 1) * (1.0 / 9.0)));
            const unsigned above = __ballot_sync(0xffffffffu, c > idx) & team_mask;
            if (!done) {
                const int f = above ? (__ffs(above) - 1) - (lane & 24) : 8;
                const double new_hi = f < 8 ? lo + width * (double)(f + 1) * (1.0 / 9.0) : hi;
                const double new_lo = f > 0 ? lo + width * (double)f * (1.0 / 9.0) : lo;
                lo = new_lo;
                hi = new_hi;
            }
        }
        if (active && sub == 0) {
            S.lam[j] = 0.5 * (lo + hi) * scale;     // in units of trace(C)
            if (hi - lo > tol) atomicOr(&S.flags[0], 1);
        }
    }
    __syncthreads();

    // ---- 4. entropy -----------------------------------------------------------------------------
    if (wid == 0) {      // one warp: lane i takes eigenvalues i, i + 32, ...; fixed-order butterfly sums
        double total = 0.0;
        if (norm) total = trace > 0.0 ? 1.0 : 0.0;
        else {
            for (int i = lane; i < k; i += 32) total += S.lam[i] > 0.0 ? S.lam[i] : 0.0;
            total = warp_sum(total);
        }
        double h = 0.0;
        if (total > 0.0) {
            for (int i = lane; i < k; i += 32) {
                const double p = (S.lam[i] > 0.0 ? S.lam[i] : 0.0) / total;
                if (p > 0.0) h -= p * log(p);
            }
        }
        h = warp_sum(h);
        if (lane == 0) {
            entropy[u] = (float)h;
            if (erank) erank[u] = (float)exp(h);
            if (S.flags[0]) atomicOr(status, (uint32_t)UNCOMP_STATUS_NOT_CONVERGED);
        }
    }
    if (spectrum && tid < k) spectrum[(size_t)u * k + tid] = S.lam[tid] * trace;
}

cudaError_t launch_eigen_f32(const Plan &p, const void *d_partials, int partials_per_unit, const uncomp_entropy_params &ep,
                             float *d_entropy, float *d_erank, double *d_spectrum, uint32_t *d_status, cudaStream_t st) {
    const int smem = n * n * (int)sizeof(float);
    cudaError_t e = cudaFuncSetAttribute(eigen_f32_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
    if (e != cudaSuccess) return e;
    eigen_f32_kernel<<<p.units, kT, smem, st>>>((const float *)d_partials, partials_per_unit, p.shape.N, ep.k_trunc, ep.center,
                                             ep.norm, ep.max_iters, d_entropy, d_erank, d_spectrum, d_status);
    return cudaGetLastError();
}

}  // namespace uncomp
