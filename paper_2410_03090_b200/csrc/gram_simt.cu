// Per-unit Gram matrix G = X^T X and column sums s = X^T 1 on the CUDA cores.
//
// Used for fp32 keys, which need fp64 accumulation: with 1e-3 noise under a unit-scale low-rank signal
// the small eigenvalues of the covariance (Eq. 1 of the paper) sit near 2e-8 of the largest one, below
// what an fp32 Gram entry resolves.  bf16 keys take the tensor-core kernel in gram_tc.cu; this kernel
// also accepts them (fp32 accumulation) and is the known-good path the tensor-core kernel is tested
// against.
//
// Grid: (P token chunks, units).  A CTA of 256 threads streams its chunk in tiles of 32 tokens through
// shared memory; thread (ty, tx) owns the 8 x 8 outputs {ty + 16 i} x {tx + 16 j}.  Each chunk writes
// its own partial [d*d + d]; the eigen kernel adds the partials in a fixed order, so results do not
// depend on scheduling.
#include "common.cuh"

namespace uncomp {

template <typename T, typename Acc>
__global__ void __launch_bounds__(256) gram_simt_kernel(const T *__restrict__ K, UnitAddr addr, int N, int chunk,
                                                        Acc *__restrict__ partials, int P) {
    constexpr int TT = 32;
    __shared__ Acc tile[TT][kD];
    const int p = blockIdx.x, u = blockIdx.y;
    const int tid = threadIdx.x, tx = tid & 15, ty = tid >> 4;
    const T *X = K + addr.base(u);
    const int t0 = p * chunk;
    const int t1 = min(N, t0 + chunk);

    Acc acc[8][8];
#pragma unroll
    for (int i = 0; i < 8; ++i)
#pragma unroll
        for (int j = 0; j < 8; ++j) acc[i][j] = Acc(0);
    Acc colsum = Acc(0);  // threads 0..127 own one column each

    for (int t = t0; t < t1; t += TT) {
        const int nt = min(TT, t1 - t);
        for (int e = tid; e < TT * kD; e += 256) {
            const int r = e >> 7, c = e & 127;
            tile[r][c] = r < nt ? Acc(to_float(X[(int64_t)(t + r) * addr.sN + c])) : Acc(0);
        }
        __syncthreads();
        if (tid < kD) {
#pragma unroll 8
            for (int r = 0; r < TT; ++r) colsum += tile[r][tid];
        }
#pragma unroll 4
        for (int r = 0; r < TT; ++r) {
            Acc a[8], b[8];
#pragma unroll
            for (int i = 0; i < 8; ++i) { a[i] = tile[r][ty + 16 * i]; b[i] = tile[r][tx + 16 * i]; }
#pragma unroll
            for (int i = 0; i < 8; ++i)
#pragma unroll
                for (int j = 0; j < 8; ++j) acc[i][j] += a[i] * b[j];
        }
        __syncthreads();
    }
    Acc *out = partials + ((size_t)u * P + p) * (kD * kD + kD);
#pragma unroll
    for (int i = 0; i < 8; ++i)
#pragma unroll
        for (int j = 0; j < 8; ++j) out[(ty + 16 * i) * kD + tx + 16 * j] = acc[i][j];
    if (tid < kD) out[kD * kD + tid] = colsum;
}

cudaError_t launch_gram_simt(const Plan &p, const void *dK, const UnitAddr &addr, void *d_partials, cudaStream_t st) {
    dim3 grid(p.gram_splits, p.units);
    if (p.shape.dtype == UNCOMP_FP32) {
        gram_simt_kernel<float, double><<<grid, 256, 0, st>>>((const float *)dK, addr, p.shape.N, p.gram_chunk,
                                                             (double *)d_partials, p.gram_splits);
    } else {
        gram_simt_kernel<__nv_bfloat16, float><<<grid, 256, 0, st>>>((const __nv_bfloat16 *)dK, addr, p.shape.N,
                                                                    p.gram_chunk, (float *)d_partials,
                                                                    p.gram_splits);
    }
    return cudaGetLastError();
}

}  // namespace uncomp
