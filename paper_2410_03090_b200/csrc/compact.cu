// Gather of the kept K / V rows into the ragged per-head cache (paper Section 3.3.3: every head keeps
// its own context window; keys and values share one selection).
//
// HBM-bound copy.  A row of d = 128 elements is 256 B (bf16) or 512 B (fp32) and is moved as 16-byte
// vectors: 16 (32) consecutive lanes read one source row and write one destination row, so every
// request is a full, aligned 256-byte (512-byte) segment.  A warp takes 32 consecutive output rows per
// step: lane l finds the unit of row t0 + l by binary search over the offsets and fetches its source
// index, then the warp walks the 32 rows with the addresses broadcast by shuffles.  The grid is a
// multiple of the SM count and strides over the output.
#include "common.cuh"

namespace uncomp {

template <int ROW_BYTES>
__global__ void __launch_bounds__(256) compact_kernel(const unsigned char *__restrict__ K,
                                                      const unsigned char *__restrict__ V, UnitAddr aK, UnitAddr aV,
                                                      int units, int N, int elem_bytes,
                                                      const int32_t *__restrict__ indices,
                                                      const int64_t *__restrict__ offsets,
                                                      unsigned char *__restrict__ Kc,
                                                      unsigned char *__restrict__ Vc,
                                                      uint32_t *__restrict__ status) {
    constexpr int LANES_PER_ROW = ROW_BYTES / 16;          // 16 or 32
    constexpr int ROWS_PER_STEP = 32 / LANES_PER_ROW;      // 2 or 1
    const int lane = threadIdx.x & 31;
    const int64_t warp = ((int64_t)blockIdx.x * blockDim.x + threadIdx.x) >> 5;
    const int64_t nwarps = ((int64_t)gridDim.x * blockDim.x) >> 5;
    const int64_t total = offsets[units];
    const int sub = lane / LANES_PER_ROW, vec = lane % LANES_PER_ROW;
    for (int64_t t0 = warp * 32; t0 < total; t0 += nwarps * 32) {
        const int64_t t = t0 + lane;
        int64_t srcK = 0, srcV = 0;
        if (t < total) {
            int lo = 0, hi = units - 1;       // largest u with offsets[u] <= t
            while (lo < hi) {
                const int mid = (lo + hi + 1) >> 1;
                if (offsets[mid] <= t) lo = mid; else hi = mid - 1;
            }
            if (!UNCOMP_INDEX_OK(lo, units, status)) lo = 0;
            int64_t idx = indices[t];
            if (idx < 0 || idx >= N) {        // never form an address outside the unit's rows
                atomicOr(status, (uint32_t)UNCOMP_STATUS_BOUNDS);
                idx = idx < 0 ? 0 : N - 1;
            }
            srcK = (aK.base(lo) + idx * aK.sN) * elem_bytes;
            srcV = (aV.base(lo) + idx * aV.sN) * elem_bytes;
        }
        const int nrows = (int)min((int64_t)32, total - t0);
#pragma unroll 4
        for (int r = 0; r < 32; r += ROWS_PER_STEP) {
            const int row = r + sub;
            const int64_t sk = __shfl_sync(0xffffffffu, srcK, row);
            const int64_t sv = __shfl_sync(0xffffffffu, srcV, row);
            if (row < nrows && UNCOMP_INDEX_OK(t0 + row, total, status)) {
                const int4 a = *reinterpret_cast<const int4 *>(K + sk + vec * 16);
                const int4 b = *reinterpret_cast<const int4 *>(V + sv + vec * 16);
                const int64_t dst = (t0 + row) * ROW_BYTES + vec * 16;
                *reinterpret_cast<int4 *>(Kc + dst) = a;
                *reinterpret_cast<int4 *>(Vc + dst) = b;
            }
        }
    }
}

cudaError_t launch_compact(const Plan &p, const void *dK, const void *dV, const UnitAddr &aK, const UnitAddr &aV,
                           const int32_t *d_indices, const int64_t *d_offsets, void *dKc, void *dVc,
                           uint32_t *d_status, cudaStream_t st) {
    int dev = 0, sms = 148;
    cudaGetDevice(&dev);
    cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
    const int grid = sms * 8;
    if (p.shape.dtype == UNCOMP_FP32)
        compact_kernel<512><<<grid, 256, 0, st>>>((const unsigned char *)dK, (const unsigned char *)dV, aK, aV,
                                                  p.units, p.shape.N, 4, d_indices, d_offsets, (unsigned char *)dKc,
                                                  (unsigned char *)dVc, d_status);
    else
        compact_kernel<256><<<grid, 256, 0, st>>>((const unsigned char *)dK, (const unsigned char *)dV, aK, aV,
                                                  p.units, p.shape.N, 2, d_indices, d_offsets, (unsigned char *)dKc,
                                                  (unsigned char *)dVc, d_status);
    return cudaGetLastError();
}

}  // namespace uncomp
