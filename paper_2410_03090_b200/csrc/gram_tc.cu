// Per-unit Gram matrix G = X^T X (d x d) and column sums s = X^T 1 for bf16 keys on the tcgen05 tensor
// cores, operands staged by TMA (the covariance of the paper's Eq. 1 is assembled from both later).
//
// The contraction runs over tokens, the strided dimension of the [tokens x d] key matrix, so both MMA
// operands are the SAME shared-memory tile read "MN-major": A[m][k] = B[m][k] = X[token k][feature m].
// A tile of 128 tokens x 128 features arrives as two TMA boxes of 64 features (128 bytes, 128B-swizzled):
// token rows 128 B apart, 8-row groups 1024 B apart, the second feature half one region (16 KB) further.
// One MMA consumes 16 tokens: M = N = 128, K = 16, fp32 accumulator of 128 lanes x 128 columns in TMEM.
// The column sums come from a second, narrow MMA of the same A against an all-ones B (N = 16).
//
// Grid (P token chunks, units), 192 threads, two CTAs per SM:
//   warps 0-3  epilogue: TMEM -> registers -> global partial [d*d + d] of this (unit, chunk)
//   warp  4    TMA producer (one elected lane), 3-stage ring of 32 KB tiles
//   warp  5    TMEM allocation and MMA issue (one elected lane)
// Tokens beyond N are zero-filled by TMA, chunk boundaries are multiples of the tile, so a ragged tail
// needs no special case.  Every mbarrier wait is bounded; a timeout raises UNCOMP_STATUS_TIMEOUT.
#include "tc_common.cuh"

namespace uncomp {

namespace {
constexpr int kTile = 128;                       // tokens per stage
constexpr int kStages = 3;
constexpr int kRegion = kTile * 128;             // bytes of one 64-feature half of a tile
constexpr int kStageBytes = 2 * kRegion;         // 32 KB
constexpr int kOnesBytes = 2048;                 // 16 token rows x 128 B of bf16 ones
constexpr int kTmemCols = 256;                   // 128 (Gram) + 16 (column sums), power of two
constexpr int kGramThreads = 192;

struct GramSmemTail {
    uint64_t full[kStages];
    uint64_t empty[kStages];
    uint64_t accum;
    uint32_t tmem_base;
    uint32_t abort;
};
constexpr int kGramSmem = 1024 /*alignment slack*/ + kStages * kStageBytes + kOnesBytes + (int)sizeof(GramSmemTail);
}  // namespace

__global__ void __launch_bounds__(kGramThreads, 2)
gram_tc_kernel(const __grid_constant__ CUtensorMap tmap, int L, int H, int N, int chunk, int P,
               float *__restrict__ partials, uint32_t *__restrict__ status) {
    extern __shared__ unsigned char smem_raw[];
    const uint32_t raw_addr = tc::smem_u32(smem_raw);
    const uint32_t pad = (1024u - (raw_addr & 1023u)) & 1023u;
    unsigned char *smem = smem_raw + pad;
    const uint32_t tiles_addr = raw_addr + pad;
    unsigned char *ones = smem + kStages * kStageBytes;
    GramSmemTail &T = *reinterpret_cast<GramSmemTail *>(ones + kOnesBytes);

    const int p = blockIdx.x, u = blockIdx.y;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int h = u % H, l = (u / H) % L, b = u / (H * L);
    const int t0 = p * chunk;
    const int t1 = min(N, t0 + chunk);
    const int ntiles = (t1 - t0 + kTile - 1) / kTile;

    if (threadIdx.x == 0) {
        for (int s = 0; s < kStages; ++s) {
            tc::mbar_init(tc::smem_u32(&T.full[s]), 1);
            tc::mbar_init(tc::smem_u32(&T.empty[s]), 1);
        }
        tc::mbar_init(tc::smem_u32(&T.accum), 1);
        T.abort = 0;
        tc::fence_mbar_init();
    }
    // all-ones B operand of the column-sum MMA
    for (int i = threadIdx.x; i < kOnesBytes / 4; i += kGramThreads)
        reinterpret_cast<uint32_t *>(ones)[i] = 0x3f803f80u;
    tc::fence_proxy_async();
    if (warp == 5) {
        tc::tmem_alloc(tc::smem_u32(&T.tmem_base), kTmemCols);
        tc::tmem_relinquish();
    }
    if (warp == 4 && lane == 0) tc::prefetch_tmap(&tmap);
    tc::tc_fence_before();
    __syncthreads();
    tc::tc_fence_after();
    const uint32_t tmem = T.tmem_base;

    if (warp == 4) {
        // ---------------- TMA producer ----------------
        if (lane == 0) {
            int issued = 0;
            for (int i = 0; i < ntiles; ++i, ++issued) {
                const int s = i % kStages;
                if (i >= kStages && !tc::mbar_wait(tc::smem_u32(&T.empty[s]), ((i / kStages) - 1) & 1, status)) {
                    T.abort = 1;
                    break;
                }
                const uint32_t bar = tc::smem_u32(&T.full[s]);
                const uint32_t dst = tiles_addr + s * kStageBytes;
                tc::mbar_expect_tx(bar, kStageBytes);
                tc::tma_load_5d(dst, &tmap, bar, 0, t0 + i * kTile, h, l, b);
                tc::tma_load_5d(dst + kRegion, &tmap, bar, 64, t0 + i * kTile, h, l, b);
            }
            if (T.abort) {
                // let the copies already in flight land before the CTA may exit (bounded)
                for (int i = max(0, issued - kStages); i < issued; ++i)
                    tc::mbar_wait(tc::smem_u32(&T.full[i % kStages]), (i / kStages) & 1, status);
            }
        }
    } else if (warp == 5) {
        // ---------------- MMA issue ----------------
        if (lane == 0) {
            constexpr uint32_t idesc_g = tc::idesc_bf16_f32(128, 128, 1, 1);
            constexpr uint32_t idesc_s = tc::idesc_bf16_f32(128, 16, 1, 1);
            // descriptors: MN-major, 128-byte swizzle; feature halves kRegion apart (LBO), 8-token groups
            // 1024 B apart (SBO).  16 tokens further = 2048 B = +128 in the address field (16-byte units).
            const uint64_t ones_desc = tc::smem_desc_sw128(tiles_addr + kStages * kStageBytes, 1024, 1024);
            const uint64_t tile_desc = tc::smem_desc_sw128(tiles_addr, kRegion, 1024);
            const uint32_t dhi = tc::desc_hi(tile_desc), ones_hi = tc::desc_hi(ones_desc);
            const uint32_t ones_lo = tc::desc_lo(ones_desc);
            bool ok = true;
            for (int i = 0; i < ntiles && ok; ++i) {
                const int s = i % kStages;
                ok = tc::mbar_wait(tc::smem_u32(&T.full[s]), (i / kStages) & 1, status);
                if (!ok) { T.abort = 1; break; }
                tc::tc_fence_after();
                const uint32_t lo = tc::desc_lo(tile_desc) + (uint32_t)(s * (kStageBytes >> 4));
#pragma unroll
                for (int k = 0; k < kTile / 16; ++k) {
                    const uint32_t acc = (i > 0 || k > 0) ? 1u : 0u;
                    tc::mma_f16_ss_lohi(tmem, lo + k * 128, lo + k * 128, dhi, idesc_g, acc);
                    tc::mma_f16_ss2(tmem + 128, lo + k * 128, dhi, ones_lo, ones_hi, idesc_s, acc);
                }
                tc::mma_commit(tc::smem_u32(&T.empty[s]));   // stage reusable once these MMAs have read it
            }
            tc::mma_commit(tc::smem_u32(&T.accum));           // accumulator complete
        }
    } else {
        // ---------------- epilogue: warps 0-3 own TMEM lanes 32*warp .. 32*warp+31 ----------------
        const bool ok = tc::mbar_wait(tc::smem_u32(&T.accum), 0, status);
        tc::tc_fence_after();
        if (ok && !T.abort) {
            const int m = warp * 32 + lane;        // feature row of the Gram matrix
            float *out = partials + ((size_t)u * P + p) * (kD * kD + kD);
            uint32_t r[32];
#pragma unroll 1
            for (int c0 = 0; c0 < 128; c0 += 32) {
                tc::tmem_ld32(tmem + ((uint32_t)(warp * 32) << 16) + c0, r);
                tc::tmem_ld_wait();
                float4 *dst = reinterpret_cast<float4 *>(out + (size_t)m * kD + c0);
#pragma unroll
                for (int q = 0; q < 8; ++q)
                    dst[q] = make_float4(__uint_as_float(r[4 * q]), __uint_as_float(r[4 * q + 1]),
                                         __uint_as_float(r[4 * q + 2]), __uint_as_float(r[4 * q + 3]));
            }
            tc::tmem_ld32(tmem + ((uint32_t)(warp * 32) << 16) + 128, r);   // only column 128 is used
            tc::tmem_ld_wait();
            out[kD * kD + m] = __uint_as_float(r[0]);
        }
    }
    tc::tc_fence_before();
    __syncthreads();
    if (warp == 5) tc::tmem_dealloc(tmem, kTmemCols);
}

cudaError_t launch_gram_tc(const Plan &p, const void *dK, const UnitAddr &addr, void *d_partials, uint32_t *d_status,
                           cudaStream_t st) {
    const uncomp_shape &s = p.shape;
    CUtensorMap tmap;
    cudaError_t e = make_key_tensor_map(&tmap, s, addr, dK, kTile);
    if (e != cudaSuccess) return e;
    e = cudaFuncSetAttribute(gram_tc_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kGramSmem);
    if (e != cudaSuccess) return e;
    dim3 grid(p.gram_splits, p.units);
    gram_tc_kernel<<<grid, kGramThreads, kGramSmem, st>>>(tmap, s.L, s.H, s.N, p.gram_chunk, p.gram_splits,
                                                          (float *)d_partials, d_status);
    return cudaGetLastError();
}

}  // namespace uncomp
