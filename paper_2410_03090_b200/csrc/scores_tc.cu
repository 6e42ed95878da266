// Observation-window scores for bf16 keys on the tcgen05 tensor cores (paper Section 3.3.3, "Dynamic KV
// Cache Eviction": the attention of the last w query positions, summed per key position).
//
// Two kernels with one pipeline skeleton; softmax needs the row statistics before the column sums:
//   pass A  S = Qw K^T with the window rows on the TMEM lanes (M = 128 rows, N = 128 tokens per MMA tile):
//           a thread owns a row, so its running maximum and sum of exponentials are thread-local;
//           every (unit, chunk) writes partial statistics (m, l) in the log2 domain;
//   merge   partials combined in index order into m'_r = m_r + log2 l_r;
//   pass B  operands swapped (M = 128 tokens on the lanes, N = 128 rows): a thread owns a token and adds
//           2^(s c - m'_r) along its TMEM row; tokens of a warp are consecutive, the store is coalesced.
// K tiles (128 tokens x 128 features, two 128B-swizzled boxes of 64 features) stream through a TMA ring;
// the unit's window queries stay in shared memory for the whole CTA.  Both operands are K-major.
//
// CTA on one SM: warps 0-15 softmax in two groups of eight that take alternate token tiles (so the four
// warps of an SM sub-partition are in different phases: while one group waits for its accumulator, the
// other keeps the exponential unit busy); inside a group warp % 4 selects the TMEM lane quarter and bit 2
// of the warp index the 64-column half of an accumulator.  Warp 16 is the TMA producer, warp 17 allocates
// TMEM and issues the MMAs.  The 128-column accumulators form one ring that both groups draw from in item
// order (item = one 128-row block of one tile): four buffers in modes 0 and 1, three in mode 2.
// Mode 2 of the kernel is pass A with the Gram stage folded in: the K tile that is in shared memory for
// Qw K^T is also the MN-major operand of G += K_tile^T K_tile, so the entropy stage costs no second sweep
// over K.  The Gram block takes the last 128 TMEM columns; the column sums s = K^T 1 are added up by two
// extra warps (18, 19) with plain global loads of the same tokens (L2 hits), in a fixed order.
// Mode 3 is pass B with the Gram stage folded in the same way, for callers who bring the row normalisers (their
// prefill attention kernel's log-sum-exp): entropy stage and scores from ONE sweep over K.
// Every wait is bounded; a timeout raises UNCOMP_STATUS_TIMEOUT and the CTA drains and exits.
#include "tc_common.cuh"

namespace uncomp {

namespace {
constexpr int kTile = 128;
constexpr int kHalfBytes = 128 * 128;            // 64 features x 128 rows/tokens, bf16
constexpr int kBlockBytes = 2 * kHalfBytes;      // one K tile or one block of 128 query rows
constexpr int kNB = 4;                           // accumulator buffers (x 128 TMEM columns = all 512)
constexpr int kSoftThreads = 512;
constexpr int kScoreThreads = kSoftThreads + 64;  // modes 0 and 1
constexpr int kGramThreads = kScoreThreads + 64;  // mode 2: two more warps for the column sums
constexpr int kMaxStages = 4;

struct ScoreTail {
    uint64_t full[kMaxStages], empty[kMaxStages], qfull, tfull[2 * kNB], tempty[kNB], gfull;
    uint32_t tmem_base;
    float sum_xch[kD];     // hand-over of the second column-sum warp (mode 2 and 3)
};

__host__ __device__ constexpr int score_stages(int MB) { return MB <= 2 ? 4 : (MB == 3 ? 3 : 2); }
__host__ __device__ constexpr int score_smem(int MB) {
    return 1024 + MB * kBlockBytes + score_stages(MB) * kBlockBytes + MB * 128 * 4 + 2 * 4 * 128 * 4 +
           (int)sizeof(ScoreTail);
}

__device__ __forceinline__ float ex2(float x) {
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}
__device__ __forceinline__ void all_soft_barrier() { asm volatile("bar.sync 3, 512;" ::: "memory"); }
__device__ __forceinline__ void group_barrier(int g) { asm volatile("bar.sync %0, 256;" ::"r"(1 + g) : "memory"); }
__device__ __forceinline__ void sum_warps_barrier() { asm volatile("bar.sync 4, 64;" ::: "memory"); }
__device__ __forceinline__ float bf16_lo(uint32_t x) { return __uint_as_float(x << 16); }
__device__ __forceinline__ float bf16_hi(uint32_t x) { return __uint_as_float(x & 0xffff0000u); }
__device__ __forceinline__ void add_bf16x8(float (&acc)[8], const uint4 &x) {
    acc[0] += bf16_lo(x.x); acc[1] += bf16_hi(x.x);
    acc[2] += bf16_lo(x.y); acc[3] += bf16_hi(x.y);
    acc[4] += bf16_lo(x.z); acc[5] += bf16_hi(x.z);
    acc[6] += bf16_lo(x.w); acc[7] += bf16_hi(x.w);
}
// 16-byte read-only global load that does not allocate in L1
__device__ __forceinline__ uint4 ld_stream16(const void *p) {
    uint4 v;
    asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0, %1, %2, %3}, [%4];"
                 : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "l"(p));
    return v;
}
__device__ __forceinline__ float max3(float a, float b, float c) {
    float d;
    asm("max.f32 %0, %1, %2, %3;" : "=f"(d) : "f"(a), "f"(b), "f"(c));
    return d;
}

// Pass A: fold 64 logits of one row into its running (m, l), log2 domain.  m only has to stay at or above
// every logit seen so far (it is the exact running maximum here, raised lazily), l = sum 2^(x c - m).
template <bool MASKED>
__device__ __forceinline__ void stats_update(uint32_t (&v)[64], float c_log2, int pos0, int last, float &m_run,
                                             float &l_run) {
    if (MASKED) {
#pragma unroll
        for (int j = 0; j < 64; ++j)
            if (pos0 + j > last) v[j] = 0xff800000u;            // -inf: not visible to this row
    }
    float pm[4] = {-INFINITY, -INFINITY, -INFINITY, -INFINITY};
#pragma unroll
    for (int j = 0; j < 64; j += 8) {
        pm[0] = max3(pm[0], __uint_as_float(v[j]), __uint_as_float(v[j + 1]));
        pm[1] = max3(pm[1], __uint_as_float(v[j + 2]), __uint_as_float(v[j + 3]));
        pm[2] = max3(pm[2], __uint_as_float(v[j + 4]), __uint_as_float(v[j + 5]));
        pm[3] = max3(pm[3], __uint_as_float(v[j + 6]), __uint_as_float(v[j + 7]));
    }
    const float mx = fmaxf(fmaxf(pm[0], pm[1]), fmaxf(pm[2], pm[3])) * c_log2;
    if (mx > m_run) {                                           // rare after the first tiles
        l_run *= ex2(m_run - mx);
        m_run = mx;
    }
    if (m_run > -INFINITY) {
        float sum[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
        for (int j = 0; j < 64; ++j) sum[j & 3] += ex2(fmaf(__uint_as_float(v[j]), c_log2, -m_run));
        l_run += (sum[0] + sum[1]) + (sum[2] + sum[3]);
    }
}

// Pass B: sum over 64 window rows of 2^(s c - m'_r) for one token.
__device__ __forceinline__ float colsum_partial(const uint32_t (&v)[64], float c_log2, const float *mrow) {
    float acc[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
    for (int j = 0; j < 64; j += 4) {
        const float4 m4 = *reinterpret_cast<const float4 *>(mrow + j);
        acc[0] += ex2(fmaf(__uint_as_float(v[j]), c_log2, -m4.x));
        acc[1] += ex2(fmaf(__uint_as_float(v[j + 1]), c_log2, -m4.y));
        acc[2] += ex2(fmaf(__uint_as_float(v[j + 2]), c_log2, -m4.z));
        acc[3] += ex2(fmaf(__uint_as_float(v[j + 3]), c_log2, -m4.w));
    }
    return (acc[0] + acc[1]) + (acc[2] + acc[3]);
}
}  // namespace

template <int MB, int MODE>   // MODE 0: pass A, 1: pass B, 2: pass A fused with the Gram stage, 3: pass B fused with it
__global__ void __launch_bounds__(kGramThreads, 1)
score_tc_kernel(const __grid_constant__ CUtensorMap tmapQ, const __grid_constant__ CUtensorMap tmapK, int L, int H,
                int N, int w, int rows, int chunk, int splits, float c_log2, float *__restrict__ stats_part,
                const float *__restrict__ mprime, float *__restrict__ raw, float *__restrict__ gram_part,
                const void *__restrict__ Kraw, const UnitAddr kaddr, uint32_t *__restrict__ status) {
    constexpr bool PASS_B = MODE == 1 || MODE == 3, GRAM = MODE >= 2;
    // Accumulator buffers (128 TMEM columns each).  An item is one 128-row block of one tile; tile i belongs to
    // softmax group i & 1.  Modes 0 and 1: four buffers, two owned by each group, which it fills alternately
    // with its own items (so each group runs up to two items ahead, independent of the other).  Mode 2: the
    // Gram block leaves room for three, which form one ring over all items in issue order.
    constexpr int NB = GRAM ? 3 : kNB;
    // Mode 2: "item n is ready" is signalled on barrier n % (2 NB).  A softmax group that waits for the first item
    // of its next tile may get there before the other group's item n - NB has completed, and with one barrier per
    // buffer the parity of that unfinished phase could not be told from the one waited for.  The user of barrier
    // n % (2 NB) before item n is item n - 2 NB, which lies in a tile this group has already consumed (2 NB > MB).
    // Modes 0 and 1 need no such care: a group only ever waits on its own buffers.
    constexpr int NF = 2 * NB;
    // item (tile i, block mb) -> buffer, ready barrier and its parity, and the drain phase the MMA thread waits for
    // (-1: the buffer has not been used yet)
    auto item_buf = [](int i, int mb) { return GRAM ? (i * MB + mb) % NB : 2 * (i & 1) + (((i >> 1) * MB + mb) & 1); };
    auto item_ready_bar = [](int i, int mb) { return GRAM ? (i * MB + mb) % NF : 2 * (i & 1) + (((i >> 1) * MB + mb) & 1); };
    auto item_ready_parity = [](int i, int mb) { return GRAM ? ((i * MB + mb) / NF) & 1 : ((((i >> 1) * MB + mb) >> 1) & 1); };
    auto item_drain_phase = [](int i, int mb) { return GRAM ? (i * MB + mb) / NB - 1 : ((((i >> 1) * MB + mb) >> 1) - 1); };
    constexpr uint32_t kGramCol = 384;               // TMEM columns of the Gram block (mode 2)
    constexpr int S = score_stages(MB);
    extern __shared__ unsigned char smem_raw[];
    const uint32_t raw_addr = tc::smem_u32(smem_raw);
    const uint32_t pad = (1024u - (raw_addr & 1023u)) & 1023u;
    unsigned char *smem = smem_raw + pad;
    const uint32_t q_addr = raw_addr + pad;
    const uint32_t k_addr = q_addr + MB * kBlockBytes;
    float *mp = reinterpret_cast<float *>(smem + (MB + S) * kBlockBytes);      // [MB * 128]
    float *colsum = mp + MB * 128;                                             // [2][4][128]
    ScoreTail &T = *reinterpret_cast<ScoreTail *>(colsum + 2 * 4 * 128);

    const int c = blockIdx.x, u = blockIdx.y;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int h = u % H, l = (u / H) % L, b = u / (H * L);
    const int P = N - w;
    const int limit = (PASS_B && !GRAM) ? P : N;   // pass B only scores the prefix; the Gram stage needs every token
    const int t0 = c * chunk;
    const int t1 = min(limit, t0 + chunk);
    const int ntiles = t1 > t0 ? (t1 - t0 + kTile - 1) / kTile : 0;

    if (threadIdx.x == 0) {
        for (int s = 0; s < S; ++s) {
            tc::mbar_init(tc::smem_u32(&T.full[s]), 1);
            tc::mbar_init(tc::smem_u32(&T.empty[s]), 1);
        }
        tc::mbar_init(tc::smem_u32(&T.qfull), 1);
        tc::mbar_init(tc::smem_u32(&T.gfull), 1);
        for (int i = 0; i < 2 * kNB; ++i) tc::mbar_init(tc::smem_u32(&T.tfull[i]), 1);
        for (int i = 0; i < kNB; ++i) tc::mbar_init(tc::smem_u32(&T.tempty[i]), kSoftThreads / 64);   // the 8 warps of one group
        tc::fence_mbar_init();
    }
    if (warp == 17) {
        tc::tmem_alloc(tc::smem_u32(&T.tmem_base), 512);
        tc::tmem_relinquish();
    }
    if (warp == 16 && lane == 0) {
        tc::prefetch_tmap(&tmapQ);
        tc::prefetch_tmap(&tmapK);
    }
    tc::tc_fence_before();
    __syncthreads();
    tc::tc_fence_after();
    const uint32_t tmem = T.tmem_base;

    if (warp == 16) {
        // ---------------- TMA producer ----------------
        if (lane == 0 && ntiles > 0) {
            const uint32_t qbar = tc::smem_u32(&T.qfull);
            tc::mbar_expect_tx(qbar, MB * kBlockBytes);
            for (int mb = 0; mb < MB; ++mb) {
                tc::tma_load_3d(q_addr + mb * kBlockBytes, &tmapQ, qbar, 0, mb * 128, u);
                tc::tma_load_3d(q_addr + mb * kBlockBytes + kHalfBytes, &tmapQ, qbar, 64, mb * 128, u);
            }
            int issued = 0;
            bool ok = true;
            for (int i = 0; i < ntiles; ++i, ++issued) {
                const int s = i % S;
                if (i >= S) ok = tc::mbar_wait(tc::smem_u32(&T.empty[s]), ((i / S) - 1) & 1, status);
                if (!ok) break;
                const uint32_t bar = tc::smem_u32(&T.full[s]);
                const uint32_t dst = k_addr + s * kBlockBytes;
                tc::mbar_expect_tx(bar, kBlockBytes);
                tc::tma_load_5d(dst, &tmapK, bar, 0, t0 + i * kTile, h, l, b);
                tc::tma_load_5d(dst + kHalfBytes, &tmapK, bar, 64, t0 + i * kTile, h, l, b);
            }
            if (!ok) {   // let the copies in flight land before the CTA may exit (bounded)
                tc::mbar_wait(qbar, 0, status);
                for (int i = max(0, issued - S); i < issued; ++i)
                    tc::mbar_wait(tc::smem_u32(&T.full[i % S]), (i / S) & 1, status);
            }
        }
    } else if (warp == 17) {
        // ---------------- MMA issue ----------------
        if (lane == 0 && ntiles > 0) {
            constexpr uint32_t idesc = tc::idesc_bf16_f32(128, 128, 0, 0);
            // descriptors: K-major, 128-byte swizzle, 8-row groups 1024 B apart.  Only the address field
            // (16-byte units) of the lower half changes: +2 per 16 features inside a 128-byte row, +1024 for
            // the second 64-feature half.
            const uint64_t d0 = tc::smem_desc_sw128(q_addr, 16, 1024);
            const uint32_t dhi = tc::desc_hi(d0);
            uint32_t q_lo[MB];
#pragma unroll
            for (int mb = 0; mb < MB; ++mb) q_lo[mb] = tc::desc_lo(d0) + (uint32_t)(mb * kBlockBytes >> 4);
            const uint32_t k_lo0 = tc::desc_lo(tc::smem_desc_sw128(k_addr, 16, 1024));
            const uint64_t gd = tc::smem_desc_sw128(k_addr, kHalfBytes, 1024);
            const uint32_t g_lo0 = tc::desc_lo(gd), g_hi = tc::desc_hi(gd);
            // Mode 2: the Gram MMAs of a tile only have to be issued before its stage is handed back, so they
            // are deferred by up to one tile and issued while this thread would otherwise wait for an
            // accumulator: the latency-critical QK^T MMAs never queue behind them.
            int g_done = 0;                    // tiles whose Gram MMAs are issued (and whose stage is released)
            auto issue_gram = [&](int t) {
                constexpr uint32_t idesc_g = tc::idesc_bf16_f32(128, 128, 1, 1);
                const int sg = t % S;
                const uint32_t g_lo = g_lo0 + (uint32_t)(sg * (kBlockBytes >> 4));
#pragma unroll
                for (int k = 0; k < kTile / 16; ++k) {
                    // the same stage read MN-major (feature halves kHalfBytes apart, 8-token groups 1024 B
                    // apart); 16 tokens further = +128 address units
                    const uint32_t acc = (t > 0 || k > 0) ? 1u : 0u;
                    tc::mma_f16_ss_lohi(tmem + kGramCol, g_lo + k * 128, g_lo + k * 128, g_hi, idesc_g, acc);
                }
                tc::mma_commit(tc::smem_u32(&T.empty[sg]));
            };
            bool ok = tc::mbar_wait(tc::smem_u32(&T.qfull), 0, status);
            for (int i = 0; i < ntiles && ok; ++i) {
                const int s = i % S;
                ok = tc::mbar_wait(tc::smem_u32(&T.full[s]), (i / S) & 1, status);
                if (!ok) break;
                const uint32_t k_lo = k_lo0 + (uint32_t)(s * (kBlockBytes >> 4));
#pragma unroll
                for (int mb = 0; mb < MB; ++mb) {
                    // the item's buffer must have been drained of its previous item
                    const int buf = item_buf(i, mb), drain = item_drain_phase(i, mb);
                    if (ok && drain >= 0) {
                        const uint32_t bar = tc::smem_u32(&T.tempty[buf]);
                        const uint32_t parity = drain & 1;
                        if (GRAM) {
                            uint32_t spins = 0;
                            while (!tc::mbar_try_wait(bar, parity)) {
                                if (g_done < i) issue_gram(g_done++);
                                else if (++spins >= tc::kSpinLimit) {
                                    atomicOr(status, (uint32_t)UNCOMP_STATUS_TIMEOUT);
                                    ok = false;
                                    break;
                                }
                            }
                        } else {
                            ok = tc::mbar_wait(bar, parity, status);
                        }
                    }
                    if (!ok) break;
                    tc::tc_fence_after();
                    const uint32_t d_tmem = tmem + buf * 128;
#pragma unroll
                    for (int k = 0; k < 8; ++k) {
                        const uint32_t off = (uint32_t)(k >> 2) * (kHalfBytes >> 4) + (uint32_t)(k & 3) * 2;
                        if (PASS_B) tc::mma_f16_ss_lohi(d_tmem, k_lo + off, q_lo[mb] + off, dhi, idesc, k > 0);
                        else tc::mma_f16_ss_lohi(d_tmem, q_lo[mb] + off, k_lo + off, dhi, idesc, k > 0);
                    }
                    tc::mma_commit(tc::smem_u32(&T.tfull[item_ready_bar(i, mb)]));
                }
                if (!ok) break;
                if (GRAM) {
                    while (g_done < i) issue_gram(g_done++);      // at most one tile may stay pending
                } else {
                    tc::mma_commit(tc::smem_u32(&T.empty[s]));
                }
            }
            if (GRAM) {
                if (ok) while (g_done < ntiles) issue_gram(g_done++);
                tc::mma_commit(tc::smem_u32(&T.gfull));
            }
        }
    } else if (warp >= 18) {
        // ---------------- column sums s = K^T 1 (mode 2 only) ----------------
        // Two warps add up the CTA's token chunk with plain 16-byte global loads (the lines are in L2: the TMA
        // stream fetches the same tokens), so the shared-memory banks stay with the MMA operands and the sums
        // need no place in the tile pipeline.  A lane owns one 16-byte chunk (8 features) of the 256-byte row and
        // one of four row phases; its rows are added in increasing order, the phases in a fixed order below.
        if (GRAM) {
            const int sw = warp - 18, ch = lane & 15, phase = 2 * sw + (lane >> 4);
            float acc[8] = {0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f};
            const unsigned char *rowp = reinterpret_cast<const unsigned char *>(Kraw) +
                                        2 * (kaddr.base(u) + (int64_t)(t0 + phase) * kaddr.sN) + 16 * ch;
            const int64_t step = 2 * 4 * kaddr.sN;                 // four rows further, in bytes
            const int nrows = t1 > t0 + phase ? (t1 - t0 - phase + 3) / 4 : 0;
            int r = 0;
            for (; r + 16 <= nrows; r += 16) {          // 16 loads in flight per lane cover the L2 latency
                uint4 x[16];
#pragma unroll
                for (int q = 0; q < 16; ++q) x[q] = ld_stream16(rowp + (int64_t)(r + q) * step);
#pragma unroll
                for (int q = 0; q < 16; ++q) add_bf16x8(acc, x[q]);
            }
            for (; r < nrows; ++r) add_bf16x8(acc, ld_stream16(rowp + (int64_t)r * step));
#pragma unroll
            for (int e = 0; e < 8; ++e) acc[e] += __shfl_xor_sync(0xffffffffu, acc[e], 16);   // phases 2 sw, 2 sw + 1
            float *xch = T.sum_xch;
            if (sw == 1 && lane < 16) {
#pragma unroll
                for (int e = 0; e < 8; ++e) xch[ch * 8 + e] = acc[e];
            }
            sum_warps_barrier();
            if (sw == 0 && lane < 16 && ntiles > 0) {
                float *out = gram_part + ((size_t)u * splits + c) * (kD * kD + kD) + kD * kD;
#pragma unroll
                for (int e = 0; e < 8; ++e) out[ch * 8 + e] = acc[e] + xch[ch * 8 + e];
            }
        }
    } else {
        // ---------------- softmax warps ----------------
        const int quarter = warp & 3, half = (warp >> 2) & 1, group = warp >> 3;
        const int lane_row = quarter * 32 + lane;          // TMEM lane: a window row (A) or a token (B)
        const uint32_t tbase = tmem + ((uint32_t)(quarter * 32) << 16) + (uint32_t)half * 64;
        bool dead = false;
        if (PASS_B) {
            for (int r = threadIdx.x; r < MB * 128; r += kSoftThreads)
                mp[r] = r < rows ? mprime[(size_t)u * kMaxRows + r] : INFINITY;
            all_soft_barrier();
        }
        float m_run[MB], l_run[MB];
#pragma unroll
        for (int mb = 0; mb < MB; ++mb) { m_run[mb] = -INFINITY; l_run[mb] = 0.f; }

        for (int i = group; i < ntiles; i += 2) {           // this group's tiles
            const int tile_t0 = t0 + i * kTile;
            const bool masked = tile_t0 + kTile > P;            // uniform over the CTA
            float acc = 0.f;
#pragma unroll
            for (int mb = 0; mb < MB; ++mb) {
                const int buf = item_buf(i, mb);
                uint32_t v[64];
                if (!dead) {
                    const bool ok = tc::mbar_wait(tc::smem_u32(&T.tfull[item_ready_bar(i, mb)]), item_ready_parity(i, mb),
                                                  status);
                    dead = !__all_sync(0xffffffffu, ok);
                }
                if (!dead) {
                    tc::tc_fence_after();
                    uint32_t va[32], vb[32];
                    tc::tmem_ld32(tbase + buf * 128, va);
                    tc::tmem_ld32(tbase + buf * 128 + 32, vb);
                    tc::tmem_ld_wait();
#pragma unroll
                    for (int j = 0; j < 32; ++j) { v[j] = va[j]; v[32 + j] = vb[j]; }
                    tc::tc_fence_before();
                    __syncwarp();
                    if (lane == 0) tc::mbar_arrive(tc::smem_u32(&T.tempty[buf]));
                } else {
#pragma unroll
                    for (int j = 0; j < 64; ++j) v[j] = 0u;
                }
                if (PASS_B) {
                    acc += colsum_partial(v, c_log2, mp + mb * 128 + half * 64);
                } else {
                    const int r = mb * 128 + lane_row;
                    const int last = P + (r % w);                       // last visible position of this row
                    const int pos0 = tile_t0 + half * 64;
                    if (masked) stats_update<true>(v, c_log2, pos0, last, m_run[mb], l_run[mb]);
                    else stats_update<false>(v, c_log2, pos0, last, m_run[mb], l_run[mb]);
                }
            }
            if (PASS_B) {
                // the two column halves of this group meet in shared memory (slot = tile parity within the group)
                float *cs = colsum + ((i >> 1) & 1) * 512 + group * 256;
                cs[half * 128 + lane_row] = acc;
                group_barrier(group);
                const int pos = tile_t0 + lane_row;
                if (half == 0 && pos < min(t1, P) && !dead) raw[(size_t)u * P + pos] = cs[lane_row] + cs[128 + lane_row];
            }
        }
        if (!PASS_B) {
            // merge the four (group, half) partials of every row in a fixed order.  Scratch: the query blocks,
            // which no MMA reads any more once both groups have consumed every accumulator (the K stages may still
            // feed deferred Gram MMAs).
            float2 *merge = reinterpret_cast<float2 *>(smem);                         // [4][MB * 128]
            all_soft_barrier();            // both groups have consumed their last accumulator
            const int slot = group * 2 + half;
#pragma unroll
            for (int mb = 0; mb < MB; ++mb) merge[slot * (MB * 128) + mb * 128 + lane_row] = make_float2(m_run[mb], l_run[mb]);
            all_soft_barrier();
            if (slot == 0 && !dead) {
#pragma unroll
                for (int mb = 0; mb < MB; ++mb) {
                    const int r = mb * 128 + lane_row;
                    if (r < rows) {
                        float m = -INFINITY;
#pragma unroll
                        for (int sl = 0; sl < 4; ++sl) m = fmaxf(m, merge[sl * (MB * 128) + r].x);
                        float lsum = 0.f;
#pragma unroll
                        for (int sl = 0; sl < 4; ++sl) {
                            const float2 ml = merge[sl * (MB * 128) + r];
                            if (ml.x > -INFINITY) lsum += ml.y * ex2(ml.x - m);
                        }
                        float *o = stats_part + (((size_t)u * splits + c) * kMaxRows + r) * 2;
                        o[0] = m;
                        o[1] = lsum;
                    }
                }
            }
        }
        if (GRAM) {
            // drain the Gram block: warp (quarter, cb) stores rows 32 quarter .. +31, columns 32 cb .. +31
            bool ok = ntiles > 0 && tc::mbar_wait(tc::smem_u32(&T.gfull), 0, status);
            ok = __all_sync(0xffffffffu, ok) && !dead;
            if (ok) {
                tc::tc_fence_after();
                const int cb = warp >> 2;
                float *out = gram_part + ((size_t)u * splits + c) * (kD * kD + kD);
                uint32_t r[32];
                tc::tmem_ld32(tmem + ((uint32_t)(quarter * 32) << 16) + kGramCol + cb * 32, r);
                tc::tmem_ld_wait();
                float4 *dst = reinterpret_cast<float4 *>(out + (size_t)lane_row * kD + cb * 32);
#pragma unroll
                for (int q4 = 0; q4 < 8; ++q4)
                    dst[q4] = make_float4(__uint_as_float(r[4 * q4]), __uint_as_float(r[4 * q4 + 1]),
                                          __uint_as_float(r[4 * q4 + 2]), __uint_as_float(r[4 * q4 + 3]));
            }
        }
    }
    tc::tc_fence_before();
    __syncthreads();
    if (warp == 17) tc::tmem_dealloc(tmem, 512);
}

// one thread per (unit, row): partial (m, l) in index order -> m' = m + log2 l
__global__ void score_tc_merge_kernel(const float *__restrict__ stats_part, int units, int rows, int parts,
                                      float *__restrict__ mprime) {
    const int idx = blockIdx.x * blockDim.x + threadIdx.x;
    if (idx >= units * rows) return;
    const int u = idx / rows, r = idx % rows;
    float m = -INFINITY;
    for (int p = 0; p < parts; ++p) m = fmaxf(m, stats_part[(((size_t)u * parts + p) * kMaxRows + r) * 2]);
    float l = 0.f;
    for (int p = 0; p < parts; ++p) {
        const float *s = stats_part + (((size_t)u * parts + p) * kMaxRows + r) * 2;
        if (s[0] > -INFINITY) l += s[1] * exp2f(s[0] - m);
    }
    mprime[(size_t)u * kMaxRows + r] = m + log2f(l);
}

// cudaFuncSetAttribute is sticky per function and device: done once per device and instantiation
template <int MB>
static cudaError_t raise_smem_limit_once() {
    static bool done[64] = {};
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    if (dev >= 0 && dev < 64 && done[dev]) return cudaSuccess;
    const int smem = score_smem(MB);
    e = cudaFuncSetAttribute(score_tc_kernel<MB, 0>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
    if (e == cudaSuccess) e = cudaFuncSetAttribute(score_tc_kernel<MB, 1>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
    if (e == cudaSuccess) e = cudaFuncSetAttribute(score_tc_kernel<MB, 2>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
    if (e == cudaSuccess && dev >= 0 && dev < 64) done[dev] = true;
    return e;
}

template <int MB>
static cudaError_t raise_smem_limit_mode3() {
    static bool done[64] = {};
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    if (dev >= 0 && dev < 64 && done[dev]) return cudaSuccess;
    e = cudaFuncSetAttribute(score_tc_kernel<MB, 3>, cudaFuncAttributeMaxDynamicSharedMemorySize, score_smem(MB));
    if (e == cudaSuccess && dev >= 0 && dev < 64) done[dev] = true;
    return e;
}

template <int MB>
static cudaError_t launch_scores_tc_mb(const Plan &p, const CUtensorMap &tq, const CUtensorMap &tk, const void *dK,
                                       const UnitAddr &addr, float c_log2,
                                       const float *d_lse, float *d_stats_part, float *d_mprime, float *d_raw,
                                       float *d_gram_part, int phases, uint32_t *d_status, Profiler *prof,
                                       cudaStream_t st) {
    const uncomp_shape &s = p.shape;
    const int smem = score_smem(MB);
    cudaError_t e = raise_smem_limit_once<MB>();
    if (e != cudaSuccess) return e;
    if (phases & kScorePhaseStats) {
        ProfScope ps(prof, d_gram_part ? kSlotGramStats : kSlotScoreStats, st);
        dim3 grid(p.score_splits, p.units);
        if (d_gram_part)
            score_tc_kernel<MB, 2><<<grid, kGramThreads, smem, st>>>(tq, tk, s.L, s.H, s.N, s.w, p.rows, p.score_chunk,
                                                                      p.score_splits, c_log2, d_stats_part, nullptr,
                                                                      nullptr, d_gram_part, dK, addr, d_status);
        else
            score_tc_kernel<MB, 0><<<grid, kScoreThreads, smem, st>>>(tq, tk, s.L, s.H, s.N, s.w, p.rows, p.score_chunk,
                                                                      p.score_splits, c_log2, d_stats_part, nullptr,
                                                                      nullptr, nullptr, nullptr, addr, d_status);
    }
    if (phases & kScorePhaseColsum) {
        const bool with_gram = (phases & kScorePhaseStats) == 0 && d_gram_part != nullptr;   // mode 3
        {
            ProfScope ps(prof, kSlotStatsMerge, st);
            if (d_lse) {
                e = launch_lse_import(p, d_lse, d_mprime, true, d_status, st);
                if (e != cudaSuccess) return e;
            } else {
                const int total = p.units * p.rows;
                score_tc_merge_kernel<<<(total + 255) / 256, 256, 0, st>>>(d_stats_part, p.units, p.rows,
                                                                           p.score_splits, d_mprime);
            }
        }
        ProfScope ps(prof, with_gram ? kSlotGramColsum : kSlotScoreColsum, st);
        const int splitsB = (p.prefix + p.score_chunk - 1) / p.score_chunk;
        if (with_gram) {
            e = raise_smem_limit_mode3<MB>();
            if (e != cudaSuccess) return e;
            dim3 grid3(p.score_splits, p.units);
            score_tc_kernel<MB, 3><<<grid3, kGramThreads, smem, st>>>(tq, tk, s.L, s.H, s.N, s.w, p.rows, p.score_chunk,
                                                                     p.score_splits, c_log2, nullptr, d_mprime, d_raw,
                                                                     d_gram_part, dK, addr, d_status);
            return cudaGetLastError();
        }
        dim3 grid(splitsB, p.units);
        score_tc_kernel<MB, 1><<<grid, kScoreThreads, smem, st>>>(tq, tk, s.L, s.H, s.N, s.w, p.rows, p.score_chunk,
                                                                  splitsB, c_log2, nullptr, d_mprime, d_raw, nullptr,
                                                                  nullptr, addr, d_status);
    }
    return cudaGetLastError();
}

cudaError_t launch_scores_tc(const Plan &p, const void *dQw, const void *dK, const UnitAddr &addr, float scale,
                             const float *d_lse, float *d_stats_part, float *d_stats, float *d_raw, float *d_gram_part,
                             int phases, uint32_t *d_status, TmapCache *cache, Profiler *prof, cudaStream_t st) {
    CUtensorMap tq, tk;
    cudaError_t e = cached_scorer_maps(cache, p, addr, dQw, dK, kTile, &tq, &tk);
    if (e != cudaSuccess) return e;
    const float c_log2 = scale * 1.4426950408889634f;
    const int MB = (p.rows + 127) / 128;
    switch (MB) {
        case 1: return launch_scores_tc_mb<1>(p, tq, tk, dK, addr, c_log2, d_lse, d_stats_part, d_stats, d_raw, d_gram_part, phases, d_status, prof, st);
        case 2: return launch_scores_tc_mb<2>(p, tq, tk, dK, addr, c_log2, d_lse, d_stats_part, d_stats, d_raw, d_gram_part, phases, d_status, prof, st);
        case 3: return launch_scores_tc_mb<3>(p, tq, tk, dK, addr, c_log2, d_lse, d_stats_part, d_stats, d_raw, d_gram_part, phases, d_status, prof, st);
        default: return launch_scores_tc_mb<4>(p, tq, tk, dK, addr, c_log2, d_lse, d_stats_part, d_stats, d_raw, d_gram_part, phases, d_status, prof, st);
    }
}

}  // namespace uncomp
