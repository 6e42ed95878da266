// Host helper: tiled tensor maps for TMA, encoded through the driver entry point that the CUDA runtime
// hands out, so the library has no link-time dependency on the driver library.
#include "tc_common.cuh"

namespace uncomp {

typedef CUresult (*EncodeTiledFn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *,
                                  const cuuint64_t *, const cuuint32_t *, const cuuint32_t *, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

cudaError_t encode_tensor_map(CUtensorMap *map, const void *base, int rank, const uint64_t *dims,
                              const uint64_t *strides_bytes, const uint32_t *box, CUtensorMapDataType dtype,
                              CUtensorMapSwizzle swizzle) {
    static EncodeTiledFn fn = nullptr;
    if (!fn) {
        void *sym = nullptr;
        cudaDriverEntryPointQueryResult q;
        cudaError_t e = cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &sym, cudaEnableDefault, &q);
        if (e != cudaSuccess) return e;
        if (q != cudaDriverEntryPointSuccess || !sym) return cudaErrorNotSupported;
        fn = reinterpret_cast<EncodeTiledFn>(sym);
    }
    cuuint64_t gdim[5], gstr[4];
    cuuint32_t bx[5], es[5];
    for (int i = 0; i < rank; ++i) { gdim[i] = dims[i]; bx[i] = box[i]; es[i] = 1; }
    for (int i = 0; i + 1 < rank; ++i) gstr[i] = strides_bytes[i];
    const CUresult r = fn(map, dtype, (cuuint32_t)rank, const_cast<void *>(base), gdim, gstr, bx, es,
                          CU_TENSOR_MAP_INTERLEAVE_NONE, swizzle, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
                          CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    return r == CUDA_SUCCESS ? cudaSuccess : cudaErrorInvalidValue;
}

// Tensor map over bf16 keys [B, L, H, N, d] with arbitrary (16-byte aligned) strides: dimensions
// (feature, token, head, layer, batch), box = 64 features x tile_tokens tokens, 128-byte swizzle.
// Tokens beyond N read as zero.
cudaError_t make_key_tensor_map(CUtensorMap *map, const uncomp_shape &s, const UnitAddr &addr, const void *dK,
                                int tile_tokens) {
    uint64_t dims[5] = {(uint64_t)s.d, (uint64_t)s.N, (uint64_t)s.H, (uint64_t)s.L, (uint64_t)s.B};
    uint64_t str[4] = {(uint64_t)addr.sN * 2, (uint64_t)addr.sH * 2, (uint64_t)addr.sL * 2, (uint64_t)addr.sB * 2};
    // a dimension of extent 1 may come with stride 0: give it a harmless valid stride
    for (int i = 0; i < 4; ++i)
        if (dims[i + 1] == 1 && str[i] == 0) str[i] = (i == 0 ? (uint64_t)s.d * 2 : str[i - 1] * dims[i]);
    uint32_t box[5] = {64, (uint32_t)tile_tokens, 1, 1, 1};
    return encode_tensor_map(map, dK, 5, dims, str, box, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, CU_TENSOR_MAP_SWIZZLE_128B);
}

// Tensor map over the window queries [units, rows, d] (contiguous bf16): box = 64 features x 128 rows.
// Rows beyond `rows` read as zero.
cudaError_t make_query_tensor_map(CUtensorMap *map, const void *dQw, int units, int rows) {
    uint64_t dims[3] = {(uint64_t)kD, (uint64_t)rows, (uint64_t)units};
    uint64_t str[2] = {(uint64_t)kD * 2, (uint64_t)rows * kD * 2};
    uint32_t box[3] = {64, 128, 1};
    return encode_tensor_map(map, dQw, 3, dims, str, box, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, CU_TENSOR_MAP_SWIZZLE_128B);
}

cudaError_t cached_scorer_maps(TmapCache *cache, const Plan &p, const UnitAddr &addr, const void *dQw, const void *dK,
                               int tile_tokens, CUtensorMap *tq, CUtensorMap *tk) {
    TmapCache local;
    if (!cache) { cache = &local; cache->k_valid = cache->q_valid = false; }
    const bool same_k = cache->k_valid && cache->k_base == dK && cache->k_addr.sB == addr.sB &&
                        cache->k_addr.sL == addr.sL && cache->k_addr.sH == addr.sH && cache->k_addr.sN == addr.sN;
    if (!same_k) {
        cache->k_valid = false;
        cudaError_t e = make_key_tensor_map(&cache->k_map, p.shape, addr, dK, tile_tokens);
        if (e != cudaSuccess) return e;
        cache->k_base = dK;
        cache->k_addr = addr;
        cache->k_valid = true;
    }
    if (!(cache->q_valid && cache->q_base == dQw)) {
        cache->q_valid = false;
        cudaError_t e = make_query_tensor_map(&cache->q_map, dQw, p.units, p.rows);
        if (e != cudaSuccess) return e;
        cache->q_base = dQw;
        cache->q_valid = true;
    }
    *tq = cache->q_map;
    *tk = cache->k_map;
    return cudaSuccess;
}

}  // namespace uncomp
