// Multi-token path (T > 1): union of the active lists + gathered tensor-core contraction.
#include "si_common.cuh"

size_t si_gemm_partial_bytes(const si_store *s, int T_max) { (void)s; (void)T_max; return 0; }

int si_multi_token_launch(const si_store *s, int layer, const void *x, int T, const int32_t *idx,
                          const int32_t *idx_offsets, int k_fixed, void *y, int y_dtype,
                          unsigned flags, void *workspace, size_t ws_bytes, int32_t *status_dev,
                          cudaStream_t stream) {
    return SI_ERR_UNSUPPORTED;
}

int si_union_launch(const si_store *s, int layer, int T, const int32_t *idx, const int32_t *idx_offsets,
                    int k_fixed, int32_t *union_out, int32_t *n_union_out, void *workspace, size_t ws_bytes,
                    cudaStream_t stream) {
    return SI_ERR_UNSUPPORTED;
}
