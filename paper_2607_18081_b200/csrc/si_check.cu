// Device-side validation of active lists (SI_FLAG_CHECK): list offsets that start at or above 0,
// never decrease and describe lists of at most k_fixed entries; every entry in [0, n_loaded) and
// no entry twice.  One CTA per list marks a shared-memory bitmap; a bit seen twice is a
// duplicate.  Only an error code is written; nothing else is touched.
#include "si_common.cuh"

namespace {

struct CheckParams {
    int n_loaded[128];
    int n_layers;
    int layer_fixed;               // >= 0: every list belongs to this layer
    const int32_t *step_layers;    // device, or nullptr: list l belongs to layer l mod n_layers
};

__global__ void __launch_bounds__(256)
si_check_lists_kernel(const __grid_constant__ CheckParams P, const int32_t *__restrict__ idx,
                      const int32_t *__restrict__ offsets, int k_fixed, int32_t *status, int min_slot) {
    extern __shared__ unsigned int bitmap[];
    const int list = blockIdx.x;
    int layer = P.layer_fixed >= 0 ? P.layer_fixed
                                   : (P.step_layers ? P.step_layers[list] : list % P.n_layers);
    if (layer < 0 || layer >= P.n_layers) { if (threadIdx.x == 0) atomicCAS(status, 0, SI_ERR_OUT_OF_RANGE); return; }
    const int n_loaded = P.n_loaded[layer];
    const int words = (n_loaded + 31) / 32;
    for (int w = threadIdx.x; w < words; w += blockDim.x) bitmap[w] = 0u;
    __syncthreads();
    int base = offsets ? offsets[list] : list * k_fixed;
    int k = offsets ? offsets[list + 1] - base : k_fixed;
    if (offsets && (base < 0 || k < 0 || k > k_fixed)) {     // a malformed offsets array: report, read no entry
        if (threadIdx.x == 0) atomicCAS(status, 0, SI_ERR_OUT_OF_RANGE);
        return;
    }
    for (int p = threadIdx.x; p < k; p += blockDim.x) {
        int s = idx[base + p];
        if (s < 0 || s >= n_loaded) { atomicCAS(status, 0, SI_ERR_OUT_OF_RANGE); continue; }
        if (s < min_slot) { atomicCAS(status, 0, SI_ERR_DUPLICATE); continue; }     // a slot of the static prefix, which the step computes anyway
        unsigned int bit = 1u << (s & 31);
        unsigned int old = atomicOr(&bitmap[s >> 5], bit);
        if (old & bit) atomicCAS(status, 0, SI_ERR_DUPLICATE);
    }
}

}  // namespace

int si_check_lists_launch_impl(const si_store *s, int n_lists, int layer_fixed, const int32_t *step_layers_dev,
                               const int32_t *idx, const int32_t *idx_offsets, int k_fixed,
                               int32_t *status_dev, cudaStream_t stream, int min_slot) {
    if (!status_dev || n_lists <= 0) return SI_OK;
    if (s->n_layers > 128) return SI_ERR_UNSUPPORTED;
    CheckParams P;
    int max_loaded = 0;
    for (int l = 0; l < s->n_layers; ++l) { P.n_loaded[l] = s->n_loaded[l]; max_loaded = max_loaded > s->n_loaded[l] ? max_loaded : s->n_loaded[l]; }
    P.n_layers = s->n_layers; P.layer_fixed = layer_fixed; P.step_layers = step_layers_dev;
    size_t smem = (size_t)((max_loaded + 31) / 32 + 1) * 4;
    if (smem > 48 * 1024) return SI_ERR_UNSUPPORTED;
    si_check_lists_kernel<<<n_lists, 256, smem, stream>>>(P, idx, idx_offsets, k_fixed, status_dev, min_slot);
    SI_CUDA_TRY(cudaGetLastError());
    return SI_OK;
}
