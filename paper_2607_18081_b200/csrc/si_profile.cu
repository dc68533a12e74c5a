// Offline profiler (Section 3) and the load set of selective loading (Section 4).
//
//   si_profile_accumulate  Eq. 1: s_n += sum over the tokens of |a_n(t)|, fp64 totals, tokens added in
//                          order (one thread per neuron), so the totals are bit-reproducible
//   si_profile_merge       merged_n += s_n / tokens: the score files are normalised by their token
//                          count and summed, in call order
//   si_profile_rank        neuron indices in decreasing order of score (ties: lower index; NaN last),
//                          by counting for every neuron how many neurons come before it
//   si_loadset             base neurons = the top n_base of the task ranking, then the model ranking
//                          in order, neurons already chosen skipped, until n_loaded neurons
// All of it is off the per-token path: it runs once per model and task.
#include "si_common.cuh"

namespace {

__global__ void profile_accumulate_kernel(const float *__restrict__ acts, int T, int n, int row_stride,
                                          double *__restrict__ scores) {
    const int i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= n) return;
    double s = scores[i];
    for (int t = 0; t < T; ++t) s += (double)fabsf(acts[(size_t)t * row_stride + i]);   // coalesced across neurons
    scores[i] = s;
}

__global__ void profile_merge_kernel(double *__restrict__ merged, const double *__restrict__ scores, double tokens, int n) {
    const int i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i < n) merged[i] += scores[i] / tokens;
}

// does neuron j come before neuron i?  decreasing score, NaN last, ties to the lower index
__device__ __forceinline__ bool before(double sj, int j, double si, int i) {
    const bool nj = sj != sj, ni = si != si;
    if (nj != ni) return ni;                   // a number comes before a NaN
    if (!nj && sj != si) return sj > si;
    return j < i;
}

// rank[i] = number of neurons that come before i; ranking[rank[i]] = i.  One block per 256 neurons, the
// scores are walked through shared memory in tiles.
__global__ void __launch_bounds__(256)
profile_rank_kernel(const double *__restrict__ scores, int n, int32_t *__restrict__ ranking) {
    __shared__ double tile[1024];
    const int i = blockIdx.x * 256 + threadIdx.x;
    const double si = i < n ? scores[i] : 0.0;
    int r = 0;
    for (int base = 0; base < n; base += 1024) {
        for (int j = threadIdx.x; j < 1024; j += 256) tile[j] = base + j < n ? scores[base + j] : 0.0;
        __syncthreads();
        const int m = n - base < 1024 ? n - base : 1024;
        if (i < n)
            for (int j = 0; j < m; ++j) r += before(tile[j], base + j, si, i) ? 1 : 0;
        __syncthreads();
    }
    if (i < n) ranking[r] = i;
}

// One block: mark the base neurons, then keep the model ranking's entries that are not marked, in
// order, until n_loaded neurons are chosen.  status: SI_ERR_OUT_OF_RANGE / SI_ERR_DUPLICATE / too short.
__global__ void __launch_bounds__(1024)
loadset_kernel(const int32_t *__restrict__ task_rank, const int32_t *__restrict__ model_rank, int n, int n_base,
               int n_loaded, int32_t *__restrict__ ids_out, uint32_t *__restrict__ chosen, int32_t *status) {
    __shared__ int warp_tot[32];
    __shared__ int carry_s;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int words = (n + 31) / 32;
    for (int w = tid; w < words; w += 1024) chosen[w] = 0u;
    __syncthreads();
    for (int j = tid; j < n_base; j += 1024) {
        const int v = task_rank[j];
        if (v < 0 || v >= n) { if (status) atomicCAS(status, 0, SI_ERR_OUT_OF_RANGE); continue; }
        const uint32_t old = atomicOr(&chosen[v >> 5], 1u << (v & 31));
        if (old & (1u << (v & 31))) { if (status) atomicCAS(status, 0, SI_ERR_DUPLICATE); }
        ids_out[j] = v;
    }
    if (tid == 0) carry_s = 0;
    __syncthreads();
    const int want = n_loaded - n_base;
    for (int base = 0; base < n; base += 1024) {
        const int carry = carry_s;
        if (carry >= want) break;                                    // uniform: read before the barrier below
        const int j = base + tid;
        int keep = 0, v = -1;
        if (j < n) {
            v = model_rank[j];
            if (v < 0 || v >= n) { if (status) atomicCAS(status, 0, SI_ERR_OUT_OF_RANGE); }
            else keep = (chosen[v >> 5] >> (v & 31)) & 1u ? 0 : 1;
        }
        int inc = keep;
        for (int o = 1; o < 32; o <<= 1) { const int t = __shfl_up_sync(0xFFFFFFFFu, inc, o); if (lane >= o) inc += t; }
        if (lane == 31) warp_tot[warp] = inc;
        __syncthreads();
        if (warp == 0) {
            const int x = warp_tot[lane];
            int xi = x;
            for (int o = 1; o < 32; o <<= 1) { const int t = __shfl_up_sync(0xFFFFFFFFu, xi, o); if (lane >= o) xi += t; }
            warp_tot[lane] = xi - x;
            if (lane == 31) carry_s = carry + xi;
        }
        __syncthreads();
        if (keep) {
            const int pos = carry + warp_tot[warp] + inc - 1;
            if (pos < want) ids_out[n_base + pos] = v;
        }
        __syncthreads();
    }
    if (tid == 0 && carry_s < want && status) atomicCAS(status, 0, SI_ERR_INVALID_ARG);   // rankings too short
}

}  // namespace

extern "C" int si_profile_accumulate(const float *acts, int T, int n, int row_stride, double *scores, void *stream) {
    if (!acts || !scores || T < 0 || n <= 0 || row_stride < n) return SI_ERR_INVALID_ARG;
    if (T == 0) return SI_OK;
    profile_accumulate_kernel<<<(n + 127) / 128, 128, 0, (cudaStream_t)stream>>>(acts, T, n, row_stride, scores);
    SI_CUDA_TRY(cudaGetLastError());
    return SI_OK;
}

extern "C" int si_profile_merge(double *merged, const double *scores, long long tokens, int n, void *stream) {
    if (!merged || !scores || tokens <= 0 || n <= 0) return SI_ERR_INVALID_ARG;
    profile_merge_kernel<<<(n + 255) / 256, 256, 0, (cudaStream_t)stream>>>(merged, scores, (double)tokens, n);
    SI_CUDA_TRY(cudaGetLastError());
    return SI_OK;
}

extern "C" int si_profile_rank(const double *scores, int n, int32_t *ranking, void *stream) {
    if (!scores || !ranking || n <= 0) return SI_ERR_INVALID_ARG;
    profile_rank_kernel<<<(n + 255) / 256, 256, 0, (cudaStream_t)stream>>>(scores, n, ranking);
    SI_CUDA_TRY(cudaGetLastError());
    return SI_OK;
}

extern "C" int si_loadset(const int32_t *task_rank, const int32_t *model_rank, int n, int n_base, int n_loaded,
                          int32_t *ids_out, void *workspace, size_t ws_bytes, int32_t *status_dev, void *stream) {
    if (!task_rank || !model_rank || !ids_out || !workspace || n <= 0) return SI_ERR_INVALID_ARG;
    if (n_base < 0 || n_base > n_loaded || n_loaded > n) return SI_ERR_INVALID_ARG;
    if (ws_bytes < (size_t)((n + 31) / 32) * 4) return SI_ERR_NOMEM;
    if (((uintptr_t)workspace) & 3u) return SI_ERR_ALIGNMENT;
    loadset_kernel<<<1, 1024, 0, (cudaStream_t)stream>>>(task_rank, model_rank, n, n_base, n_loaded, ids_out,
                                                        (uint32_t *)workspace, status_dev);
    SI_CUDA_TRY(cudaGetLastError());
    return SI_OK;
}
