// Prefill selection of the dynamic neurons (Section 5): with the activations of all loaded
// neurons at hand for every prompt token, keep each token's top alpha, count how often every
// neuron occurs over the prompt's tokens, take the beta most frequent as the dynamic candidates
// and combine them with the static neurons until phi neurons are chosen.
//
// Everything is built from the radix selector (one CTA per score row, ties to the lower index):
//   1. T rows of activations          -> T lists of alpha indices
//   2. histogram of the lists          -> counts[n]
//   3. select top beta of counts       -> candidates (count descending, slot ascending)
//   4. candidates that are not static and occur at least once keep their count as score, all
//      other slots get -1; select the top (phi - static) of these scores; drop the -1 entries
//   5. output = static prefix 0 .. n_static-1, then the kept candidates (ascending)
// All decisions are integer comparisons on counts or on the selector's order-preserving keys, so
// the result is exact and unique.
#include "si_common.cuh"

namespace {

struct VoteLayout {
    size_t lists, counts, score_a, score_b, cand_a, cand_b, selws, total;
};

VoteLayout vote_layout(int T, int n, int alpha) {
    VoteLayout L;
    size_t off = 0;
    auto take = [&](size_t &o, size_t bytes) { o = off; off += si_align_up(bytes, 256); };
    take(L.lists, (size_t)T * (alpha > 0 ? alpha : 1) * 4);
    take(L.counts, (size_t)n * 4);
    take(L.score_a, (size_t)n * 4);
    take(L.score_b, (size_t)n * 4);
    take(L.cand_a, (size_t)n * 4);
    take(L.cand_b, (size_t)n * 4);
    take(L.selws, (size_t)(T > 1 ? T : 1) * si_select_ws_bytes_impl(n));
    L.total = off;
    return L;
}

__global__ void vote_histogram_kernel(const int32_t *__restrict__ lists, long long n_entries, int n, int *counts) {
    for (long long e = (long long)blockIdx.x * blockDim.x + threadIdx.x; e < n_entries; e += (long long)gridDim.x * blockDim.x) {
        const int i = lists[e];
        if (i >= 0 && i < n) atomicAdd(&counts[i], 1);
    }
}

// score_a[i] = count as a float (exact below 2^24 tokens); score_b[i] = -1
__global__ void vote_scores_kernel(const int *__restrict__ counts, int n, float *score_a, float *score_b) {
    const int i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i < n) { score_a[i] = (float)counts[i]; score_b[i] = -1.f; }
}

// candidates outside the static prefix that occur in at least one list keep their count as score
__global__ void vote_mark_kernel(const int32_t *__restrict__ cand, int n_cand, const int *__restrict__ counts, int n_static,
                                 float *score_b) {
    const int j = blockIdx.x * blockDim.x + threadIdx.x;
    if (j >= n_cand) return;
    const int i = cand[j];
    if (i >= n_static && counts[i] > 0) score_b[i] = (float)counts[i];
}

// out = 0 .. n_static-1, then the entries of cand (ascending) whose score_b is positive.  One block.
__global__ void __launch_bounds__(1024)
vote_assemble_kernel(const int32_t *__restrict__ cand, int n_cand, const float *__restrict__ score_b, int n_static,
                     int32_t *__restrict__ out, int cap, int32_t *__restrict__ n_out) {
    __shared__ int warp_tot[32];
    __shared__ int carry_s;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    for (int i = tid; i < n_static && i < cap; i += 1024) out[i] = i;
    if (tid == 0) carry_s = 0;
    __syncthreads();
    for (int base = 0; base < n_cand; base += 1024) {
        const int carry = carry_s;              // kept entries before this block of candidates
        const int j = base + tid;
        const int i = j < n_cand ? cand[j] : -1;
        const int keep = (i >= 0 && score_b[i] > 0.f) ? 1 : 0;
        int inc = keep;
        for (int o = 1; o < 32; o <<= 1) { const int t = __shfl_up_sync(0xFFFFFFFFu, inc, o); if (lane >= o) inc += t; }
        if (lane == 31) warp_tot[warp] = inc;
        __syncthreads();
        if (warp == 0) {
            const int v = warp_tot[lane];
            int vi = v;
            for (int o = 1; o < 32; o <<= 1) { const int t = __shfl_up_sync(0xFFFFFFFFu, vi, o); if (lane >= o) vi += t; }
            warp_tot[lane] = vi - v;
            if (lane == 31) carry_s = carry + vi;
        }
        __syncthreads();
        if (keep) {
            const int pos = n_static + carry + warp_tot[warp] + inc - 1;
            if (pos < cap) out[pos] = i;
        }
        __syncthreads();
    }
    if (tid == 0 && n_out) *n_out = n_static + carry_s;
}

}  // namespace

size_t si_prefill_vote_ws_bytes_impl(int T, int n, int alpha) { return vote_layout(T, n, alpha).total; }

// the register selector takes the rows as they are (any score type) and counts while it selects
bool si_prefill_vote_fused_ok(int n, int alpha) { return alpha > 0 && alpha < n && n <= 32 * 1024; }

int si_prefill_vote_launch(const void *acts, int acts_dtype, int T, int n, int row_stride, int alpha, int beta, int n_static,
                           int phi_count, unsigned flags, int32_t *idx_out, int cap, int32_t *n_out,
                           int32_t *counts_out, void *workspace, size_t ws_bytes, cudaStream_t stream) {
    const VoteLayout L = vote_layout(T, n, alpha);
    if (ws_bytes < L.total) return SI_ERR_NOMEM;
    char *w = (char *)workspace;
    int32_t *lists = (int32_t *)(w + L.lists);
    int *counts = (int *)(w + L.counts);
    float *score_a = (float *)(w + L.score_a), *score_b = (float *)(w + L.score_b);
    int32_t *cand_a = (int32_t *)(w + L.cand_a), *cand_b = (int32_t *)(w + L.cand_b);
    const int st = n_static < phi_count ? n_static : phi_count;       // static neurons that are chosen
    const int m = phi_count - st;                                     // dynamic neurons wanted

    SI_CUDA_TRY(cudaMemsetAsync(counts, 0, (size_t)n * 4, stream));
    if (alpha > 0 && T > 0) {
        // steps 1 and 2 in one launch where the rows fit the register selector: every selected slot adds
        // one to its count; otherwise lists first, then their histogram (fp32 rows only)
        int rc = si_select_vote_launch(acts, acts_dtype, T, n, row_stride, alpha, flags & SI_FLAG_SCORE_ABS, counts, stream);
        if (rc == SI_ERR_UNSUPPORTED) {
            if (acts_dtype != SI_F32) return SI_ERR_UNSUPPORTED;
            rc = si_select_launch((const float *)acts, T, n, row_stride, SI_SELECT_TOPK, alpha, 0.f, flags & SI_FLAG_SCORE_ABS,
                                  lists, alpha, alpha, nullptr, w + L.selws, (size_t)T * si_select_ws_bytes_impl(n), stream);
            if (rc) return rc;
            const long long entries = (long long)T * alpha;
            const int blocks = (int)((entries + 255) / 256 < 1184 ? (entries + 255) / 256 : 1184);
            vote_histogram_kernel<<<blocks, 256, 0, stream>>>(lists, entries, n, counts);
        } else if (rc) {
            return rc;
        }
    }
    if (counts_out) SI_CUDA_TRY(cudaMemcpyAsync(counts_out, counts, (size_t)n * 4, cudaMemcpyDeviceToDevice, stream));
    vote_scores_kernel<<<(n + 255) / 256, 256, 0, stream>>>(counts, n, score_a, score_b);
    int n_dyn = 0;
    if (beta > 0 && m > 0) {
        int rc = si_select_launch(score_a, 1, n, n, SI_SELECT_TOPK, beta, 0.f, 0, cand_a, beta, beta, nullptr,
                                  w + L.selws, si_select_ws_bytes_impl(n), stream);
        if (rc) return rc;
        vote_mark_kernel<<<(beta + 255) / 256, 256, 0, stream>>>(cand_a, beta, counts, st, score_b);
        n_dyn = m < beta ? m : beta;
        rc = si_select_launch(score_b, 1, n, n, SI_SELECT_TOPK, n_dyn, 0.f, 0, cand_b, n_dyn, n_dyn, nullptr,
                              w + L.selws, si_select_ws_bytes_impl(n), stream);
        if (rc) return rc;
    }
    vote_assemble_kernel<<<1, 1024, 0, stream>>>(cand_b, n_dyn, score_b, st, idx_out, cap, n_out);
    SI_CUDA_TRY(cudaGetLastError());
    return SI_OK;
}

extern "C" int si_prefill_vote_workspace_bytes(int T, int n, int alpha, size_t *bytes_out) {
    if (T < 0 || n < 0 || alpha < 0 || !bytes_out) return SI_ERR_INVALID_ARG;
    *bytes_out = si_prefill_vote_ws_bytes_impl(T, n, alpha);
    return SI_OK;
}

extern "C" int si_prefill_vote(const float *acts, int T, int n, int row_stride, int alpha, int beta, int n_static,
                               int phi_count, unsigned flags, int32_t *idx_out, int cap, int32_t *n_out,
                               int32_t *counts_out, void *workspace, size_t ws_bytes, void *stream) {
    if (!acts || !idx_out || !workspace || T < 0 || n <= 0 || row_stride < n) return SI_ERR_INVALID_ARG;
    if (alpha < 0 || alpha > n || beta < 0 || beta > n || n_static < 0 || n_static > n || phi_count < 0 || phi_count > n)
        return SI_ERR_INVALID_ARG;
    if (cap < phi_count) return SI_ERR_NOMEM;
    if (!si_aligned16(acts) || !si_aligned16(idx_out) || (((uintptr_t)workspace) & 255u)) return SI_ERR_ALIGNMENT;
    return si_prefill_vote_launch(acts, SI_F32, T, n, row_stride, alpha, beta, n_static, phi_count, flags, idx_out, cap,
                                  n_out, counts_out, workspace, ws_bytes, (cudaStream_t)stream);
}
