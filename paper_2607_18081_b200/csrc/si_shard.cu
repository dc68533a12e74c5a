// Neuron shards over several devices (Section 5: the layer output is a sum over the selected
// neurons, so partial outputs of disjoint neuron shares add up to it).
//
//   si_shard_lists   per list: keep the entries s with s mod world == rank as s div world, order kept,
//                    lists packed back to back with offsets.  Two kernels: count per list (the block
//                    that finishes last turns the counts into offsets), then an ordered compaction.
//   si_shard_reduce  y = (x +) sum of the devices' fp32 partial outputs in rank order.
#include "si_common.cuh"

namespace {

__device__ __forceinline__ void list_range(const int32_t *offsets, int k_fixed, int t, int &base, int &len) {
    base = offsets ? offsets[t] : t * k_fixed;
    len = offsets ? offsets[t + 1] - base : k_fixed;
}

// counts[t] = entries of list t owned by `rank`; the last block writes offsets_out[0 .. n_lists]
__global__ void __launch_bounds__(256)
shard_count_kernel(const int32_t *__restrict__ idx, const int32_t *__restrict__ offsets, int k_fixed, int n_lists, int rank,
                   int world, int32_t *counts, unsigned *ticket, int32_t *__restrict__ offsets_out, int32_t *status) {
    __shared__ int warp_tot[8];
    __shared__ int carry_s, is_last;
    const int t = blockIdx.x, tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    int base, len;
    list_range(offsets, k_fixed, t, base, len);
    int c = 0;
    for (int e = tid; e < len; e += 256) {
        const int s = idx[base + e];
        if (s < 0) { if (status) atomicCAS(status, 0, SI_ERR_OUT_OF_RANGE); continue; }
        c += (s % world == rank) ? 1 : 0;
    }
    for (int o = 16; o > 0; o >>= 1) c += __shfl_xor_sync(0xFFFFFFFFu, c, o);
    if (lane == 0) warp_tot[warp] = c;
    __syncthreads();
    if (tid == 0) {
        int tot = 0;
        for (int w = 0; w < 8; ++w) tot += warp_tot[w];
        counts[t] = tot;
        __threadfence();
        is_last = atomicAdd(ticket, 1u) == gridDim.x - 1;
    }
    __syncthreads();
    if (!is_last) return;
    __threadfence();
    // exclusive prefix sum of counts -> offsets_out, 256 lists per round
    if (tid == 0) carry_s = 0;
    __syncthreads();
    for (int b0 = 0; b0 < n_lists; b0 += 256) {
        const int carry = carry_s;
        const int v = b0 + tid < n_lists ? __ldcg(counts + b0 + tid) : 0;
        int inc = v;
        for (int o = 1; o < 32; o <<= 1) { const int u = __shfl_up_sync(0xFFFFFFFFu, inc, o); if (lane >= o) inc += u; }
        if (lane == 31) warp_tot[warp] = inc;
        __syncthreads();
        int wbase = 0;
        for (int w = 0; w < warp; ++w) wbase += warp_tot[w];
        if (b0 + tid < n_lists) offsets_out[b0 + tid] = carry + wbase + inc - v;
        __syncthreads();
        if (tid == 255) carry_s = carry + wbase + inc;
        __syncthreads();
    }
    if (tid == 0) offsets_out[n_lists] = carry_s;
}

// list t: owned entries, renumbered, written in order from offsets_out[t]
__global__ void __launch_bounds__(256)
shard_compact_kernel(const int32_t *__restrict__ idx, const int32_t *__restrict__ offsets, int k_fixed, int rank, int world,
                     const int32_t *__restrict__ offsets_out, int32_t *__restrict__ idx_out) {
    __shared__ int warp_tot[8];
    __shared__ int carry_s;
    const int t = blockIdx.x, tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    int base, len;
    list_range(offsets, k_fixed, t, base, len);
    int32_t *out = idx_out + offsets_out[t];
    if (tid == 0) carry_s = 0;
    __syncthreads();
    for (int e0 = 0; e0 < len; e0 += 256) {
        const int carry = carry_s;
        const int e = e0 + tid;
        const int s = e < len ? idx[base + e] : -1;
        const int keep = (s >= 0 && s % world == rank) ? 1 : 0;
        int inc = keep;
        for (int o = 1; o < 32; o <<= 1) { const int u = __shfl_up_sync(0xFFFFFFFFu, inc, o); if (lane >= o) inc += u; }
        if (lane == 31) warp_tot[warp] = inc;
        __syncthreads();
        int wbase = 0;
        for (int w = 0; w < warp; ++w) wbase += warp_tot[w];
        if (keep) out[carry + wbase + inc - 1] = s / world;
        __syncthreads();
        if (tid == 255) carry_s = carry + wbase + inc;
        __syncthreads();
    }
}

template <int DT>
__global__ void shard_reduce_kernel(const float *const *__restrict__ parts, int world, const uint16_t *__restrict__ x,
                                    long long n4, void *__restrict__ y, int y_f32, int residual) {
    const long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x;      // one float4 group
    if (i >= n4) return;
    float4 a = make_float4(0.f, 0.f, 0.f, 0.f);
    for (int r0 = 0; r0 < world; r0 += 8) {                                     // up to 8 loads in flight, added in rank order
        float4 v[8];
#pragma unroll
        for (int j = 0; j < 8; ++j)
            v[j] = r0 + j < world ? __ldcg(reinterpret_cast<const float4 *>(parts[r0 + j]) + i) : make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
        for (int j = 0; j < 8; ++j) { a.x += v[j].x; a.y += v[j].y; a.z += v[j].z; a.w += v[j].w; }
    }
    if (residual) {
        const uint2 xw = *reinterpret_cast<const uint2 *>(x + 4 * i);
        a.x += si_cvt<DT>::lo(xw.x); a.y += si_cvt<DT>::hi(xw.x); a.z += si_cvt<DT>::lo(xw.y); a.w += si_cvt<DT>::hi(xw.y);
    }
    if (y_f32) {
        reinterpret_cast<float4 *>(y)[i] = a;
    } else {
        uint2 w;
        w.x = (uint32_t)si_cvt<DT>::from_float(a.x) | ((uint32_t)si_cvt<DT>::from_float(a.y) << 16);
        w.y = (uint32_t)si_cvt<DT>::from_float(a.z) | ((uint32_t)si_cvt<DT>::from_float(a.w) << 16);
        reinterpret_cast<uint2 *>(y)[i] = w;
    }
}

}  // namespace

extern "C" int si_shard_count(int n, int rank, int world, int *count_out) {
    if (n < 0 || world <= 0 || rank < 0 || rank >= world || !count_out) return SI_ERR_INVALID_ARG;
    *count_out = n > rank ? (n - rank + world - 1) / world : 0;
    return SI_OK;
}

extern "C" int si_shard_lists(const int32_t *idx, const int32_t *idx_offsets, int k_fixed, int n_lists, int rank, int world,
                              int32_t *idx_out, int32_t *offsets_out, void *workspace, size_t ws_bytes,
                              int32_t *status_dev, void *stream_) {
    if (!idx_out || !offsets_out || !workspace || n_lists < 0 || k_fixed < 0) return SI_ERR_INVALID_ARG;
    if (world <= 0 || rank < 0 || rank >= world) return SI_ERR_INVALID_ARG;
    if (!idx && (idx_offsets || (long long)n_lists * k_fixed > 0)) return SI_ERR_INVALID_ARG;
    if (ws_bytes < ((size_t)n_lists + 64) * 4) return SI_ERR_NOMEM;
    if (!si_aligned16(workspace) || (((uintptr_t)offsets_out | (uintptr_t)idx_out) & 3u)) return SI_ERR_ALIGNMENT;
    cudaStream_t stream = (cudaStream_t)stream_;
    if (n_lists == 0) {
        SI_CUDA_TRY(cudaMemsetAsync(offsets_out, 0, 4, stream));
        return SI_OK;
    }
    unsigned *ticket = (unsigned *)workspace;
    int32_t *counts = (int32_t *)workspace + 64;
    SI_CUDA_TRY(cudaMemsetAsync(ticket, 0, 256, stream));
    shard_count_kernel<<<n_lists, 256, 0, stream>>>(idx, idx_offsets, k_fixed, n_lists, rank, world, counts, ticket,
                                                    offsets_out, status_dev);
    shard_compact_kernel<<<n_lists, 256, 0, stream>>>(idx, idx_offsets, k_fixed, rank, world, offsets_out, idx_out);
    SI_CUDA_TRY(cudaGetLastError());
    return SI_OK;
}

extern "C" int si_shard_reduce(const float *const *parts_dev, int world, const void *x, int x_dtype, int T, int d_model,
                               void *y, int y_dtype, unsigned flags, void *stream_) {
    if (!parts_dev || !y || world <= 0 || T < 0 || d_model <= 0 || d_model % 4 != 0) return SI_ERR_INVALID_ARG;
    if (x_dtype != SI_F16 && x_dtype != SI_BF16) return SI_ERR_INVALID_ARG;
    if (y_dtype != SI_F32 && y_dtype != x_dtype) return SI_ERR_INVALID_ARG;
    const bool residual = (flags & SI_FLAG_RESIDUAL) != 0;
    if (residual && !x) return SI_ERR_INVALID_ARG;
    if (!si_aligned16(y) || (x && !si_aligned16(x)) || (((uintptr_t)parts_dev) & 7u)) return SI_ERR_ALIGNMENT;
    const long long n4 = (long long)T * d_model / 4;
    if (n4 == 0) return SI_OK;
    const int blocks = (int)((n4 + 255) / 256);
    cudaStream_t stream = (cudaStream_t)stream_;
    if (x_dtype == SI_BF16)
        shard_reduce_kernel<SI_BF16><<<blocks, 256, 0, stream>>>(parts_dev, world, (const uint16_t *)x, n4, y, y_dtype == SI_F32, residual);
    else
        shard_reduce_kernel<SI_F16><<<blocks, 256, 0, stream>>>(parts_dev, world, (const uint16_t *)x, n4, y, y_dtype == SI_F32, residual);
    SI_CUDA_TRY(cudaGetLastError());
    return SI_OK;
}
