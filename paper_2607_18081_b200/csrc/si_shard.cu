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

// ---------------------------------------------------------------------------------------------
// Batch-1 decode on a neuron shard with the all-reduce inside the kernel that finishes the down
// projection.  A block owns 32 output columns: it adds this device's partial rows for them (the cross-SM
// sum of the decode), stores the 32 sums into EVERY device's receive area with plain (peer) stores, marks
// the block as delivered on every device, waits -- with a limit -- until every device has delivered the
// same block here, adds the devices' sums in rank order, adds the residual, rounds and writes y.  No
// collective call, no second kernel; what crosses the links is world x d_model floats per device and step.
// The kernel handles the ranks rank_base + blockIdx.y: one rank per process in production (gridDim.y = 1);
// all ranks of an emulated group in one cooperative launch when they share a GPU (tests).
struct ShardRank {
    const float *partial;     // this rank's partial rows [rows][d_model]
    int rows;
    const uint16_t *x;        // residual input or nullptr
    void *y;
};
struct ShardExchange {
    ShardRank rk[8];          // by blockIdx.y
    float *recv[8];           // by rank: that device's receive area, fp32 [2][world][d_model]
    unsigned *flag[8];        // by rank: that device's delivery marks, uint32 [world][d_model / 32]
    int world, rank_base, d, y_f32, residual;
    unsigned epoch;           // this call's number (> 0, increasing): marks carry it, its parity picks the receive buffer
    long long wait_cycles;
    int32_t *status;
};

template <int DT>
__global__ void __launch_bounds__(256)
shard_reduce_exchange_kernel(const __grid_constant__ ShardExchange P) {
    __shared__ float4 part[8][8];
    __shared__ int timed_out;
    const ShardRank &R = P.rk[blockIdx.y];
    const int rank = P.rank_base + blockIdx.y, d = P.d, nblk = d / 32;
    const int g = threadIdx.x & 7, rc = threadIdx.x >> 3, warp = threadIdx.x >> 5;
    const int col = (blockIdx.x * 8 + g) * 4;
    // ---- this device's rows of the block's columns, in a fixed order (as in the unsharded reduce kernel)
    float4 a = make_float4(0.f, 0.f, 0.f, 0.f);
    for (int r0 = rc; r0 < R.rows; r0 += 32 * 5) {
        float4 v[5];
#pragma unroll
        for (int j = 0; j < 5; ++j) {
            const int r = r0 + 32 * j;
            v[j] = r < R.rows ? __ldg(reinterpret_cast<const float4 *>(R.partial + (size_t)r * d + col)) : make_float4(0.f, 0.f, 0.f, 0.f);
        }
#pragma unroll
        for (int j = 0; j < 5; ++j) { a.x += v[j].x; a.y += v[j].y; a.z += v[j].z; a.w += v[j].w; }
    }
#pragma unroll
    for (int o = 8; o <= 16; o <<= 1) {
        a.x += __shfl_xor_sync(0xFFFFFFFFu, a.x, o); a.y += __shfl_xor_sync(0xFFFFFFFFu, a.y, o);
        a.z += __shfl_xor_sync(0xFFFFFFFFu, a.z, o); a.w += __shfl_xor_sync(0xFFFFFFFFu, a.w, o);
    }
    if ((threadIdx.x & 31) < 8) part[warp][g] = a;
    if (threadIdx.x == 0) timed_out = 0;
    __syncthreads();
    const size_t buf = (size_t)(P.epoch & 1u) * P.world * d;
    if (threadIdx.x < 8) {
        a = part[0][g];
#pragma unroll
        for (int w = 1; w < 8; ++w) { const float4 v = part[w][g]; a.x += v.x; a.y += v.y; a.z += v.z; a.w += v.w; }
        // ---- deliver the block to every device (this one included), system-scope stores
        for (int q = 0; q < P.world; ++q) {
            float *dst = P.recv[q] + buf + (size_t)rank * d + col;
            asm volatile("st.relaxed.sys.global.v4.f32 [%0], {%1, %2, %3, %4};" ::"l"(dst), "f"(a.x), "f"(a.y), "f"(a.z), "f"(a.w) : "memory");
        }
    }
    __syncwarp();
    if (threadIdx.x == 0) {
        __threadfence_system();                              // the eight lanes' stores before the marks
        for (int q = 0; q < P.world; ++q) {
            unsigned *m = P.flag[q] + (size_t)rank * nblk + blockIdx.x;
            asm volatile("st.release.sys.global.u32 [%0], %1;" ::"l"(m), "r"(P.epoch) : "memory");
        }
        // ---- wait for the same block from every device (bounded)
        const unsigned *mine = P.flag[rank] + blockIdx.x;
        const long long t0 = clock64();
        for (int q = 0; q < P.world; ++q) {
            unsigned v;
            do {
                asm volatile("ld.acquire.sys.global.u32 %0, [%1];" : "=r"(v) : "l"(mine + (size_t)q * nblk) : "memory");
                if (v < P.epoch && clock64() - t0 > P.wait_cycles) { timed_out = 1; break; }
            } while (v < P.epoch);
            if (timed_out) break;
        }
        if (timed_out && P.status) atomicCAS(P.status, 0, SI_ERR_TIMEOUT);
    }
    __syncthreads();
    if (timed_out || threadIdx.x >= 8 || col >= d) return;
    // ---- the devices' sums in rank order
    const float *rb = P.recv[rank] + buf + col;
    float4 y4 = make_float4(0.f, 0.f, 0.f, 0.f);
    for (int q = 0; q < P.world; ++q) {
        float4 v;
        asm volatile("ld.relaxed.sys.global.v4.f32 {%0, %1, %2, %3}, [%4];" : "=f"(v.x), "=f"(v.y), "=f"(v.z), "=f"(v.w) : "l"(rb + (size_t)q * d) : "memory");
        y4.x += v.x; y4.y += v.y; y4.z += v.z; y4.w += v.w;
    }
    if (P.residual) {
        const uint2 xw = *reinterpret_cast<const uint2 *>(R.x + col);
        y4.x += si_cvt<DT>::lo(xw.x); y4.y += si_cvt<DT>::hi(xw.x); y4.z += si_cvt<DT>::lo(xw.y); y4.w += si_cvt<DT>::hi(xw.y);
    }
    if (P.y_f32) {
        *reinterpret_cast<float4 *>(reinterpret_cast<float *>(R.y) + col) = y4;
    } else {
        uint2 w;
        w.x = (uint32_t)si_cvt<DT>::from_float(y4.x) | ((uint32_t)si_cvt<DT>::from_float(y4.y) << 16);
        w.y = (uint32_t)si_cvt<DT>::from_float(y4.z) | ((uint32_t)si_cvt<DT>::from_float(y4.w) << 16);
        *reinterpret_cast<uint2 *>(reinterpret_cast<uint16_t *>(R.y) + col) = w;
    }
}

// ranks [rank_base, rank_base + n_here) of `world` are computed by this launch (n_here = 1 in production)
int shard_exchange_launch(const si_store *const *stores, int n_here, int rank_base, int world, int layer, const void *const *x,
                          const int32_t *const *idx, const int *k, void *const *y, int y_dtype, unsigned flags,
                          float *const *recv, unsigned *const *flag, unsigned epoch, float *const *partial, long long wait_cycles,
                          int32_t *status_dev, cudaStream_t stream) {
    ShardExchange P;
    const si_store *s0 = stores[0];
    P.world = world; P.rank_base = rank_base; P.d = s0->d_model; P.y_f32 = y_dtype == SI_F32;
    P.residual = (flags & SI_FLAG_RESIDUAL) != 0; P.epoch = epoch; P.status = status_dev;
    P.wait_cycles = wait_cycles > 0 ? wait_cycles : 4000000000ll;
    for (int q = 0; q < world; ++q) { P.recv[q] = recv[q]; P.flag[q] = flag[q]; }
    for (int i = 0; i < n_here; ++i) {
        int rows = 0;
        int rc = si_decode_partial_launch(stores[i], layer, x[i], idx[i], k[i], partial[i], status_dev, stream, &rows);
        if (rc) return rc;
        P.rk[i].partial = partial[i]; P.rk[i].rows = rows; P.rk[i].x = (const uint16_t *)x[i]; P.rk[i].y = y[i];
    }
    dim3 grid(P.d / 32, n_here), block(256);
    void *args[] = {(void *)&P};
    // blocks of several ranks in one launch wait for one another: they must all be resident (cooperative launch)
    if (s0->dtype == SI_BF16) {
        if (n_here > 1) SI_CUDA_TRY(cudaLaunchCooperativeKernel((void *)shard_reduce_exchange_kernel<SI_BF16>, grid, block, args, 0, stream));
        else shard_reduce_exchange_kernel<SI_BF16><<<grid, block, 0, stream>>>(P);
    } else {
        if (n_here > 1) SI_CUDA_TRY(cudaLaunchCooperativeKernel((void *)shard_reduce_exchange_kernel<SI_F16>, grid, block, args, 0, stream));
        else shard_reduce_exchange_kernel<SI_F16><<<grid, block, 0, stream>>>(P);
    }
    SI_CUDA_TRY(cudaGetLastError());
    return SI_OK;
}

}  // namespace

static int shard_fused_check(const si_store_t *store, int layer, const void *x, const int32_t *idx, int k, const void *y, int y_dtype) {
    if (!si_store_ok(store) || !x || !y) return SI_ERR_INVALID_ARG;
    if (y_dtype != SI_F32 && y_dtype != store->dtype) return SI_ERR_INVALID_ARG;
    if (layer < 0 || layer >= store->n_layers || k < 0 || !store->loaded[layer]) return SI_ERR_INVALID_ARG;
    if (k > store->n_loaded[layer]) return SI_ERR_OUT_OF_RANGE;
    if (k > 0 && !idx) return SI_ERR_INVALID_ARG;
    if (!si_aligned16(x) || !si_aligned16(y) || (idx && !si_aligned16(idx))) return SI_ERR_ALIGNMENT;
    if (store->d_model % 128 != 0 || store->d_model > 8192) return SI_ERR_UNSUPPORTED;
    return SI_OK;
}

extern "C" int si_ffn_forward_sharded(const si_store_t *store, int layer, const void *x, const int32_t *idx, int k, void *y,
                                      int y_dtype, unsigned flags, int rank, int world, float *const *recv, unsigned *const *marks,
                                      unsigned epoch, void *workspace, size_t ws_bytes, int32_t *status_dev, void *stream) {
    int rc = shard_fused_check(store, layer, x, idx, k, y, y_dtype);
    if (rc) return rc;
    if (world < 1 || world > 8 || rank < 0 || rank >= world || !recv || !marks || epoch == 0 || !workspace) return SI_ERR_INVALID_ARG;
    for (int q = 0; q < world; ++q) if (!recv[q] || !marks[q] || !si_aligned16(recv[q])) return SI_ERR_INVALID_ARG;
    if ((rc = si_check_device(store))) return rc;
    const si_ws_layout ws = si_ws_carve(store, 1, k, 1);
    if (ws_bytes < ws.total) return SI_ERR_NOMEM;
    float *partial = (float *)((char *)workspace + ws.partial_off);
    return shard_exchange_launch(&store, 1, rank, world, layer, &x, &idx, &k, &y, y_dtype, flags, recv, marks, epoch, &partial, 0,
                                 status_dev, (cudaStream_t)stream);
}

extern "C" int si_debug_ffn_forward_sharded_group(const si_store_t *const *stores, int n_here, int rank_base, int world, int layer,
                                                  const void *const *x, const int32_t *const *idx, const int *k, void *const *y,
                                                  int y_dtype, unsigned flags, float *const *recv, unsigned *const *marks,
                                                  unsigned epoch, void *const *workspaces, size_t ws_bytes, long long wait_cycles,
                                                  int32_t *status_dev, void *stream) {
    if (!stores || n_here < 1 || world < 1 || world > 8 || rank_base < 0 || rank_base + n_here > world || !x || !idx || !k || !y ||
        !recv || !marks || !workspaces || epoch == 0)
        return SI_ERR_INVALID_ARG;
    float *partial[8];
    for (int i = 0; i < n_here; ++i) {
        int rc = shard_fused_check(stores[i], layer, x[i], idx[i], k[i], y[i], y_dtype);
        if (rc) return rc;
        if (!workspaces[i] || stores[i]->d_model != stores[0]->d_model || stores[i]->dtype != stores[0]->dtype) return SI_ERR_INVALID_ARG;
        const si_ws_layout ws = si_ws_carve(stores[i], 1, k[i], 1);
        if (ws_bytes < ws.total) return SI_ERR_NOMEM;
        partial[i] = (float *)((char *)workspaces[i] + ws.partial_off);
    }
    for (int q = 0; q < world; ++q) if (!recv[q] || !marks[q]) return SI_ERR_INVALID_ARG;
    int rc = si_check_device(stores[0]);
    if (rc) return rc;
    return shard_exchange_launch(stores, n_here, rank_base, world, layer, x, idx, k, y, y_dtype, flags, recv, marks, epoch, partial,
                                 wait_cycles, status_dev, (cudaStream_t)stream);
}

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
