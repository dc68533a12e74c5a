// Neuron store: layout, handle, and the selective loader (Section 4, "Selective Loading").
//
// HBM layout per layer (all 16-bit elements in the store dtype):
//   records  : n_loaded x [ gate row (d_model) | up row (d_model) | W_down[:, id] (d_model) ]
//              one contiguous, 256-byte aligned record per loaded neuron (slot), so a
//              selected neuron is a single 6*d_model-byte burst for the decode kernel and
//              three rows of a [3*n_loaded, d_model] matrix for the tensor-core path.
//   slot_to_global int32 [n_loaded], global_to_slot int32 [d_ff] (-1 = not loaded).
#include <algorithm>
#include <new>

#include "si_common.cuh"

namespace {

struct Offsets {
    std::vector<size_t> rec, s2g, g2s;
    size_t total;
};

bool compute_offsets(int n_layers, int d_model, int d_ff, const int *n_loaded, Offsets &o) {
    o.rec.resize(n_layers); o.s2g.resize(n_layers); o.g2s.resize(n_layers);
    size_t off = 0;
    for (int l = 0; l < n_layers; ++l) {
        if (n_loaded[l] < 0 || n_loaded[l] > d_ff) return false;
        o.rec[l] = off;
        off = si_align_up(off + (size_t)n_loaded[l] * 3 * d_model * 2, 256);
    }
    for (int l = 0; l < n_layers; ++l) {
        o.s2g[l] = off; off = si_align_up(off + (size_t)n_loaded[l] * 4, 256);
        o.g2s[l] = off; off = si_align_up(off + (size_t)d_ff * 4, 256);
    }
    o.total = off;
    return true;
}

bool shape_ok(int n_layers, int d_model, int d_ff, int dtype) {
    return n_layers > 0 && d_model > 0 && d_model % 64 == 0 && d_model <= 16384 && d_ff > 0 &&
           (dtype == SI_F16 || dtype == SI_BF16);
}

// gate and up rows: one CTA per (slot, matrix); 16-byte copies.
__global__ void si_pack_rows_kernel(const uint4 *__restrict__ w_gate, const uint4 *__restrict__ w_up,
                                    const int32_t *__restrict__ ids, int n_loaded, int chunks,
                                    uint4 *__restrict__ records) {
    int s = blockIdx.x, which = blockIdx.y;
    if (s >= n_loaded) return;
    const uint4 *src = (which == 0 ? w_gate : w_up) + (size_t)ids[s] * chunks;
    uint4 *dst = records + ((size_t)s * 3 + which) * chunks;
    for (int c = threadIdx.x; c < chunks; c += blockDim.x) dst[c] = __ldg(src + c);
}

// down columns: 64 (model dims j) x 64 (slots) tiles transposed through shared memory,
// so that the strided column reads become 128-byte contiguous record writes.
__global__ void __launch_bounds__(256)
si_pack_down_kernel(const uint16_t *__restrict__ w_down, const int32_t *__restrict__ ids,
                    int n_loaded, int d_model, int d_ff, uint16_t *__restrict__ records) {
    __shared__ uint16_t tile[64][64 + 2];      // [slot][j]
    __shared__ int32_t tile_ids[64];
    int s0 = blockIdx.x * 64, j0 = blockIdx.y * 64;
    if (threadIdx.x < 64) {
        int s = s0 + threadIdx.x;
        tile_ids[threadIdx.x] = s < n_loaded ? ids[s] : -1;
    }
    __syncthreads();
    for (int e = threadIdx.x; e < 64 * 64; e += 256) {
        int jj = e >> 6, ss = e & 63;
        int id = tile_ids[ss];
        tile[ss][jj] = id >= 0 ? w_down[(size_t)(j0 + jj) * d_ff + id] : (uint16_t)0;
    }
    __syncthreads();
    for (int e = threadIdx.x; e < 64 * 8; e += 256) {    // 64 slots x 8 chunks of 8 values
        int ss = e >> 3, c = e & 7;
        int s = s0 + ss;
        if (s >= n_loaded) continue;
        uint32_t w[4];
#pragma unroll
        for (int q = 0; q < 4; ++q)
            w[q] = (uint32_t)tile[ss][c * 8 + 2 * q] | ((uint32_t)tile[ss][c * 8 + 2 * q + 1] << 16);
        uint4 v = make_uint4(w[0], w[1], w[2], w[3]);
        *reinterpret_cast<uint4 *>(records + ((size_t)s * 3 + 2) * d_model + j0 + c * 8) = v;
    }
}

__global__ void si_build_maps_kernel(const int32_t *__restrict__ ids, int n_loaded,
                                     int32_t *__restrict__ g2s, int d_ff, int phase) {
    int i = blockIdx.x * blockDim.x + threadIdx.x;
    if (phase == 0) { if (i < d_ff) g2s[i] = -1; }
    else            { if (i < n_loaded) g2s[ids[i]] = i; }
}

}  // namespace

extern "C" const char *si_strerror(int status) {
    switch (status) {
        case SI_OK: return "ok";
        case SI_ERR_INVALID_ARG: return "invalid argument";
        case SI_ERR_OUT_OF_RANGE: return "index out of range";
        case SI_ERR_DUPLICATE: return "duplicate index";
        case SI_ERR_ALIGNMENT: return "pointer not 16-byte aligned";
        case SI_ERR_NOMEM: return "caller-supplied buffer too small";
        case SI_ERR_CUDA: return "CUDA runtime error";
        case SI_ERR_TIMEOUT: return "bounded device-side wait expired";
        case SI_ERR_UNSUPPORTED: return "unsupported configuration";
        case SI_ERR_TOO_LARGE: return "size exceeds a fixed built-in limit";
        default: return "unknown status";
    }
}

int &si_last_cuda_error_code() {
    static thread_local int code = 0;
    return code;
}

extern "C" const char *si_last_cuda_error(void) {
    return cudaGetErrorString((cudaError_t)si_last_cuda_error_code());
}

extern "C" const char *si_build_info(void) {
    return "libselectinfer sm_100a (persistent TMA decode, tcgen05 gathered GEMM, radix select)";
}

extern "C" int si_store_bytes(int n_layers, int d_model, int d_ff, const int *n_loaded, int dtype,
                              size_t *bytes_out) {
    if (!n_loaded || !bytes_out || !shape_ok(n_layers, d_model, d_ff, dtype)) return SI_ERR_INVALID_ARG;
    Offsets o;
    if (!compute_offsets(n_layers, d_model, d_ff, n_loaded, o)) return SI_ERR_INVALID_ARG;
    *bytes_out = o.total;
    return SI_OK;
}

extern "C" int si_store_create(si_store_t **store_out, void *store_mem, size_t store_mem_bytes,
                               int n_layers, int d_model, int d_ff, const int *n_loaded, int dtype) {
    if (!store_out || !store_mem || !n_loaded || !shape_ok(n_layers, d_model, d_ff, dtype))
        return SI_ERR_INVALID_ARG;
    if (((uintptr_t)store_mem) & 255u) return SI_ERR_ALIGNMENT;
    Offsets o;
    if (!compute_offsets(n_layers, d_model, d_ff, n_loaded, o)) return SI_ERR_INVALID_ARG;
    if (store_mem_bytes < o.total) return SI_ERR_NOMEM;
    int dev = 0, sms = 0;
    SI_CUDA_TRY(cudaGetDevice(&dev));
    SI_CUDA_TRY(cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev));
    si_store *s = new (std::nothrow) si_store();
    if (!s) return SI_ERR_NOMEM;
    s->magic = SI_MAGIC; s->device = dev; s->num_sms = sms > 0 ? sms : SI_NUM_SMS_FALLBACK;
    s->n_layers = n_layers; s->d_model = d_model; s->d_ff = d_ff; s->dtype = dtype;
    s->mem = (char *)store_mem; s->mem_bytes = store_mem_bytes;
    s->n_loaded.assign(n_loaded, n_loaded + n_layers);
    s->n_base.assign(n_layers, 0);
    s->loaded.assign(n_layers, 0);
    s->rec_off = o.rec; s->s2g_off = o.s2g; s->g2s_off = o.g2s;
    *store_out = s;
    return SI_OK;
}

extern "C" int si_store_free(si_store_t *store) {
    if (!si_store_ok(store)) return SI_ERR_INVALID_ARG;
    cudaError_t e = cudaDeviceSynchronize();
    store->magic = 0;
    delete store;
    return e == cudaSuccess ? SI_OK : SI_ERR_CUDA;
}

extern "C" int si_load_neurons(si_store_t *store, int layer, const void *w_gate, const void *w_up,
                               const void *w_down, const int32_t *neuron_ids, int n_loaded,
                               int n_base, void *stream_) {
    if (!si_store_ok(store) || !w_gate || !w_up || !w_down) return SI_ERR_INVALID_ARG;
    if (layer < 0 || layer >= store->n_layers) return SI_ERR_INVALID_ARG;
    if (n_loaded != store->n_loaded[layer] || n_base < 0 || n_base > n_loaded) return SI_ERR_INVALID_ARG;
    if (n_loaded > 0 && !neuron_ids) return SI_ERR_INVALID_ARG;
    if (!si_aligned16(w_gate) || !si_aligned16(w_up) || !si_aligned16(w_down)) return SI_ERR_ALIGNMENT;
    if (int rc = si_check_device(store)) return rc;
    const int d = store->d_model, F = store->d_ff;
    {   // host-side validation of the neuron file: in range, distinct
        std::vector<char> seen((size_t)F, 0);
        for (int s = 0; s < n_loaded; ++s) {
            int id = neuron_ids[s];
            if (id < 0 || id >= F) return SI_ERR_OUT_OF_RANGE;
            if (seen[id]) return SI_ERR_DUPLICATE;
            seen[id] = 1;
        }
    }
    cudaStream_t stream = (cudaStream_t)stream_;
    int32_t *s2g = store->s2g(layer), *g2s = store->g2s(layer);
    uint16_t *rec = const_cast<uint16_t *>(store->records(layer));
    store->n_base[layer] = n_base;
    if (n_loaded > 0) {
        // ids are read by the copy engine before this call returns only if the source is
        // pageable memory; to be safe for pinned sources too, stage through a private copy
        // that outlives the enqueue by synchronising the copy (the loader is not a hot path).
        SI_CUDA_TRY(cudaMemcpyAsync(s2g, neuron_ids, (size_t)n_loaded * 4, cudaMemcpyHostToDevice, stream));
        SI_CUDA_TRY(cudaStreamSynchronize(stream));
    }
    si_build_maps_kernel<<<(F + 255) / 256, 256, 0, stream>>>(s2g, n_loaded, g2s, F, 0);
    if (n_loaded > 0) {
        si_build_maps_kernel<<<(n_loaded + 255) / 256, 256, 0, stream>>>(s2g, n_loaded, g2s, F, 1);
        dim3 grid_rows(n_loaded, 2);
        si_pack_rows_kernel<<<grid_rows, 128, 0, stream>>>((const uint4 *)w_gate, (const uint4 *)w_up, s2g,
                                                           n_loaded, d / 8, (uint4 *)rec);
        dim3 grid_down((n_loaded + 63) / 64, d / 64);
        si_pack_down_kernel<<<grid_down, 256, 0, stream>>>((const uint16_t *)w_down, s2g, n_loaded, d, F, rec);
    }
    SI_CUDA_TRY(cudaGetLastError());
    store->loaded[layer] = 1;
    return SI_OK;
}

extern "C" int si_store_slot_to_global(const si_store_t *store, int layer, const int32_t **dev_ptr_out,
                                       int *n_loaded_out, int *n_base_out) {
    if (!si_store_ok(store) || layer < 0 || layer >= store->n_layers) return SI_ERR_INVALID_ARG;
    if (dev_ptr_out) *dev_ptr_out = store->s2g(layer);
    if (n_loaded_out) *n_loaded_out = store->n_loaded[layer];
    if (n_base_out) *n_base_out = store->n_base[layer];
    return SI_OK;
}

extern "C" int si_store_global_to_slot(const si_store_t *store, int layer, const int32_t **dev_ptr_out) {
    if (!si_store_ok(store) || layer < 0 || layer >= store->n_layers || !dev_ptr_out) return SI_ERR_INVALID_ARG;
    *dev_ptr_out = store->g2s(layer);
    return SI_OK;
}

extern "C" int si_store_records(const si_store_t *store, int layer, const void **dev_ptr_out,
                                size_t *record_bytes_out) {
    if (!si_store_ok(store) || layer < 0 || layer >= store->n_layers) return SI_ERR_INVALID_ARG;
    if (dev_ptr_out) *dev_ptr_out = store->records(layer);
    if (record_bytes_out) *record_bytes_out = store->record_bytes();
    return SI_OK;
}

extern "C" int si_layer_range(int n_layers, int first, int last, int *first_out, int *last_out) {
    if (!first_out || !last_out || n_layers <= 0 || first < 0 || last > 0) return SI_ERR_INVALID_ARG;
    const int end = n_layers + last;          // one past the last selective layer
    if (first >= end || end > n_layers) return SI_ERR_INVALID_ARG;
    *first_out = first;
    *last_out = end;
    return SI_OK;
}

// ---------------------------------------------------------------------------------------------
// Diagnostics: read-only streaming kernel (bandwidth ceiling of plain loads).
namespace {
__global__ void __launch_bounds__(512)
si_read_bandwidth_kernel(const uint4 *__restrict__ p, size_t n16, unsigned int *checksum) {
    const size_t stride = (size_t)gridDim.x * blockDim.x;
    size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
    unsigned int acc = 0;
    // eight independent 16-byte loads per thread and round
    for (; i + 7 * stride < n16; i += 8 * stride) {
        uint4 v[8];
#pragma unroll
        for (int j = 0; j < 8; ++j) v[j] = __ldcs(p + i + j * stride);
#pragma unroll
        for (int j = 0; j < 8; ++j) acc ^= v[j].x ^ v[j].y ^ v[j].z ^ v[j].w;
    }
    for (; i < n16; i += stride) { const uint4 v = __ldcs(p + i); acc ^= v.x ^ v.y ^ v.z ^ v.w; }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) acc ^= __shfl_xor_sync(0xFFFFFFFFu, acc, o);
    if ((threadIdx.x & 31) == 0 && acc != 0) atomicXor(checksum, acc);
}
}  // namespace

extern "C" int si_debug_read_bandwidth(const void *mem, size_t bytes, unsigned int *checksum_dev, void *stream) {
    if (!mem || !checksum_dev || (bytes & 15) || (((uintptr_t)mem) & 15)) return SI_ERR_INVALID_ARG;
    int dev = 0, sms = 0;
    SI_CUDA_TRY(cudaGetDevice(&dev));
    SI_CUDA_TRY(cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev));
    SI_CUDA_TRY(cudaMemsetAsync(checksum_dev, 0, 4, (cudaStream_t)stream));
    si_read_bandwidth_kernel<<<sms * 4, 512, 0, (cudaStream_t)stream>>>((const uint4 *)mem, bytes / 16, checksum_dev);
    SI_CUDA_TRY(cudaGetLastError());
    return SI_OK;
}
