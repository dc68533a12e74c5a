// Internal declarations shared by the translation units of libselectinfer.
#pragma once

#include <cuda_runtime.h>
#include <cuda_bf16.h>
#include <cuda_fp16.h>
#include <stdint.h>
#include <stddef.h>
#include <atomic>
#include <vector>

#include "selectinfer.h"

#define SI_MAGIC 0x53494E46u /* "SINF" */
#define SI_NUM_SMS_FALLBACK 148

struct si_store {
    uint32_t magic;
    int device;
    int n_layers, d_model, d_ff, dtype;
    int num_sms;
    char *mem;
    size_t mem_bytes;
    std::vector<int> n_loaded, n_base;
    std::vector<char> loaded;              // layer packed at least once
    std::vector<size_t> rec_off, s2g_off, g2s_off;
    // multi-token calls alternate between the two copies of the union stage's outputs (see si_ws_carve)
    mutable std::atomic<unsigned> mt_calls{0};
    size_t record_bytes() const { return (size_t)3 * d_model * 2; }
    const uint16_t *records(int l) const { return (const uint16_t *)(mem + rec_off[l]); }
    int32_t *s2g(int l) const { return (int32_t *)(mem + s2g_off[l]); }
    int32_t *g2s(int l) const { return (int32_t *)(mem + g2s_off[l]); }
};

static inline size_t si_align_up(size_t v, size_t a) { return (v + a - 1) / a * a; }
static inline bool si_aligned16(const void *p) { return (((uintptr_t)p) & 15u) == 0; }
static inline bool si_store_ok(const si_store *s) { return s && s->magic == SI_MAGIC; }
// A store's kernels, grid sizes and pointers belong to the device it was created on: that device has
// to be current in every call that launches work on it.
static inline int si_check_device(const si_store *s) {
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess) { (void)cudaGetLastError(); return SI_ERR_CUDA; }
    return dev == s->device ? SI_OK : SI_ERR_INVALID_ARG;
}

// last CUDA runtime error seen by this library on the calling thread (si_last_cuda_error)
int &si_last_cuda_error_code();

#define SI_CUDA_TRY(expr)                                   \
    do {                                                    \
        cudaError_t e__ = (expr);                           \
        if (e__ != cudaSuccess) {                           \
            si_last_cuda_error_code() = (int)e__;           \
            (void)cudaGetLastError();                       \
            return SI_ERR_CUDA;                             \
        }                                                   \
    } while (0)

// ---- workspace carving (all sizes 256-byte aligned) -------------------------------
// [0, 256)            : control words (barrier counters, tickets), zero on entry to every call
// then                : fp32 partial outputs [max_ctas][T][d_model] (decode: T = 1)
// then                : lists selected by si_layer_forward, union arrays, masks, H
struct si_ws_layout {
    size_t ctrl_off, ctrl_bytes;
    size_t partial_off, partial_bytes;
    size_t sel_off, sel_bytes;         // int32 [T_max][k_max] selected lists + [T_max] counts
    size_t union_off, union_bytes;     // 2 x (int32 [n_loaded_max] union + count)
    size_t mask_off, mask_bytes;       // 2 x (uint32 [T_max + 1][ceil(n_loaded_max / 32)] slot bitmaps, then counters)
    size_t union_half, mask_half;      // bytes of one of the two copies
    size_t h_off, h_bytes;             // 16-bit H [T_pad][n_loaded_max padded]
    size_t selws_off, selws_bytes;     // selector scratch
    size_t steps_off, steps_bytes;     // per-step descriptors for stack calls
    size_t total;
};
si_ws_layout si_ws_carve(const si_store *s, int T_max, int k_max, int max_steps);

// What a decode launch may carry beyond the arguments of si_decode_stack_forward: the chained mode of
// si_decode_chain_forward and the per-call diagnostics of si_debug_decode_stack_forward.
struct si_decode_extra {
    int n_static = 0;              // static prefix (persistent kernel only)
    int chain_len = 0;             // > 0: chained steps (persistent kernel only)
    int chain_form = 0;            // 0: the library's choice; 1: the SMs exchange partial output rows; 2: split form (activations)
    int prenorm = 0;
    float norm_eps = 0.f;
    void *xn_out = nullptr;
    int skip_mask = 0, ring_stages = 0, step_groups = 0, withhold = 0;
    long long wait_cycles = 0;     // 0: the default limit
    long long *profile = nullptr;
};

// implemented in si_decode.cu
int si_decode_launch(const si_store *s, int n_steps, const int32_t *layers_host, const void *x,
                     const int32_t *idx, const int32_t *idx_offsets, int k_fixed, void *y,
                     int y_dtype, unsigned flags, void *workspace, size_t ws_bytes,
                     int32_t *status_dev, cudaStream_t stream, const si_decode_extra *ex = nullptr);

int si_decode_partial_launch(const si_store *s, int layer, const void *x, const int32_t *idx, int k, float *partial,
                             int32_t *status_dev, cudaStream_t stream, int *rows_out);

// implemented in si_gemm.cu
int si_multi_token_launch(const si_store *s, int layer, const void *x, int T, const int32_t *idx,
                          const int32_t *idx_offsets, int k_fixed, void *y, int y_dtype,
                          unsigned flags, void *workspace, size_t ws_bytes, int32_t *status_dev,
                          cudaStream_t stream, long long spin_limit = 0, int withhold = 0);
int si_union_masks_launch(const si_store *s, int layer, int T, const int32_t *idx, const int32_t *idx_offsets,
                          int k_fixed, int32_t *union_out, int32_t *n_union_out, uint32_t *masks_out,
                          void *workspace, size_t ws_bytes, cudaStream_t stream);

// implemented in si_select.cu
size_t si_select_ws_bytes_impl(int n);
int si_select_launch(const float *scores, int n_rows, int n, int row_stride, int mode, int k,
                     float tau, unsigned flags, int32_t *idx_out, int out_stride, int cap,
                     int32_t *n_out, void *workspace, size_t ws_bytes, cudaStream_t stream);
// top-k of every row counted straight into counts[n]; scores of src_dtype (SI_F32 / SI_F16 / SI_BF16), row_stride
// in elements; SI_ERR_UNSUPPORTED when the rows do not fit the register kernel
int si_select_vote_launch(const void *scores, int src_dtype, int n_rows, int n, int row_stride, int k, unsigned flags,
                          int *counts, cudaStream_t stream);

// implemented in si_vote.cu
size_t si_prefill_vote_ws_bytes_impl(int T, int n, int alpha);
// acts: [T] rows of acts_dtype (SI_F32, or a 16-bit type where the register selector applies: see
// si_prefill_vote_fused_ok), row_stride in elements
bool si_prefill_vote_fused_ok(int n, int alpha);
int si_prefill_vote_launch(const void *acts, int acts_dtype, int T, int n, int row_stride, int alpha, int beta, int n_static,
                           int phi_count, unsigned flags, int32_t *idx_out, int cap, int32_t *n_out,
                           int32_t *counts_out, void *workspace, size_t ws_bytes, cudaStream_t stream);

// implemented in si_check.cu: device-side list validation for SI_FLAG_CHECK
int si_check_lists_launch_impl(const si_store *s, int n_lists, int layer_fixed,
                               const int32_t *step_layers_dev, const int32_t *idx,
                               const int32_t *idx_offsets, int k_fixed, int32_t *status_dev,
                               cudaStream_t stream, int min_slot = 0);

// implemented in si_gemm.cu
size_t si_gemm_partial_bytes(const si_store *s, int T_max);
size_t si_gemm_counter_bytes(const si_store *s, size_t nl_pad, size_t t_pad);
int si_union_launch(const si_store *s, int layer, int T, const int32_t *idx, const int32_t *idx_offsets,
                    int k_fixed, int32_t *union_out, int32_t *n_union_out, void *workspace,
                    size_t ws_bytes, cudaStream_t stream);

// ---- device helpers ---------------------------------------------------------------
template <int DT> struct si_cvt;
template <> struct si_cvt<SI_BF16> {
    // two bf16 packed in a 32-bit word -> two floats (exact)
    __device__ __forceinline__ static float lo(uint32_t w) { return __uint_as_float(w << 16); }
    __device__ __forceinline__ static float hi(uint32_t w) { return __uint_as_float(w & 0xFFFF0000u); }
    __device__ __forceinline__ static uint16_t from_float(float f) {
        return __bfloat16_as_ushort(__float2bfloat16_rn(f));
    }
};
template <> struct si_cvt<SI_F16> {
    __device__ __forceinline__ static float lo(uint32_t w) {
        return __half2float(__ushort_as_half((unsigned short)(w & 0xFFFFu)));
    }
    __device__ __forceinline__ static float hi(uint32_t w) {
        return __half2float(__ushort_as_half((unsigned short)(w >> 16)));
    }
    __device__ __forceinline__ static uint16_t from_float(float f) {
        return __half_as_ushort(__float2half_rn(f));
    }
};

__device__ __forceinline__ float si_silu_mul(float g, float u) {
    return __fdividef(g, 1.0f + __expf(-g)) * u;   // fast division: ~2 ulp, far inside the tolerance
}
