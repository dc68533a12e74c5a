// Entry points that tie the steps together: workspace carving, si_ffn_forward,
// si_layer_forward (selection + FFN), si_decode_stack_forward, si_union.
#include "si_common.cuh"
#include "si_decode_persistent.cuh"
#include "selectinfer_debug.h"
#include "si_tc.cuh"

si_ws_layout si_ws_carve(const si_store *s, int T_max, int k_max, int max_steps) {
    si_ws_layout w;
    if (T_max < 1) T_max = 1;
    if (k_max < 0) k_max = 0;
    if (max_steps < 1) max_steps = 1;
    int nl_max = 0;
    for (int l = 0; l < s->n_layers; ++l) nl_max = nl_max > s->n_loaded[l] ? nl_max : s->n_loaded[l];
    const size_t nl_pad = si_align_up((size_t)nl_max, 128);
    // tokens are padded to 16; beyond 128 they run in token tiles of 128 or 256, padded to whole tiles
    const size_t t_pad = T_max <= 128 ? si_align_up((size_t)T_max, 16) : si_align_up((size_t)T_max, 256);
    size_t off = 0;
    auto take = [&](size_t &o, size_t &b, size_t bytes) { o = off; b = si_align_up(bytes, 256); off += b; };
    take(w.ctrl_off, w.ctrl_bytes, 256);
    size_t part = si_persistent_partial_bytes(s);   // >= the per-step kernels' [2 * SMs][d_model]
    size_t gpart = si_gemm_partial_bytes(s, T_max);
    take(w.partial_off, w.partial_bytes, part > gpart ? part : gpart);
    take(w.sel_off, w.sel_bytes, (size_t)T_max * (size_t)(k_max + 1) * 4);
    // the union stage's outputs exist twice (w.half_* bytes each): the union of a call is built while the contractions
    // of the call before it still read theirs
    w.union_half = T_max > 1 ? si_align_up(nl_pad * 4 + 256, 256) : 0;
    w.mask_half = T_max > 1 ? si_align_up((t_pad + 1) * (nl_pad / 32) * 4 + si_gemm_counter_bytes(s, nl_pad, t_pad), 256) : 0;
    take(w.union_off, w.union_bytes, 2 * w.union_half);   // union, count
    take(w.mask_off, w.mask_bytes, 2 * w.mask_half);      // token slot bitmaps, union bitmap, counters
    take(w.h_off, w.h_bytes, T_max > 1 ? t_pad * nl_pad * 2 : 0);
    take(w.selws_off, w.selws_bytes, (size_t)T_max * si_select_ws_bytes_impl(nl_max));
    take(w.steps_off, w.steps_bytes, si_align_up((size_t)max_steps * 4, 256) + 256 + (size_t)max_steps * 256);   // layer ids, control words, 2 counter lines per step
    w.total = off;
    return w;
}

extern "C" int si_workspace_bytes(const si_store_t *store, int T_max, int k_max, int max_steps,
                                  size_t *bytes_out) {
    if (!si_store_ok(store) || !bytes_out || T_max < 1 || k_max < 0 || max_steps < 1) return SI_ERR_INVALID_ARG;
    *bytes_out = si_ws_carve(store, T_max, k_max, max_steps).total;
    return SI_OK;
}

static int check_common(const si_store *s, const void *x, const void *y, int y_dtype, const void *workspace,
                        const int32_t *status_dev) {
    if (!si_store_ok(s) || !x || !y || !workspace) return SI_ERR_INVALID_ARG;
    if (y_dtype != SI_F32 && y_dtype != s->dtype) return SI_ERR_INVALID_ARG;
    if (!si_aligned16(x) || !si_aligned16(y) || (((uintptr_t)workspace) & 255u)) return SI_ERR_ALIGNMENT;
    if (status_dev && (((uintptr_t)status_dev) & 3u)) return SI_ERR_ALIGNMENT;
    return si_check_device(s);
}

extern "C" int si_ffn_forward(const si_store_t *store, int layer, const void *x, int T, const int32_t *idx,
                              const int32_t *idx_offsets, int k_fixed, void *y, int y_dtype, unsigned flags,
                              void *workspace, size_t ws_bytes, int32_t *status_dev, void *stream_) {
    int rc = check_common(store, x, y, y_dtype, workspace, status_dev);
    if (rc) return rc;
    if (layer < 0 || layer >= store->n_layers || T <= 0 || k_fixed < 0) return SI_ERR_INVALID_ARG;
    if (!store->loaded[layer]) return SI_ERR_INVALID_ARG;
    if (k_fixed > store->n_loaded[layer]) return SI_ERR_OUT_OF_RANGE;
    if (k_fixed > 0 && !idx) return SI_ERR_INVALID_ARG;
    if (idx && !si_aligned16(idx)) return SI_ERR_ALIGNMENT;
    cudaStream_t stream = (cudaStream_t)stream_;
    if (ws_bytes < si_ws_carve(store, T, k_fixed, 1).total) return SI_ERR_NOMEM;
    if (flags & SI_FLAG_CHECK) {
        rc = si_check_lists_launch_impl(store, (flags & SI_FLAG_SHARED_LIST) ? 1 : T, layer, nullptr, idx, idx_offsets,
                                        k_fixed, status_dev, stream);
        if (rc) return rc;
    }
    if (T == 1 && !(flags & SI_FLAG_UNION_PATH)) {
        int32_t l = layer;
        return si_decode_launch(store, 1, &l, x, idx, idx_offsets, k_fixed, y, y_dtype, flags, workspace,
                                ws_bytes, status_dev, stream);
    }
    // (Taking a few tokens through the decode kernel one after the other was faster than the union path while that
    // path summed its K splits through global memory: 37.0 against 42.9 us at T = 4 on a 7B-shaped layer.  With the
    // cluster sums it is the other way round -- 31.3 against 37.0 us at T = 4, 25.5 against 27.6 at T = 2 -- so every
    // call with more than one token forms the union.)
    return si_multi_token_launch(store, layer, x, T, idx, idx_offsets, k_fixed, y, y_dtype, flags, workspace,
                                 ws_bytes, status_dev, stream);
}

extern "C" int si_layer_forward(const si_store_t *store, int layer, const void *x, int T, const float *scores,
                                int k, const int32_t *idx, const int32_t *idx_offsets, void *y, int y_dtype,
                                unsigned flags, void *workspace, size_t ws_bytes, int32_t *status_dev,
                                void *stream_) {
    if (!scores)
        return si_ffn_forward(store, layer, x, T, idx, idx_offsets, k, y, y_dtype, flags, workspace, ws_bytes,
                              status_dev, stream_);
    int rc = check_common(store, x, y, y_dtype, workspace, status_dev);
    if (rc) return rc;
    if (layer < 0 || layer >= store->n_layers || T <= 0 || k < 0) return SI_ERR_INVALID_ARG;
    if (!store->loaded[layer]) return SI_ERR_INVALID_ARG;      // before the selector is enqueued
    const int n = store->n_loaded[layer];
    if (k > n) return SI_ERR_OUT_OF_RANGE;
    if (!si_aligned16(scores)) return SI_ERR_ALIGNMENT;
    si_ws_layout ws = si_ws_carve(store, T, k, 1);
    if (ws_bytes < ws.total) return SI_ERR_NOMEM;
    cudaStream_t stream = (cudaStream_t)stream_;
    char *wsb = (char *)workspace;
    int32_t *lists = (int32_t *)(wsb + ws.sel_off);
    int32_t *counts = lists + (size_t)T * k;
    rc = si_select_launch(scores, T, n, n, SI_SELECT_TOPK, k, 0.f, flags, lists, k, k, counts,
                          wsb + ws.selws_off, ws.selws_bytes, stream);
    if (rc) return rc;
    return si_ffn_forward(store, layer, x, T, lists, nullptr, k, y, y_dtype, flags & ~SI_FLAG_CHECK, workspace,
                          ws_bytes, status_dev, stream_);
}

// si_decode_stack_forward and si_decode_chain_forward (ex->chain_len > 0) share their checks.
static int decode_stack_impl(const si_store_t *store, int n_steps, const int32_t *layers, const void *x,
                             const int32_t *idx, const int32_t *idx_offsets, int k_fixed, void *y, int y_dtype,
                             unsigned flags, void *workspace, size_t ws_bytes, int32_t *status_dev, void *stream_,
                             const si_decode_extra *ex) {
    int rc = check_common(store, x, y, y_dtype, workspace, status_dev);
    if (rc) return rc;
    if (n_steps <= 0 || k_fixed < 0) return SI_ERR_INVALID_ARG;
    if (k_fixed > 0 && !idx) return SI_ERR_INVALID_ARG;
    if (idx && !si_aligned16(idx)) return SI_ERR_ALIGNMENT;
    int min_loaded = store->d_ff;
    for (int st = 0; st < n_steps; ++st) {
        int l = layers ? layers[st] : st % store->n_layers;
        if (l < 0 || l >= store->n_layers) return SI_ERR_INVALID_ARG;
        if (!store->loaded[l]) return SI_ERR_INVALID_ARG;          // before anything is enqueued
        min_loaded = min_loaded < store->n_loaded[l] ? min_loaded : store->n_loaded[l];
    }
    const int n_static = ex ? ex->n_static : 0;
    if (n_static < 0 || n_static > min_loaded) return SI_ERR_OUT_OF_RANGE;
    if (!idx_offsets && k_fixed > min_loaded - n_static) return SI_ERR_OUT_OF_RANGE;
    if ((flags & SI_FLAG_LIST_PER_LAYER) && idx_offsets) return SI_ERR_INVALID_ARG;   // per-layer lists have one fixed length
    if (n_static > 0 && !si_persistent_supported(store)) return SI_ERR_UNSUPPORTED;
    if (ex && ex->chain_len > 0) {
        if (y_dtype != store->dtype) return SI_ERR_INVALID_ARG;    // a step's output is the next step's input
        if (!si_persistent_supported(store)) return SI_ERR_UNSUPPORTED;
        if (ex->xn_out && !si_aligned16(ex->xn_out)) return SI_ERR_ALIGNMENT;
        if (ex->prenorm && !(ex->norm_eps >= 0.f)) return SI_ERR_INVALID_ARG;
    }
    cudaStream_t stream = (cudaStream_t)stream_;
    si_ws_layout ws = si_ws_carve(store, 1, k_fixed, n_steps);
    if (ws_bytes < ws.total) return SI_ERR_NOMEM;
    if (flags & SI_FLAG_CHECK) {
        const int32_t *layers_dev = nullptr;
        if (layers) {
            int32_t *dst = (int32_t *)((char *)workspace + ws.steps_off);
            SI_CUDA_TRY(cudaMemcpyAsync(dst, layers, (size_t)n_steps * 4, cudaMemcpyHostToDevice, stream));
            layers_dev = dst;
        }
        if ((flags & SI_FLAG_LIST_PER_LAYER) && !idx_offsets) {     // one list per layer: check list l against layer l
            for (int l = 0; l < store->n_layers; ++l) {
                rc = si_check_lists_launch_impl(store, 1, l, nullptr, idx + (size_t)l * k_fixed, nullptr, k_fixed, status_dev, stream, n_static);
                if (rc) return rc;
            }
        } else {
            rc = si_check_lists_launch_impl(store, n_steps, -1, layers_dev, idx, idx_offsets, k_fixed, status_dev, stream, n_static);
            if (rc) return rc;
        }
    }
    return si_decode_launch(store, n_steps, layers, x, idx, idx_offsets, k_fixed, y, y_dtype, flags, workspace,
                            ws_bytes, status_dev, stream, ex);
}

static si_decode_extra extra_of(const si_debug_decode_opts_t *o) {
    si_decode_extra ex;
    if (o) {
        ex.skip_mask = o->skip_mask; ex.ring_stages = o->ring_stages; ex.step_groups = o->step_groups;
        ex.withhold = o->withhold; ex.wait_cycles = o->wait_cycles; ex.profile = (long long *)o->profile;
        ex.chain_form = o->chain_form;
    }
    return ex;
}

extern "C" int si_decode_stack_forward(const si_store_t *store, int n_steps, const int32_t *layers,
                                       const void *x, const int32_t *idx, const int32_t *idx_offsets,
                                       int k_fixed, void *y, int y_dtype, unsigned flags, void *workspace,
                                       size_t ws_bytes, int32_t *status_dev, void *stream) {
    return decode_stack_impl(store, n_steps, layers, x, idx, idx_offsets, k_fixed, y, y_dtype, flags, workspace, ws_bytes,
                             status_dev, stream, nullptr);
}

extern "C" int si_debug_decode_stack_forward(const si_store_t *store, int n_steps, const int32_t *layers,
                                             const void *x, const int32_t *idx, const int32_t *idx_offsets,
                                             int k_fixed, void *y, int y_dtype, unsigned flags, void *workspace,
                                             size_t ws_bytes, int32_t *status_dev, void *stream,
                                             const si_debug_decode_opts_t *opts) {
    if (opts && (opts->ring_stages < 0 || opts->step_groups < 0 || opts->wait_cycles < 0)) return SI_ERR_INVALID_ARG;
    const si_decode_extra ex = extra_of(opts);
    return decode_stack_impl(store, n_steps, layers, x, idx, idx_offsets, k_fixed, y, y_dtype, flags, workspace, ws_bytes,
                             status_dev, stream, &ex);
}

static int chain_impl(const si_store_t *store, int n_steps, const int32_t *layers, int chain_len, const void *x,
                      const int32_t *idx, const int32_t *idx_offsets, int k_fixed, void *y, void *xn_out,
                      float norm_eps, unsigned flags, void *workspace, size_t ws_bytes, int32_t *status_dev,
                      void *stream, const si_debug_decode_opts_t *opts, int n_static = 0) {
    if (chain_len < 1 || !si_store_ok(store)) return SI_ERR_INVALID_ARG;
    if (flags & (SI_FLAG_STEPS_ANY_ORDER | SI_FLAG_SIMPLE_KERNELS)) return SI_ERR_INVALID_ARG;   // neither applies to a chain
    if (opts && (opts->ring_stages < 0 || opts->wait_cycles < 0)) return SI_ERR_INVALID_ARG;
    si_decode_extra ex = extra_of(opts);
    ex.step_groups = 0;
    ex.n_static = n_static;
    ex.chain_len = chain_len;
    ex.prenorm = (flags & SI_FLAG_PRENORM) != 0;
    ex.norm_eps = norm_eps;
    ex.xn_out = ex.prenorm ? xn_out : nullptr;
    return decode_stack_impl(store, n_steps, layers, x, idx, idx_offsets, k_fixed, y, store->dtype, flags, workspace,
                             ws_bytes, status_dev, stream, &ex);
}

extern "C" int si_decode_chain_forward(const si_store_t *store, int n_steps, const int32_t *layers, int chain_len,
                                       const void *x, const int32_t *idx, const int32_t *idx_offsets, int k_fixed,
                                       void *y, void *xn_out, float norm_eps, unsigned flags, void *workspace,
                                       size_t ws_bytes, int32_t *status_dev, void *stream) {
    return chain_impl(store, n_steps, layers, chain_len, x, idx, idx_offsets, k_fixed, y, xn_out, norm_eps, flags, workspace,
                      ws_bytes, status_dev, stream, nullptr);
}

extern "C" int si_debug_decode_chain_forward(const si_store_t *store, int n_steps, const int32_t *layers, int chain_len,
                                             const void *x, const int32_t *idx, const int32_t *idx_offsets, int k_fixed,
                                             void *y, void *xn_out, float norm_eps, unsigned flags, void *workspace,
                                             size_t ws_bytes, int32_t *status_dev, void *stream,
                                             const si_debug_decode_opts_t *opts) {
    return chain_impl(store, n_steps, layers, chain_len, x, idx, idx_offsets, k_fixed, y, xn_out, norm_eps, flags, workspace,
                      ws_bytes, status_dev, stream, opts);
}

extern "C" int si_decode_prefix_forward(const si_store_t *store, int n_steps, const int32_t *layers, int n_static, int chain_len,
                                        const void *x, const int32_t *idx, const int32_t *idx_offsets, int k_fixed,
                                        void *y, int y_dtype, void *xn_out, float norm_eps, unsigned flags, void *workspace,
                                        size_t ws_bytes, int32_t *status_dev, void *stream) {
    if (n_static < 0 || chain_len < 0) return SI_ERR_INVALID_ARG;
    if (chain_len > 0) {
        if (si_store_ok(store) && y_dtype != store->dtype) return SI_ERR_INVALID_ARG;
        return chain_impl(store, n_steps, layers, chain_len, x, idx, idx_offsets, k_fixed, y, xn_out, norm_eps, flags, workspace,
                          ws_bytes, status_dev, stream, nullptr, n_static);
    }
    if (flags & (SI_FLAG_PRENORM | SI_FLAG_SIMPLE_KERNELS)) return SI_ERR_INVALID_ARG;     // the norm belongs to chains; prefixes to the persistent kernel
    si_decode_extra ex;
    ex.n_static = n_static;
    return decode_stack_impl(store, n_steps, layers, x, idx, idx_offsets, k_fixed, y, y_dtype, flags, workspace, ws_bytes,
                             status_dev, stream, &ex);
}

extern "C" int si_debug_ffn_forward_waits(const si_store_t *store, int layer, const void *x, int T, const int32_t *idx,
                                          const int32_t *idx_offsets, int k_fixed, void *y, int y_dtype, unsigned flags,
                                          void *workspace, size_t ws_bytes, int32_t *status_dev, void *stream,
                                          long long spin_limit, int withhold) {
    int rc = check_common(store, x, y, y_dtype, workspace, status_dev);
    if (rc) return rc;
    if (layer < 0 || layer >= store->n_layers || T <= 1 || k_fixed <= 0 || spin_limit < 0) return SI_ERR_INVALID_ARG;
    if (!store->loaded[layer] || !idx) return SI_ERR_INVALID_ARG;
    if (k_fixed > store->n_loaded[layer]) return SI_ERR_OUT_OF_RANGE;
    if (!si_aligned16(idx)) return SI_ERR_ALIGNMENT;
    if (ws_bytes < si_ws_carve(store, T, k_fixed, 1).total) return SI_ERR_NOMEM;
    return si_multi_token_launch(store, layer, x, T, idx, idx_offsets, k_fixed, y, y_dtype, flags, workspace, ws_bytes,
                                 status_dev, (cudaStream_t)stream, spin_limit, withhold);
}

extern "C" int si_debug_pair_plan(int d_model, int union_cap, int T, int num_sms, int out[6]) {
    if (!out || T <= 128 || d_model <= 0 || d_model % 128 != 0 || union_cap <= 0 || union_cap % 128 != 0 || num_sms < 2)
        return SI_ERR_INVALID_ARG;
    si_pair_plan_t plan;
    si_pair_plan(d_model, union_cap, T, num_sms, &plan);
    out[0] = plan.gateup_w; out[1] = plan.gateup_sub; out[2] = plan.gateup_pairs;
    out[3] = plan.down_n; out[4] = plan.down_ksplit; out[5] = plan.down_ctas;
    return SI_OK;
}

extern "C" int si_debug_union_masks(const si_store_t *store, int layer, int T, const int32_t *idx,
                                    const int32_t *idx_offsets, int k_fixed, int32_t *union_out, int32_t *n_union_out,
                                    uint32_t *masks_out, void *workspace, size_t ws_bytes, void *stream) {
    if (!si_store_ok(store) || layer < 0 || layer >= store->n_layers || T <= 0 || k_fixed < 0 || !union_out ||
        !n_union_out || !masks_out || !workspace)
        return SI_ERR_INVALID_ARG;
    if (k_fixed > 0 && !idx) return SI_ERR_INVALID_ARG;
    int rc = si_check_device(store);
    if (rc) return rc;
    return si_union_masks_launch(store, layer, T, idx, idx_offsets, k_fixed, union_out, n_union_out, masks_out, workspace,
                                 ws_bytes, (cudaStream_t)stream);
}

extern "C" int si_union(const si_store_t *store, int layer, int T, const int32_t *idx,
                        const int32_t *idx_offsets, int k_fixed, int32_t *union_out, int32_t *n_union_out,
                        void *workspace, size_t ws_bytes, void *stream) {
    if (!si_store_ok(store) || layer < 0 || layer >= store->n_layers || T <= 0 || k_fixed < 0 || !union_out ||
        !n_union_out || !workspace)
        return SI_ERR_INVALID_ARG;
    if (k_fixed > 0 && !idx) return SI_ERR_INVALID_ARG;
    if (int rc = si_check_device(store)) return rc;
    return si_union_launch(store, layer, T, idx, idx_offsets, k_fixed, union_out, n_union_out, workspace,
                           ws_bytes, (cudaStream_t)stream);
}

// ---------------------------------------------------------------------------------------------
// Prefill of one layer with the selection of the dynamic neurons (Section 5): the FFN over ALL loaded
// neurons for the prompt's T tokens, then the vote on the activations h = SiLU(g) * u that this very
// computation produced (H of the gathered contraction, in the store dtype).
namespace {
__global__ void si_iota_kernel(int32_t *out, int n) {
    const int i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i < n) out[i] = i;
}
template <int DT>
__global__ void si_widen_h_kernel(const uint16_t *__restrict__ h, int h_stride, int T, int n, float *__restrict__ acts) {
    const int i = blockIdx.x * blockDim.x + threadIdx.x, t = blockIdx.y;
    if (i < n && t < T) acts[(size_t)t * n + i] = si_cvt<DT>::lo((uint32_t)h[(size_t)t * h_stride + i]);
}
}  // namespace

extern "C" int si_prefill_forward(const si_store_t *store, int layer, const void *x, int T, void *y, int y_dtype,
                                  int alpha, int beta, int n_static, int phi_count, unsigned flags,
                                  int32_t *idx_out, int cap, int32_t *n_out, float *acts_out, void *workspace,
                                  size_t ws_bytes, void *vote_workspace, size_t vote_ws_bytes, int32_t *status_dev,
                                  void *stream_) {
    int rc = check_common(store, x, y, y_dtype, workspace, status_dev);
    if (rc) return rc;
    if (layer < 0 || layer >= store->n_layers || T <= 0 || !store->loaded[layer]) return SI_ERR_INVALID_ARG;
    const int n = store->n_loaded[layer];
    if (n <= 0 || !idx_out || !vote_workspace) return SI_ERR_INVALID_ARG;
    if (alpha < 0 || alpha > n || beta < 0 || beta > n || n_static < 0 || n_static > n || phi_count < 0 || phi_count > n)
        return SI_ERR_INVALID_ARG;
    if (cap < phi_count) return SI_ERR_NOMEM;
    if (!si_aligned16(idx_out) || (((uintptr_t)vote_workspace) & 255u) || (acts_out && !si_aligned16(acts_out)))
        return SI_ERR_ALIGNMENT;
    cudaStream_t stream = (cudaStream_t)stream_;
    const si_ws_layout ws = si_ws_carve(store, T < 2 ? 2 : T, n, 1);      // the multi-token regions exist from T_max = 2 on
    if (ws_bytes < ws.total) return SI_ERR_NOMEM;
    char *wsb = (char *)workspace;
    // one shared list: every loaded slot, so the union is the store in slot order (position p = slot p)
    int32_t *all = (int32_t *)(wsb + ws.sel_off);
    si_iota_kernel<<<(n + 255) / 256, 256, 0, stream>>>(all, n);
    rc = si_multi_token_launch(store, layer, x, T, all, nullptr, n, y, y_dtype,
                               (flags & SI_FLAG_RESIDUAL) | SI_FLAG_SHARED_LIST, workspace, ws_bytes, status_dev, stream);
    if (rc) return rc;
    const int h_stride = (int)si_align_up((size_t)n, 128);
    const uint16_t *h = (const uint16_t *)(wsb + ws.h_off);
    // The vote ranks the activations the contraction itself produced: H, in the store dtype.  Where the
    // register selector applies it reads H as it is (widening is exact, so the order is that of the fp32
    // values); fp32 copies are made only for a caller who asks for them, or for the general selector.
    const bool fused = si_prefill_vote_fused_ok(n, alpha);
    float *acts = acts_out;
    if (acts || !fused) {
        if (!acts) {
            if ((size_t)T * n * 4 > ws.partial_bytes) return SI_ERR_NOMEM;
            acts = (float *)(wsb + ws.partial_off);       // the partial-tile area is free again
        }
        dim3 grid((n + 255) / 256, T);
        if (store->dtype == SI_BF16) si_widen_h_kernel<SI_BF16><<<grid, 256, 0, stream>>>(h, h_stride, T, n, acts);
        else si_widen_h_kernel<SI_F16><<<grid, 256, 0, stream>>>(h, h_stride, T, n, acts);
        SI_CUDA_TRY(cudaGetLastError());
    }
    if (fused)
        return si_prefill_vote_launch(h, store->dtype, T, n, h_stride, alpha, beta, n_static, phi_count, flags, idx_out, cap,
                                      n_out, nullptr, vote_workspace, vote_ws_bytes, stream);
    return si_prefill_vote_launch(acts, SI_F32, T, n, n, alpha, beta, n_static, phi_count, flags, idx_out, cap, n_out, nullptr,
                                  vote_workspace, vote_ws_bytes, stream);
}
