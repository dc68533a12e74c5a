/*
 * selectinfer_debug.h -- diagnostics of libselectinfer: entry points for tests and measurements.
 *
 * Nothing here is part of the method (the paper has no counterpart to any of it) and nothing here
 * keeps state between calls: every knob is an argument of the call it applies to.
 */
#ifndef SELECTINFER_DEBUG_H
#define SELECTINFER_DEBUG_H

#include "selectinfer.h"

#ifdef __cplusplus
extern "C" {
#endif

/* Options of one persistent decode launch.  All zero = normal operation. */
typedef struct si_debug_decode_opts {
    int skip_mask;         /* bit 0: leave out the arithmetic; bit 1: the loads of the cross-SM sum; bit 2: the
                              cross-SM exchange altogether.  y is then meaningless; timing such a launch gives
                              the practical ceiling of the record stream on the same lists.  Bit 3: ring stages
                              are handed to the consumers without their record being copied; bit 4 (chained
                              calls in the split form): the down slices are not copied -- with both set a
                              chained launch reads no weights at all and its time is what the exchanges and
                              the arithmetic of the dependent steps cost by themselves. */
    int ring_stages;       /* ring stages per consumer set (0 = as many as fit); results stay correct */
    int step_groups;       /* step groups the SMs are split into, whatever the flags say (0 = the library's
                              choice: one, or up to four with SI_FLAG_STEPS_ANY_ORDER); results stay correct */
    int withhold;          /* 1: the producer warp of the first CTA never issues the second item of its first
                              ring, so that CTA's consumers wait for a record that does not come: with a short
                              wait_cycles this exercises the time-out path (status SI_ERR_TIMEOUT, grid-wide
                              abort, clean return).  Nothing faults and no wait is unbounded. */
    int chain_form;        /* si_debug_decode_chain_forward: 0 = the library's choice; 1 = the SMs exchange partial
                              output rows; 2 = the split form that exchanges the activations (SI_ERR_UNSUPPORTED where
                              it does not apply); results agree up to fp32 summation order */
    long long wait_cycles; /* limit of every device-side wait in clock cycles (0 = the default, about 2 s) */
    void *profile;         /* device int64 [num_SMs][16] or NULL: per-SM cycle counts of the phases.  Slots 0..5:
                              first consumer set (wait for x, wait for a record + copy to registers, record
                              arithmetic, accumulator hand-over, wait for the hand-over buffer, dot products +
                              exchange); 6..7: second set (wait for the hand-over buffer, wait for a record);
                              8..13: first reducer warp (idle, wait for a free partial-ring slot, copy
                              accumulators out, publish, wait for all SMs, reduce + write y).
                              Chained launches: slots 0..7 first consumer set, 8..15 second set.  Form 1:
                              wait for the input row, normalisation + records, wait for the second set / park
                              the accumulators, store the CTA's row, wait for every CTA's row, gather the rows,
                              wait for the class sums, column sums + y + next input row.  Form 2 (split): 0 input
                              row, 1 records, 4 gather h, 5 wait for all h and the slices, 6 partial sums,
                              7 final sums + y + next input row. */
} si_debug_decode_opts_t;

/* si_decode_stack_forward with the options above (opts == NULL: identical to it). */
int si_debug_decode_stack_forward(const si_store_t *store, int n_steps, const int32_t *layers,
                                  const void *x, const int32_t *idx, const int32_t *idx_offsets,
                                  int k_fixed, void *y, int y_dtype, unsigned flags, void *workspace,
                                  size_t ws_bytes, int32_t *status_dev, void *stream,
                                  const si_debug_decode_opts_t *opts);

/* si_decode_chain_forward with the options above (step_groups is ignored: a chain has one). */
int si_debug_decode_chain_forward(const si_store_t *store, int n_steps, const int32_t *layers, int chain_len,
                                  const void *x, const int32_t *idx, const int32_t *idx_offsets, int k_fixed,
                                  void *y, void *xn_out, float norm_eps, unsigned flags, void *workspace,
                                  size_t ws_bytes, int32_t *status_dev, void *stream,
                                  const si_debug_decode_opts_t *opts);

/* One launch that reads `bytes` bytes (a multiple of 16) at the 16-byte-aligned device pointer `mem`
 * once with plain 16-byte loads, all SMs busy, and stores a checksum of them in *checksum_dev (device
 * uint32).  Timing it on the neuron store gives the read bandwidth a kernel with no other work reaches
 * on this GPU, the practical ceiling quoted beside the decode kernel. */
int si_debug_read_bandwidth(const void *mem, size_t bytes, unsigned int *checksum_dev, void *stream);

/* The first stage of a multi-token si_ffn_forward call run on its own, with everything it leaves for
 * the contractions copied out: the ascending union (union_out device int32 [n_loaded], *n_union_out
 * device int32) and the tokens' slot bitmaps, which decide which union entries a token uses --
 * masks_out device uint32 [T][mask_words], bit (s & 31) of word s >> 5 of row t set iff slot s is in
 * list t; mask_words = ceil(n_loaded / 128) * 4.  Same kernels, same choice between them as in
 * si_ffn_forward.  workspace as for si_ffn_forward with the same T and k_fixed. */
int si_debug_union_masks(const si_store_t *store, int layer, int T, const int32_t *idx,
                         const int32_t *idx_offsets, int k_fixed, int32_t *union_out, int32_t *n_union_out,
                         uint32_t *masks_out, void *workspace, size_t ws_bytes, void *stream);

/* si_ffn_forward for T > 1 (union path) with a limit on the probes of every device-side wait of the two
 * contraction kernels (0 = the default) and, with withhold = 1, one operand tile of the first CTA of the
 * gate/up kernel never loaded: its tensor-core warp waits for a stage that is never filled, the wait
 * runs out, the kernel records SI_ERR_TIMEOUT in *status_dev, releases its tensor memory and returns. */
int si_debug_ffn_forward_waits(const si_store_t *store, int layer, const void *x, int T, const int32_t *idx,
                               const int32_t *idx_offsets, int k_fixed, void *y, int y_dtype, unsigned flags,
                               void *workspace, size_t ws_bytes, int32_t *status_dev, void *stream,
                               long long spin_limit, int withhold);

/* Host logic only (no device is touched): the kernel shapes si_ffn_forward picks for a call with T tokens (T > 128) whose
 * union has room for union_cap entries (a multiple of 128), on a device of num_sms SMs.
 *   out[0], out[1] : gate/up tiles: neurons per sub-tile (128, 112 or 96) and sub-tiles per tile (1 or 2)
 *   out[2]         : CTA pairs of the gate/up launch
 *   out[3], out[4] : down tiles: output columns per pair tile (128 or 256) and pairs that share a tile, each with a
 *                    part of K (1 or 2)
 *   out[5]         : CTAs of the down launch
 * SI_ERR_INVALID_ARG for T <= 128, d_model not a multiple of 128, union_cap not a positive multiple of 128. */
int si_debug_pair_plan(int d_model, int union_cap, int T, int num_sms, int out[6]);

/* si_ffn_forward_sharded for the ranks rank_base .. rank_base + n_here - 1 of a group that share this GPU, in ONE
 * launch (kernels of different ranks that wait on one another may not run as separate launches on one GPU): the
 * ranks' first kernels one after the other, then one cooperative launch of the finishing kernel over all of them.
 * All arrays are HOST arrays of n_here entries (stores, x, idx, k, y, workspaces) or of `world` entries (recv,
 * marks).  With n_here < world the missing ranks never deliver: with a short wait_cycles (0 = the default)
 * this exercises the time-out (SI_ERR_TIMEOUT in *status_dev, clean return). */
int si_debug_ffn_forward_sharded_group(const si_store_t *const *stores, int n_here, int rank_base, int world, int layer,
                                       const void *const *x, const int32_t *const *idx, const int *k, void *const *y,
                                       int y_dtype, unsigned flags, float *const *recv, unsigned *const *marks,
                                       unsigned epoch, void *const *workspaces, size_t ws_bytes, long long wait_cycles,
                                       int32_t *status_dev, void *stream);

#ifdef __cplusplus
}
#endif
#endif /* SELECTINFER_DEBUG_H */
