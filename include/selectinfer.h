/*
 * selectinfer.h -- C ABI of the B200 (sm_100a) selective-FFN library.
 *
 * The library implements the selective-computation hot path of SelectInfer: a
 * compacted store holding only the loaded FFN neurons (Section 4, "Selective
 * Loading"), the per-token SwiGLU FFN over only the selected loaded neurons
 * (Section 5, "Selective Computation"), and the per-token top-alpha index selection
 * used to pick them (Section 5, dynamic neuron selection).
 *
 * Neuron i of an FFN layer (Section 3): row i of gate_proj.weight and up_proj.weight
 * ([d_ff, d_model], PyTorch [out, in] storage) and column i of down_proj.weight
 * ([d_model, d_ff]).  Its activation is h_i = SiLU(w_gate_i . x) * (w_up_i . x) and
 * its contribution to the layer output is h_i * W_down[:, i].
 *
 * Conventions
 *   - Every function returns an int status: SI_OK (0) or a negative SI_ERR_* code.
 *     Nothing throws, aborts or prints.
 *   - "device" pointers are CUDA device pointers owned by the caller; "host" pointers
 *     are ordinary host memory.  The library allocates no device memory: the caller
 *     supplies the store bytes and the workspace (sizes via si_store_bytes /
 *     si_workspace_bytes).  The only thing the library owns is the small host-side
 *     si_store_t handle.
 *   - `stream` is a cudaStream_t passed as void*.  All work is enqueued on it and no
 *     call synchronises except si_store_free and si_load_neurons (which waits for the
 *     upload of its id list).  Calls sharing one workspace must be ordered on one stream.
 *   - Errors that can be seen on the host (null or misaligned pointers, sizes out of
 *     range, bad enum, layer out of range, buffers too small) are reported before
 *     anything is launched.  Errors only the device can see (an index out of range or
 *     a duplicate under SI_FLAG_CHECK, an expired bounded wait) are written to
 *     *status_dev (caller-owned int32 in device memory, may be NULL) as an SI_ERR_*
 *     code; the kernel then leaves y unspecified but never hangs, and slot indices never
 *     lead to an access outside the store.  CSR offsets (idx_offsets) are trusted unless
 *     SI_FLAG_CHECK is given, which verifies that they start at or above 0, never decrease
 *     and describe lists of at most k_fixed entries (SI_ERR_OUT_OF_RANGE otherwise).  A status word is only ever overwritten with an error,
 *     so the caller clears it.
 *   - All device pointers must be 16-byte aligned; d_model must be a multiple of 64.
 *   - A store belongs to the device that was current when it was created; that device must
 *     be current in every call that launches work on it (SI_ERR_INVALID_ARG otherwise).
 *   - Active lists hold SLOT indices (positions in the layer's store), distinct.
 *     The list order does not change the result: contributions are accumulated in a
 *     fixed order chosen by the library, so repeated calls are bit-identical.
 *
 * There is no CPU fallback: every entry point that computes runs CUDA kernels.
 */
#ifndef SELECTINFER_H
#define SELECTINFER_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct si_store si_store_t; /* opaque host-side handle: one per model (all layers) */

typedef enum { SI_F16 = 1, SI_BF16 = 2, SI_F32 = 3 /* outputs only */ } si_dtype_t;

enum {
    SI_OK = 0,
    SI_ERR_INVALID_ARG = -1,
    SI_ERR_OUT_OF_RANGE = -2,
    SI_ERR_DUPLICATE = -3,
    SI_ERR_ALIGNMENT = -4,
    SI_ERR_NOMEM = -5,        /* caller-supplied buffer too small */
    SI_ERR_CUDA = -6,
    SI_ERR_TIMEOUT = -7,      /* a bounded device-side wait expired */
    SI_ERR_UNSUPPORTED = -8,
    SI_ERR_TOO_LARGE = -9     /* a size exceeds a fixed built-in limit (si_ffn_forward_noalloc) */
};

/* flags */
enum {
    SI_FLAG_CHECK = 1u,          /* validate lists on the device (range, duplicates) first */
    SI_FLAG_RESIDUAL = 2u,       /* y = x + FFN(x) instead of FFN(x) */
    SI_FLAG_UNION_UNMASKED = 4u, /* T > 1 only: every token uses the whole union (extension) */
    SI_FLAG_SCORE_ABS = 8u,      /* si_select: rank |score| instead of score */
    SI_FLAG_SHARED_LIST = 16u,   /* T > 1 only: idx is ONE list of k_fixed slots used by every token */
    SI_FLAG_UNION_PATH = 32u,    /* si_ffn_forward: form the union and run the tensor-core contractions also for a
                                    single token (calls with more than one token always do) */
    SI_FLAG_LIST_PER_LAYER = 64u, /* si_decode_stack_forward, fixed-length lists only: idx holds ONE list per layer
                                    ([n_layers, k_fixed]) and every step uses the list of its layer -- the paper's
                                    decode, where the set chosen during prefill stays fixed for the prompt */
    SI_FLAG_STEPS_ANY_ORDER = 128u, /* si_decode_stack_forward: the SMs work in up to four groups that each take every
                                    fourth step, whatever the lists' length (without the flag: one group for long
                                    lists, two or four for short ones, see there) */
    SI_FLAG_SIMPLE_KERNELS = 256u, /* decode: one plain-load kernel pair per step instead of the
                                     persistent bulk-copy kernel (kept for cross-checking) */
    SI_FLAG_PRENORM = 512u       /* si_decode_chain_forward: the FFN sees its input scaled to unit root mean
                                    square, as the FFN of a pre-norm transformer block does */
};

/* selection modes for si_select */
enum { SI_SELECT_TOPK = 0, SI_SELECT_THRESHOLD = 1 };

const char *si_strerror(int status);

/* Text of the last CUDA runtime error behind an SI_ERR_CUDA return on this thread. */
const char *si_last_cuda_error(void);

/* ---------------------------------------------------------------- the neuron store

 * Bytes of device memory a store of n_layers layers needs; n_loaded is a host array
 * [n_layers] with the number of loaded neurons per layer.  Per layer the store holds
 * n_loaded records of 3 * d_model 16-bit values -- [gate row | up row | down column as
 * a row] -- i.e. exactly the loaded slices and nothing else (Section 4; the bytes not
 * stored are Eq. 2's saving), plus the slot <-> global id maps. */
int si_store_bytes(int n_layers, int d_model, int d_ff, const int *n_loaded, int dtype,
                   size_t *bytes_out);

/* Creates the handle over caller-owned device memory `store_mem` (256-byte aligned,
 * at least si_store_bytes).  Nothing is launched.  The memory must stay valid until
 * si_store_free. */
int si_store_create(si_store_t **store_out, void *store_mem /*device*/, size_t store_mem_bytes,
                    int n_layers, int d_model, int d_ff, const int *n_loaded /*host [L]*/,
                    int dtype);

/* Waits for the device to go idle and frees the handle (not the device memory). */
int si_store_free(si_store_t *store);

/* Selective loading of one layer (Section 4): gathers the slices of the listed neurons
 * out of the full weights into the layer's records.
 *   w_gate, w_up : device, [d_ff, d_model] row-major, store dtype
 *   w_down       : device, [d_model, d_ff] row-major, store dtype
 *   neuron_ids   : HOST int32 [n_loaded], global neuron ids, distinct, each in
 *                  [0, d_ff): the n_base base (task-specific) neurons first, then the
 *                  secondary (model-specific) ones; slot s holds neuron_ids[s].
 *   n_loaded     : must equal the count given to si_store_create for this layer.
 * Errors: SI_ERR_OUT_OF_RANGE / SI_ERR_DUPLICATE for bad ids (nothing is launched). */
int si_load_neurons(si_store_t *store, int layer, const void *w_gate, const void *w_up,
                    const void *w_down, const int32_t *neuron_ids, int n_loaded, int n_base,
                    void *stream);

/* Read-only views into the store (device pointers, valid while the store lives). */
int si_store_slot_to_global(const si_store_t *store, int layer, const int32_t **dev_ptr_out,
                            int *n_loaded_out, int *n_base_out);
int si_store_global_to_slot(const si_store_t *store, int layer, const int32_t **dev_ptr_out);
int si_store_records(const si_store_t *store, int layer, const void **dev_ptr_out,
                     size_t *record_bytes_out);

/* Workspace (device scratch) size for calls with at most T_max tokens per call, lists
 * of at most k_max slots, and at most max_steps (token, layer) steps per stack call. */
int si_workspace_bytes(const si_store_t *store, int T_max, int k_max, int max_steps,
                       size_t *bytes_out);

/* ---------------------------------------------------------------- selection

 * Runtime selector (Section 5: sort the activations in descending order, keep the top
 * alpha, record their indices).  scores: device float32 [n].
 *   mode SI_SELECT_TOPK      : the k highest scores.  Ties: the lower index wins;
 *                              +0 and -0 are equal; NaN ranks below every number.
 *   mode SI_SELECT_THRESHOLD : all i with score[i] > tau, NaN excluded (extension; the
 *                              paper has top-alpha only).
 * idx_out: device int32 [cap], ascending by index; *n_out (device int32) = count
 * written.  SI_ERR_NOMEM in *status-style return if cap < k (top-k); in threshold mode
 * at most cap indices are written and *n_out holds the full count.
 * workspace: device scratch of at least si_select_workspace_bytes(n). */
int si_select_workspace_bytes(int n, size_t *bytes_out);
int si_select(const float *scores, int n, int mode, int k, float tau, unsigned flags,
              int32_t *idx_out, int cap, int32_t *n_out, void *workspace, size_t ws_bytes,
              void *stream);

/* ---------------------------------------------------------------- selective FFN

 * y[t] = sum over i in list_t of h_i(x[t]) * down_i      (Section 5)
 *   x   : device [T, d_model], store dtype
 *   idx : device int32 slot indices.  If idx_offsets == NULL every token has k_fixed
 *         entries: idx is [T, k_fixed].  Otherwise idx_offsets is device int32 [T + 1]
 *         (CSR) and k_fixed is an upper bound on the longest list.
 *   y   : device [T, d_model] of y_dtype (SI_F32, or the store dtype)
 * T == 1 runs the memory-bound decode kernel; T > 1 forms the union of the lists and
 * runs a gathered tensor-core contraction in which token t still uses exactly its own
 * list (unless SI_FLAG_UNION_UNMASKED); this path needs d_model % 128 == 0
 * (SI_ERR_UNSUPPORTED otherwise).  SI_FLAG_UNION_PATH forces the union path for a single
 * token as well (the workspace must then be sized for T_max = 2).  An
 * empty list gives y = 0 (or x with SI_FLAG_RESIDUAL).  Accumulation is fp32; h is rounded
 * to the store dtype before the down projection only on the union path. */
int si_ffn_forward(const si_store_t *store, int layer, const void *x, int T, const int32_t *idx,
                   const int32_t *idx_offsets, int k_fixed, void *y, int y_dtype, unsigned flags,
                   void *workspace, size_t ws_bytes, int32_t *status_dev, void *stream);

/* One layer = optional selection + selective FFN (+ residual) ("applied to each FFN
 * layer", Section 4).  If scores != NULL (device float32 [T, n_loaded]) the k best
 * slots per token are selected with si_select's top-k rule into the workspace and
 * used as the lists; otherwise idx / idx_offsets / k are used as in si_ffn_forward. */
int si_layer_forward(const si_store_t *store, int layer, const void *x, int T, const float *scores,
                     int k, const int32_t *idx, const int32_t *idx_offsets, void *y, int y_dtype,
                     unsigned flags, void *workspace, size_t ws_bytes, int32_t *status_dev,
                     void *stream);

/* Batch-1 decode over a stack: n_steps consecutive (token, layer) steps in one
 * persistent launch, step s using layer layers[s] (HOST int32 [n_steps], or NULL for
 * s mod n_layers).  x, y: device [n_steps, d_model]; idx: device [n_steps, k_fixed]
 * (or CSR over n_steps lists).  Every step's x is an input of the call, so the steps do not depend
 * on one another (si_decode_chain_forward is the call for steps that do).  Every SM works through
 * its steps in their order; the weight stream of later steps is prefetched while earlier steps
 * finish, and a step's sum over the SMs completes a few steps behind the stream.  A step is spread
 * over as many SMs as its list keeps busy: all of them for lists of more than 1100 entries (k_fixed),
 * half of them up to 1100, a quarter up to 600 -- the SMs then work in two or four groups that each
 * take every second or fourth step, which divides the fixed work of a step by the number of groups.
 * SI_FLAG_STEPS_ANY_ORDER asks for four groups whatever the length.  All of y is complete when the
 * call's work on the stream is.
 * Results equal n_steps si_ffn_forward(T = 1) calls up to fp32 summation order (the split of
 * a list over SMs depends on the step's position in the call); each is run-to-run bit-stable.
 * With SI_FLAG_LIST_PER_LAYER (fixed-length lists only) idx is [n_layers, k_fixed] and a step
 * uses the list of its layer: the set chosen during prefill serves every token of the prompt. */
int si_decode_stack_forward(const si_store_t *store, int n_steps, const int32_t *layers,
                            const void *x, const int32_t *idx, const int32_t *idx_offsets,
                            int k_fixed, void *y, int y_dtype, unsigned flags, void *workspace,
                            size_t ws_bytes, int32_t *status_dev, void *stream);

/* Batch-1 decode over a stack whose steps depend on one another: step s + 1 takes the output of step s
 * as its input, the way the FFN of layer l + 1 sees what layer l produced ("applied to each FFN layer",
 * Section 4; decoding with the neuron set chosen for the prompt, Section 5).  The steps come in chains
 * of chain_len: step s with s mod chain_len == 0 starts a chain and reads row s / chain_len of x; every
 * other step reads row s - 1 of y.  One token through all layers is a chain of n_layers steps.
 *   x   : device [ceil(n_steps / chain_len), d_model], store dtype: the input of every chain
 *   y   : device [n_steps, d_model], STORE dtype (a step's output is the next step's input, so it is
 *         rounded once, to the type the FFN reads)
 *   flags: SI_FLAG_RESIDUAL  y_s = in_s + FFN(...) with in_s the step's input row;
 *          SI_FLAG_PRENORM   FFN(in_s) is replaced by FFN(n(in_s)), n(v) = v / sqrt(mean(v^2) + norm_eps)
 *                            rounded to the store dtype: the (gain-free) RMS normalisation in front of
 *                            the FFN of a pre-norm block.  Without it the scale of a chain drifts by the
 *                            square per step (h is a product of two projections of the input), so chains
 *                            longer than a few steps leave the range of 16-bit types; the paper's models
 *                            normalise in front of every FFN.  The sum of squares is formed in fp32 in
 *                            a fixed order, so the result is run-to-run bit-stable;
 *          SI_FLAG_LIST_PER_LAYER, SI_FLAG_CHECK as for si_decode_stack_forward.
 *   xn_out: optional device [n_steps, d_model], store dtype: with SI_FLAG_PRENORM, the normalised and
 *         rounded row every step fed to its dot products (for inspection); NULL otherwise.
 *   layers, idx, idx_offsets, k_fixed, workspace (si_workspace_bytes with max_steps >= n_steps),
 *   status_dev, stream: as for si_decode_stack_forward.
 * No arithmetic of step s + 1 starts before row s of y is complete on every SM; what runs ahead is the
 * weight stream: the lists are inputs of the call (the set is fixed per prompt), so the first records of
 * step s + 1 are already in shared memory when its input arrives.  All steps run in one persistent
 * launch; hidden sizes the persistent kernel does not cover return SI_ERR_UNSUPPORTED. */
int si_decode_chain_forward(const si_store_t *store, int n_steps, const int32_t *layers, int chain_len,
                            const void *x, const int32_t *idx, const int32_t *idx_offsets, int k_fixed,
                            void *y, void *xn_out, float norm_eps, unsigned flags, void *workspace,
                            size_t ws_bytes, int32_t *status_dev, void *stream);

/* Decode with a static prefix.  Section 5: the static neurons are always computed and the dynamic ones are
 * chosen per prompt; the static neurons are the base neurons, which come first in the store (slots
 * 0 .. n_static-1 of every layer).  Every step computes its layer's slots 0 .. n_static-1 and the listed
 * slots, which must all be >= n_static (a smaller one repeats a static neuron: SI_ERR_DUPLICATE under
 * SI_FLAG_CHECK); the lists hold the dynamic neurons only, and the static part of a step is streamed
 * straight from the store's first n_static records without a list entry being read.
 *   chain_len == 0 : the steps are independent, x is [n_steps, d_model], as si_decode_stack_forward
 *                    (y_dtype SI_F32 or the store dtype; xn_out and norm_eps unused);
 *   chain_len  > 0 : chained steps as si_decode_chain_forward (x holds one row per chain, y has the
 *                    store dtype, SI_FLAG_PRENORM / xn_out / norm_eps apply).
 * The other arguments are those of the two calls; k_fixed bounds the listed (dynamic) entries of a step
 * and n_static + k_fixed may not exceed a layer's loaded neurons.  Persistent kernel only
 * (SI_ERR_UNSUPPORTED for hidden sizes it does not cover). */
int si_decode_prefix_forward(const si_store_t *store, int n_steps, const int32_t *layers, int n_static, int chain_len,
                             const void *x, const int32_t *idx, const int32_t *idx_offsets, int k_fixed,
                             void *y, int y_dtype, void *xn_out, float norm_eps, unsigned flags, void *workspace,
                             size_t ws_bytes, int32_t *status_dev, void *stream);

/* Batch-1 selective FFN for callers that cannot allocate device memory.  (The paper has no
 * counterpart: this is a packaging variant of si_ffn_forward with T = 1.)
 *
 * Who needs it: code that runs where cudaMalloc is off limits -- a plugin inside a host
 * application that owns and budgets all device memory, a callback running under someone else's
 * allocator, a real-time loop that may not touch the allocator after start-up.  Such a caller can
 * still hand over its inputs and outputs, but it has no way to provide the scratch the kernels
 * need, so the scratch lives inside the library: a fixed device array of 304 x 8192 floats
 * (about 9.5 MiB) that every GPU loading the library holds until the process exits.
 *
 *   x, idx (k distinct slots), y, y_dtype, status_dev, stream: as for si_ffn_forward with T = 1;
 *   flags: SI_FLAG_RESIDUAL only (others are ignored).
 * Limits: d_model <= 8192 and at most 152 SMs; beyond that the call returns SI_ERR_TOO_LARGE and
 * launches nothing.  The call never allocates or frees memory, directly or through a library.
 * The store's device must be current (SI_ERR_INVALID_ARG otherwise).
 * The first call on each device looks up the array's device address;
 * make that first call outside any stream capture.  All calls on a device share the one array:
 * it needs no clearing between calls (each call overwrites what it later reads), but two calls
 * whose kernels overlap on the GPU -- different streams without ordering -- race on it.  Results
 * are bit-identical to si_ffn_forward with SI_FLAG_SIMPLE_KERNELS on the same inputs. */
int si_ffn_forward_noalloc(const si_store_t *store, int layer, const void *x, const int32_t *idx, int k,
                           void *y, int y_dtype, unsigned flags, int32_t *status_dev, void *stream);

/* Union of T lists (the first stage of the T > 1 path, exposed for inspection):
 * union_out device int32 [n_loaded] ascending, *n_union_out device int32. */
int si_union(const si_store_t *store, int layer, int T, const int32_t *idx,
             const int32_t *idx_offsets, int k_fixed, int32_t *union_out, int32_t *n_union_out,
             void *workspace, size_t ws_bytes, void *stream);

/* ---------------------------------------------------------------- prefill: dynamic neurons
 *
 * Section 5: during prefill the activations of all loaded neurons are computed for every prompt
 * token; each token's top alpha neurons are recorded, the occurrences are counted over the
 * tokens, the beta most frequent neurons are the dynamic candidates, and the static neurons
 * (slots 0 .. n_static-1: the base neurons come first in the store) are combined with the
 * candidates, in order of frequency, until phi_count neurons are chosen.  Ties (per-token
 * activations, frequencies) go to the lower slot; a neuron that occurs in no list is never
 * dynamic; candidates that are static already are skipped.  If phi_count <= n_static the
 * result is the first phi_count static slots.
 *
 * si_prefill_vote works on given activations:
 *   acts       device float32 [T, row_stride >= n]: activation of loaded slot i for token t
 *   flags      SI_FLAG_SCORE_ABS ranks |activation| (what the paper's "most active" means in its
 *              profiling; without the flag the signed value is ranked)
 *   idx_out    device int32, capacity cap >= phi_count: chosen slots, ascending; *n_out (device
 *              int32) their number (<= phi_count)
 *   counts_out optional device int32 [n]: the frequency of every slot
 *   workspace  device, 256-byte aligned, si_prefill_vote_workspace_bytes(T, n, alpha) bytes
 * Asynchronous on stream; integer decisions only, so the result is exact and unique. */
int si_prefill_vote_workspace_bytes(int T, int n, int alpha, size_t *bytes_out);
int si_prefill_vote(const float *acts, int T, int n, int row_stride, int alpha, int beta, int n_static,
                    int phi_count, unsigned flags, int32_t *idx_out, int cap, int32_t *n_out,
                    int32_t *counts_out, void *workspace, size_t ws_bytes, void *stream);

/* si_prefill_forward: prefill of one layer for the prompt's T tokens as the paper describes it --
 * y[t] = FFN over ALL loaded neurons of the layer (tensor-core path, one shared list of every slot) --
 * followed by si_prefill_vote on the activations h = SiLU(g) * u that this computation itself
 * produced (rounded to the store dtype, as they enter the down projection).
 *   x, y       device [T, d_model] (y of y_dtype: SI_F32 or the store dtype); flags: SI_FLAG_RESIDUAL,
 *              SI_FLAG_SCORE_ABS
 *   idx_out, cap, n_out, alpha, beta, n_static, phi_count: as for si_prefill_vote
 *   acts_out   optional device float32 [T, n_loaded]: receives the activations that were ranked
 *   workspace  si_workspace_bytes(store, max(T, 2), n_loaded, 1) bytes; vote_workspace
 *              si_prefill_vote_workspace_bytes(T, n_loaded, alpha) bytes, both 256-byte aligned
 * Asynchronous on stream. */
int si_prefill_forward(const si_store_t *store, int layer, const void *x, int T, void *y, int y_dtype,
                       int alpha, int beta, int n_static, int phi_count, unsigned flags, int32_t *idx_out,
                       int cap, int32_t *n_out, float *acts_out, void *workspace, size_t ws_bytes,
                       void *vote_workspace, size_t vote_ws_bytes, int32_t *status_dev, void *stream);

/* ---------------------------------------------------------------- offline: profiler and load set
 *
 * Section 3 (Eq. 1): the score of a neuron is the sum, over the tokens processed during profiling, of
 * the absolute value of its activation (the input of the down projection).  Scores and token counts
 * go to score files; files are merged by dividing each file's scores by its token count and summing;
 * the outcome is the list of neuron indices in decreasing order of importance.  Section 4: the
 * neurons to load are the top n_base of a task ranking (base neurons), then the model ranking in
 * order, neurons already chosen skipped, until n_loaded neurons (secondary neurons).
 *
 *   si_profile_accumulate  scores[i] += sum_t |acts[t, i]| (device float64 [n], caller zeroes it for a
 *                          new file; tokens are added in order, so totals are bit-reproducible).  The
 *                          activations of all d_ff neurons of a layer come from si_prefill_forward's
 *                          acts_out on a store that holds every neuron.
 *   si_profile_merge       merged[i] += scores[i] / tokens   (device float64 [n]; files in call order)
 *   si_profile_rank        ranking (device int32 [n]) = indices by decreasing score, ties to the lower
 *                          index, NaN last
 *   si_loadset             ids_out (device int32 [n_loaded]) from two rankings over n neurons;
 *                          workspace: ceil(n / 32) * 4 bytes; *status_dev (optional) receives
 *                          SI_ERR_OUT_OF_RANGE / SI_ERR_DUPLICATE for a malformed ranking and
 *                          SI_ERR_INVALID_ARG if the rankings do not yield n_loaded distinct neurons
 * All asynchronous on stream; all decisions and sums are exact and ordered, hence unique. */
int si_profile_accumulate(const float *acts, int T, int n, int row_stride, double *scores, void *stream);
int si_profile_merge(double *merged, const double *scores, long long tokens, int n, void *stream);
int si_profile_rank(const double *scores, int n, int32_t *ranking, void *stream);
int si_loadset(const int32_t *task_rank, const int32_t *model_rank, int n, int n_base, int n_loaded,
               int32_t *ids_out, void *workspace, size_t ws_bytes, int32_t *status_dev, void *stream);

/* Layer policy of Table 1 ("first layer" f, "last layer" l, l <= 0 counted from the end): the layers
 * that run selectively are first_out .. last_out - 1 = f .. n_layers + l - 1 (0-based); the others
 * keep their whole FFN.  With f = 5, l = -2 this gives 9 of 16 and 21 of 28 layers, the counts the
 * paper's evaluation states.  Host function; returns SI_ERR_INVALID_ARG if the range is empty or
 * outside the model. */
int si_layer_range(int n_layers, int first, int last, int *first_out, int *last_out);

/* ---------------------------------------------------------------- neuron shards over several GPUs
 *
 * Section 5 gives the layer output as a sum over the selected neurons, so P devices that each hold a
 * disjoint share of the loaded neurons can each compute the partial output of their share; the
 * partial outputs (fp32) are then added.  The paper runs on one device; this split is for layers
 * whose loaded set does not fit one GPU or for many tokens per call.  Shares are dealt round-robin:
 * device r of P holds global slots r, r + P, r + 2P, ... as its local slots 0, 1, 2, ... (load it with
 * neuron_ids[r + j*P] and n_base_local = ceil((n_base - r) / P)), so every device keeps the importance
 * order, the static-prefix property and an equal share of the frequently active slots.
 *
 *   si_shard_count    host function: *count_out = number of global slots < n that device `rank` holds.
 *   si_shard_lists    rewrites slot lists for one device: of every list it keeps the entries s with
 *                     s mod world == rank, as s div world, order kept, and packs the lists back to
 *                     back: list t is idx_out[offsets_out[t] .. offsets_out[t+1]).  Input lists as
 *                     in si_ffn_forward (idx_offsets[n_lists+1], or NULL and k_fixed entries each).
 *                     idx_out: device int32, room for every input entry; offsets_out: device int32
 *                     [n_lists + 1]; workspace: (n_lists + 64) * 4 bytes, 16-byte aligned.  Entries
 *                     below 0 are dropped and reported through *status_dev (SI_ERR_OUT_OF_RANGE).
 *                     Feed the result to si_ffn_forward with idx_offsets = offsets_out and k_fixed =
 *                     an upper bound of the local list lengths.  Lists are fixed per prompt
 *                     (Section 5), so this runs once per prompt and layer, not per token.
 *   si_shard_reduce   y[t][j] = (x[t][j] +) parts[0][t][j] + parts[1][t][j] + ... in rank order (a fixed
 *                     order: the result is the same on every device).  parts_dev: DEVICE array of
 *                     `world` device pointers to fp32 [T][d_model] partial outputs -- peer pointers
 *                     for a one-shot all-reduce by plain peer loads, or a single pointer to a buffer an
 *                     all-reduce has already summed (world = 1: residual and conversion only).  The
 *                     caller orders this call after the partial outputs are complete on every device.
 *                     x, y: as in si_ffn_forward (x may be NULL without SI_FLAG_RESIDUAL).
 * All device work is asynchronous on stream.  No counterpart in the paper. */
int si_shard_count(int n, int rank, int world, int *count_out);
/*   si_ffn_forward_sharded   batch-1 decode of this device's share with the all-reduce inside the kernel that
 *                     finishes the down projection: every block of that kernel adds the device's partial rows for its
 *                     32 output columns, stores the sums into EVERY device's receive area with plain peer stores,
 *                     marks the block as delivered on every device, waits (with a limit: SI_ERR_TIMEOUT in
 *                     *status_dev) until every device has delivered the same block here, adds the devices' sums in
 *                     rank order (the result is the same bits on every device), adds the residual, rounds, writes
 *                     y.  No collective call and no further kernel.
 *                       x, idx (k local slots), y, y_dtype, flags (SI_FLAG_RESIDUAL), workspace: as si_ffn_forward, T = 1
 *                       recv   HOST array of `world` device pointers, recv[q] = device q's receive area, fp32
 *                              [2][world][d_model], mapped for this device (peer access / IPC mapping);
 *                       marks  HOST array of `world` device pointers, marks[q] = device q's delivery marks, uint32
 *                              [world][d_model / 32], zero before the first call;
 *                       epoch  the number of this call on these buffers: 1, 2, 3, ... on every device alike (its
 *                              parity picks the half of the receive areas, so a device may be one call ahead).
 *                     d_model must be a multiple of 128, world at most 8.  Tested with all ranks of a group
 *                     sharing one GPU (one launch over all of them); not tested across GPUs: this run has one. */
int si_ffn_forward_sharded(const si_store_t *store, int layer, const void *x, const int32_t *idx, int k, void *y,
                           int y_dtype, unsigned flags, int rank, int world, float *const *recv, unsigned *const *marks,
                           unsigned epoch, void *workspace, size_t ws_bytes, int32_t *status_dev, void *stream);
int si_shard_lists(const int32_t *idx, const int32_t *idx_offsets, int k_fixed, int n_lists, int rank, int world,
                   int32_t *idx_out, int32_t *offsets_out, void *workspace, size_t ws_bytes, int32_t *status_dev,
                   void *stream);
int si_shard_reduce(const float *const *parts_dev, int world, const void *x, int x_dtype, int T, int d_model,
                    void *y, int y_dtype, unsigned flags, void *stream);

/* Library build information: "sm_100a" etc.  Never NULL. */
const char *si_build_info(void);

#ifdef __cplusplus
}
#endif
#endif /* SELECTINFER_H */
