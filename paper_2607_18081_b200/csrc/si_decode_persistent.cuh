// Persistent batch-1 selective decode for sm_100a.
//
// One CTA per SM runs any number of (token, layer) steps in a single launch.  Roles in a CTA:
//   * warp 0 (producer) streams each selected neuron record -- 6*d_model contiguous bytes:
//     gate row | up row | down row -- from HBM into shared memory with one bulk async copy
//     (cp.async.bulk, completion on an mbarrier).  There are two rings, one per consumer set;
//     every ring stage has its own issuing lane, and the copy descriptors (source address,
//     bytes) are prepared 16 at a time per set and kept in shared memory, so the slot index
//     loads are off the issue path.  The rings run ahead across step boundaries.
//   * warps 1..16 (consumers) form two independent sets of 8 warps.  List position p of a
//     step goes to set (p + rot) mod 2G (rot = list entries before the step, so records are
//     dealt round-robin across steps).  A bulk copy takes several microseconds to land and
//     bandwidth needs every ring stage in flight, so a landed record is copied into
//     registers and its stage handed back at once; the set then forms the two dot products
//     (thread slices, warp butterfly, 8-warp exchange through a hardware named barrier), applies SiLU(g)*u and
//     accumulates h * down for its columns in fp32 registers -- while its next record is
//     already on the way.  At the end of a step each set leaves its accumulators in shared
//     memory for the reducer warps and goes straight on to the next step.
//   * warps 17..19 (reducers, step s goes to warp s mod 3) own everything that involves other
//     SMs: they add the two sets' accumulators, store the CTA's partial y into a ring of D
//     global buffers, publish it (grid-scope fence + atomic), and kLag steps later -- when every
//     CTA has long published that step -- sum the partial rows of this CTA's column groups in a
//     fixed order (lane rows ascending, warp butterfly: deterministic split-K) and write y
//     once.  The reduction trails the record stream and never stalls it.
//
// Chained mode (template parameter CH; Params::chain_len > 0): step s takes the output row of step s - 1
// as its input unless s is the first step of a chain (s mod chain_len == 0), the way the FFN of layer
// l + 1 sees what layer l produced.  Nothing of a step's arithmetic can start before the step before it is
// complete, so the time between the last record of a step and the first dot product of the next is pure
// latency and the kernel is built to make it short: the reducer warps stay out of it; the consumers
// themselves store the CTA's partial row as 8-byte words {value, tag}, gather their CTA's columns of every
// row by polling those words (no fence, no flag, no second round trip), add them in a fixed order, write y
// and publish the next input row the same way, and every consumer polls the words of the row it needs.
// The record rings are not held back: the lists are known up front (the set is fixed per prompt), so a
// step's first records are in shared memory, and the ones behind them on their way into L2, before its
// input exists.  With Params::prenorm the input row is normalised to unit root mean square (and rounded
// to the store type) before the dot products.
//
// Every wait is bounded: on expiry the kernel records SI_ERR_TIMEOUT, raises a grid-wide
// abort flag, lets its outstanding copies land and returns.
#pragma once

#include "si_common.cuh"

#define SI_MAX_LAYERS 128

namespace si_persist {

constexpr int kSets = 2;                          // independent consumer sets, each with its own ring (one set of 16 warps for wide rows)
constexpr int kSetWarps = 8;
constexpr int kSetThreads = kSetWarps * 32;
constexpr int kConsumers = kSets * kSetThreads;
constexpr int kConsumerWarps = kConsumers / 32;
constexpr int kReducerWarps = 3;
constexpr int kThreads = 32 + kConsumers + 32 * kReducerWarps;        // producer, consumers, reducers
constexpr int kThreadsChained = 32 + kConsumers;                      // chained mode has no reducer warps
constexpr int kMaxGroups = 32;                    // most float4 column groups one CTA reduces (d_model / 4 / CTAs per step group, rounded up)
constexpr int kCounterStride = 64;                // uint32 per step: written at +0, reduced at +32 (own 128-byte lines)
constexpr int kMaxStages = 16;
constexpr int kDescRing = 64;                     // copy descriptors per set kept ahead of the issue lanes
constexpr int kPartialDepth = 10;                 // D: partial-y buffers in flight
constexpr int kFewSteps = 16;                     // launches this short carry their layer ids as kernel arguments
constexpr int kProfSlots = 16;                    // int64 cycle counters per SM in the optional phase profile
constexpr int kLag = 4;                           // a step's cross-SM reduction starts this many steps later
constexpr long long kWaitCycles = 4000000000ll;   // default limit of every wait: ~2 s at 1.9 GHz
constexpr long long kDrainCycles = 40000000ll;    // least time a leaving producer gives its copies in flight to land
constexpr int kLLRows = 8;                        // chained mode: most partial rows one consumer thread gathers per step
constexpr int kChainCmb = 0, kChainXch = 1, kChainRows = 2;   // chained mode: which hand-over barrier serves what
constexpr int kSplitSlicesFull = 0, kSplitSlicesFree = 1, kSplitH = 2, kSplitRed = 3, kSplitHint = 4, kSplitInput = 5;   // split form: accfull[q][w] taken as [q * 3 + w]
constexpr int kSplitLoaderWarps = 2;                          // split form: warps that copy the down slices
constexpr int kThreadsSplit = 32 + kConsumers + 32 * kSplitLoaderWarps;
constexpr int kSplitKCapMax = 1856;                           // split form: list entries whose slices fit beside six ring stages at d_model 4096

struct Params {
    const char *store_base;
    unsigned long long rec_off[SI_MAX_LAYERS];
    int n_loaded[SI_MAX_LAYERS];
    int n_layers, n_steps, k_fixed, d_model, chunks, nstage;
    const int32_t *step_layers;   // device int32 [n_steps] or nullptr (then: few_layers, else step mod n_layers)
    int n_few;                    // > 0: the launch has n_few <= kFewSteps steps, their layers are in few_layers
    unsigned char few_layers[16];
    const uint16_t *x;            // [n_steps, d_model]
    const int32_t *idx;           // [n_steps, k_fixed] or CSR payload
    const int32_t *idx_offsets;   // CSR [n_steps + 1] or nullptr
    void *y;
    int y_f32, residual;
    int per_layer_lists;          // fixed-length lists only: idx is [n_layers][k_fixed], a step uses the list of its layer
    int n_static;                 // every step also computes slots 0 .. n_static-1 of its layer (the static neurons, which come
                                  // first in the store) ahead of its listed entries: positions 0 .. n_static-1 of the step need
                                  // no list load at all
    int n_groups;                 // step groups: CTA c belongs to group c mod n_groups and, with the other CTAs of its
                                  // group, runs the steps s = group (mod n_groups); 1 = every CTA works on every step
    float *partial;               // [n_groups][D][G][d_model], G = CTAs per group
    unsigned int *ctrl;           // [1] abort flag (zero at launch)
    unsigned int *counters;       // [n_steps][kCounterStride], zero at launch: +0 "written" = CTAs that
                                  // stored their partial of the step, +32 "reduced" = CTAs that finished
                                  // reading the step's partials
    int32_t *status;
    long long *prof;              // optional phase profile: int64 [G][kProfSlots] cycle counters, or nullptr
    int stream_only;              // diagnostics bit mask (si_debug_decode_opts_t::skip_mask)
    long long wait_cycles;        // limit of every wait, in clock cycles
    int withhold;                 // diagnostics: the producer of CTA 0 never issues the second item of its first set
    // chained mode
    int chain_len;                // 0: every step's x is an input of the call; > 0: x holds one row per chain
                                  // ([ceil(n_steps / chain_len)][d_model]) and step s with s mod chain_len != 0
                                  // reads row s - 1 of y (store dtype) as its input
    int prenorm;                  // the input row is scaled to unit root mean square before the FFN
    float norm_eps;
    uint16_t *xn_out;             // optional [n_steps][d_model]: the normalised, rounded input every step used
    // chained mode: the two exchanges between the SMs go through words that carry their own "ready" mark --
    // 8 bytes = {payload, tag}, written and read as a whole, tag = 1 + step -- so a reader polls the data
    // itself and no fence, flag or second round trip stands between a store and its use
    uint2 *ll_partial;            // [G][d_model] {fp32 partial sum of the CTA's records, tag}, zero at launch
    uint2 *ll_x;                  // [2][d_model / 2] {two 16-bit values of the next input row, tag}, zero at launch
    unsigned csum_off;            // chained mode: byte offset of the [columns][classes] class sums in shared memory
    // chained mode, split form (template parameter CH == 2): a step is cut at the activations instead of
    // at the output.  Every set computes h for its records from the gate and up rows alone and publishes it
    // as one {h, tag} word; every CTA gathers all h of the step (a few KB) and forms the output columns it owns
    // from 16-byte slices of ALL the step's down rows, which a loader warp pair has copied into shared memory
    // long before (their addresses depend on the list alone).  What crosses between the SMs per step is then
    // k + d_model words instead of the SMs x d_model partial sums of the other form.
    unsigned stage_bytes;         // bytes of a ring stage (a whole record, or its gate and up rows)
    unsigned copy_bytes;          // bytes the producer copies per record
    unsigned sm_off;              // byte offset of the Smem struct
    unsigned sbuf_off, hbuf_off, red_off, prev_off;   // split form: down slices [k_cap][64 B], h [k_cap], partial sums, last outputs
    int k_cap;                    // split form: most list entries per step (what the slice buffer holds)
    uint2 *ll_h;                  // split form: [2][k_cap] {h, tag}, zero at launch
};

__device__ __forceinline__ uint32_t smem_u32(const void *p) {
    return (uint32_t)__cvta_generic_to_shared(p);
}
__device__ __forceinline__ void mbar_init(uint64_t *bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint64_t *bar) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(bar)) : "memory");
}
__device__ __forceinline__ void mbar_arrive_expect_tx(uint64_t *bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(bar)), "r"(bytes)
                 : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint64_t *bar, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok) : "r"(smem_u32(bar)), "r"(parity) : "memory");
    return ok != 0;
}
// Non-blocking probe (try_wait may suspend the thread for a while when the phase is not complete,
// which would hold back the other lanes of a polling warp).
__device__ __forceinline__ bool mbar_test_wait(uint64_t *bar, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.test_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok) : "r"(smem_u32(bar)), "r"(parity) : "memory");
    return ok != 0;
}
// Bounded wait; also gives up when the CTA-local abort flag is raised.
__device__ __forceinline__ bool mbar_wait_bounded(uint64_t *bar, uint32_t parity, volatile int *cta_abort, long long limit) {
    if (mbar_try_wait(bar, parity)) return true;
    long long t0 = clock64();
    while (true) {
        for (int i = 0; i < 64; ++i)
            if (mbar_try_wait(bar, parity)) return true;
        if (*cta_abort) return false;
        if (clock64() - t0 > limit) return false;
    }
}
// The same wait as a spin on the non-blocking probe: a thread suspended inside try_wait is not woken the
// moment the phase completes, which costs the chained steps (whose every wait is on the critical path)
// far more than the issue slots of a spin.
__device__ __forceinline__ bool mbar_spin_bounded(uint64_t *bar, uint32_t parity, volatile int *cta_abort, long long limit) {
    if (mbar_test_wait(bar, parity)) return true;
    long long t0 = clock64();
    while (true) {
        for (int i = 0; i < 32; ++i)
            if (mbar_test_wait(bar, parity)) return true;
        if (*cta_abort) return false;
        if (clock64() - t0 > limit) return false;
    }
}
// Strong (gpu-scope) vector store and vector add-reduction at L2; one thread issues both to the same
// address in program order, so the add lands on the stored value.
__device__ __forceinline__ void st_relaxed_gpu_f4(float4 *p, float4 v) {
    asm volatile("st.relaxed.gpu.global.v4.f32 [%0], {%1, %2, %3, %4};" ::"l"(p), "f"(v.x), "f"(v.y), "f"(v.z), "f"(v.w)
                 : "memory");
}
__device__ __forceinline__ void red_add_gpu_f4(float4 *p, float4 v) {
    asm volatile("red.relaxed.gpu.global.add.v4.f32 [%0], {%1, %2, %3, %4};" ::"l"(p), "f"(v.x), "f"(v.y), "f"(v.z), "f"(v.w)
                 : "memory");
}
// 16 bytes = two {payload, tag} words; each 8-byte word is written by one store and read whole
__device__ __forceinline__ uint4 ld_relaxed_gpu_v4(const uint4 *p) {
    uint4 v;
    asm volatile("ld.relaxed.gpu.global.v4.u32 {%0, %1, %2, %3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "l"(p) : "memory");
    return v;
}
__device__ __forceinline__ void st_relaxed_gpu_v4(uint4 *p, uint4 v) {
    asm volatile("st.relaxed.gpu.global.v4.u32 [%0], {%1, %2, %3, %4};" ::"l"(p), "r"(v.x), "r"(v.y), "r"(v.z), "r"(v.w) : "memory");
}
__device__ __forceinline__ void st_relaxed_gpu_v2(uint2 *p, uint2 v) {
    asm volatile("st.relaxed.gpu.global.v2.u32 [%0], {%1, %2};" ::"l"(p), "r"(v.x), "r"(v.y) : "memory");
}
__device__ __forceinline__ unsigned ld_acquire_gpu(const unsigned *p) {
    unsigned v;
    asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
    return v;
}
__device__ __forceinline__ unsigned ld_relaxed_gpu(const unsigned *p) {
    unsigned v;
    asm volatile("ld.relaxed.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
    return v;
}
// Bounded wait until *ctr >= target; gives up on the grid-wide or CTA-local abort flag.
__device__ __forceinline__ bool counter_wait_bounded(const unsigned *ctr, unsigned target, const unsigned *grid_abort,
                                                     volatile int *cta_abort, long long limit) {
    if (ld_acquire_gpu(ctr) >= target) return true;
    long long t0 = clock64();
    while (true) {
        for (int i = 0; i < 16; ++i) {
            if (ld_acquire_gpu(ctr) >= target) return true;
            __nanosleep(64);
        }
        if (*cta_abort || ld_relaxed_gpu(grid_abort)) return false;
        if (clock64() - t0 > limit) return false;
    }
}
// Chained mode: lane 0 of a warp polls an arrival counter that is only a hint ("the words you are about to
// read have probably all been written") -- the words carry their own tags, so nothing depends on the counter
// being ordered with them.  Returns false when the wait ran out or an abort flag is up.
// One thread of the CTA polls (thousands of lanes polling one word would queue up in front of the very
// increments they wait for) and passes the news on through a shared-memory barrier with one expected arrival.
__device__ __forceinline__ bool hint_wait_cta(const unsigned *ctr, unsigned target, const unsigned *grid_abort,
                                              volatile int *cta_abort, long long limit, bool poller, uint64_t *bar, uint32_t parity) {
    if (poller) {
        const long long t0 = clock64();
        unsigned spins = 0;
        while (ld_relaxed_gpu(ctr) < target) {
            if ((++spins & 31u) == 0 && (*cta_abort || ld_relaxed_gpu(grid_abort) || clock64() - t0 > limit)) return false;
        }
        mbar_arrive(bar);
        return true;
    }
    return mbar_spin_bounded(bar, parity, cta_abort, limit);
}
__device__ __forceinline__ void red_add_relaxed_gpu(unsigned *p, unsigned v) {
    asm volatile("red.relaxed.gpu.global.add.u32 [%0], %1;" ::"l"(p), "r"(v) : "memory");
}
__device__ __forceinline__ uint64_t l2_policy_evict_first() {
    uint64_t pol;
    asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(pol));
    return pol;
}
__device__ __forceinline__ void bulk_g2s(void *dst_smem, const void *src_gmem, uint32_t bytes, uint64_t *bar,
                                         uint64_t policy) {
    asm volatile(
        "cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes.L2::cache_hint [%0], [%1], %2, [%3], %4;"
        ::"r"(smem_u32(dst_smem)), "l"(src_gmem), "r"(bytes), "r"(smem_u32(bar)), "l"(policy)
        : "memory");
}

// Hardware barrier over the 256 threads of consumer set q (barrier id 1 + q) that also ORs a flag:
// every thread of the set learns whether any of them has a failed wait, so the set always leaves
// its loops together and nobody is left waiting at the barrier.
template <int kSetThreadsT>
__device__ __forceinline__ bool set_barrier_or(int q, bool v) {
    uint32_t r;
    asm volatile(
        "{\n\t.reg .pred p, f;\n\t"
        "setp.ne.u32 f, %1, 0;\n\t"
        "bar.red.or.pred p, %2, %3, f;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(r) : "r"((uint32_t)v), "r"(1 + q), "n"(kSetThreadsT) : "memory");
    return r != 0;
}

template <int DT>
__device__ __forceinline__ void unpack8(const uint4 &v, float (&f)[8]) {
    f[0] = si_cvt<DT>::lo(v.x); f[1] = si_cvt<DT>::hi(v.x);
    f[2] = si_cvt<DT>::lo(v.y); f[3] = si_cvt<DT>::hi(v.y);
    f[4] = si_cvt<DT>::lo(v.z); f[5] = si_cvt<DT>::hi(v.z);
    f[6] = si_cvt<DT>::lo(v.w); f[7] = si_cvt<DT>::hi(v.w);
}
template <int DT>
__device__ __forceinline__ float dot8(const uint4 &v, const float (&x)[8]) {
    float f[8];
    unpack8<DT>(v, f);
    float a = 0.f;
#pragma unroll
    for (int e = 0; e < 8; ++e) a = fmaf(f[e], x[e], a);
    return a;
}

// Packed pairs of fp32 values in 64-bit registers and the two-wide fp32 FMA of sm_100: half the
// FMA instructions of the scalar form for the dot products and the down accumulate.
__device__ __forceinline__ unsigned long long pack2(float lo, float hi) {
    unsigned long long r;
    asm("mov.b64 %0, {%1, %2};" : "=l"(r) : "f"(lo), "f"(hi));
    return r;
}
__device__ __forceinline__ void unpack2(unsigned long long v, float &lo, float &hi) {
    asm("mov.b64 {%0, %1}, %2;" : "=f"(lo), "=f"(hi) : "l"(v));
}
__device__ __forceinline__ unsigned long long fma2(unsigned long long a, unsigned long long b, unsigned long long c) {
    unsigned long long d;
    asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(d) : "l"(a), "l"(b), "l"(c));
    return d;
}
// the two 16-bit elements of a 32-bit word as a packed fp32 pair (element order kept)
template <int DT>
__device__ __forceinline__ unsigned long long pair_of(uint32_t w) {
    return pack2(si_cvt<DT>::lo(w), si_cvt<DT>::hi(w));
}
template <int DT>
__device__ __forceinline__ void unpack8p(const uint4 &v, unsigned long long (&f)[4]) {
    f[0] = pair_of<DT>(v.x); f[1] = pair_of<DT>(v.y); f[2] = pair_of<DT>(v.z); f[3] = pair_of<DT>(v.w);
}
// a += (v[0..7] * x[0..7]) pairwise: even elements accumulate in the low half, odd ones in the high half
template <int DT>
__device__ __forceinline__ unsigned long long dot8p(const uint4 &v, const unsigned long long (&x)[4], unsigned long long a) {
    a = fma2(pair_of<DT>(v.x), x[0], a); a = fma2(pair_of<DT>(v.y), x[1], a);
    a = fma2(pair_of<DT>(v.z), x[2], a); a = fma2(pair_of<DT>(v.w), x[3], a);
    return a;
}

// Per-step list geometry: which entries of the step's list belong to virtual CTA b of G.
// (k counts the static prefix and the listed entries; base is where the listed entries start in idx)
struct StepGeom { int base, k, first, cnt; };
__device__ __forceinline__ StepGeom step_geom(const Params &P, int step, int G, int b) {
    StepGeom g;
    long long before;
    if (P.idx_offsets) {
        int o0 = __ldg(P.idx_offsets + step), o1 = __ldg(P.idx_offsets + step + 1);
        g.base = o0; g.k = o1 - o0 < 0 ? 0 : o1 - o0; before = o0;
    } else {
        g.base = step * P.k_fixed; g.k = P.k_fixed; before = (long long)step * P.k_fixed;
    }
    g.k += P.n_static; before += (long long)step * P.n_static;     // the static prefix comes first in every step
    int rot = (int)(before % G);
    g.first = (b - rot + G) % G;
    g.cnt = g.k > g.first ? (g.k - g.first + G - 1) / G : 0;
    return g;
}

struct Smem {
    uint64_t full[kMaxStages];         // stage index = set * S + stage-in-set
    uint64_t empty[kMaxStages];
    // consumer set -> reducers hand-over of a step's accumulators (one buffer per set); one barrier
    // per reducer warp (slot s mod 3), so that each waiter follows the phases of its own barrier
    uint64_t accfull[kSets][kReducerWarps], accempty[kSets][kReducerWarps];
    int meta[kMaxStages];
    uint4 desc[kSets][kDescRing];      // {src lo, src hi, bytes (0: nothing to copy), meta}
    float2 setpart[kSets][2][2 * kSetWarps];   // [set][buf][warp] = (gate, up) partial dot products (16 warps in the one wide set)
    volatile int cta_abort;
};
static_assert(sizeof(Smem) <= 3008, "the eight ring stages of d_model = 4096 leave 3008 bytes for this struct");

__device__ __forceinline__ void raise_abort(const Params &P, Smem *sm, int code) {
    if (!sm->cta_abort) {
        sm->cta_abort = 1;
        if (P.status) atomicCAS(P.status, 0, code);
        atomicExch(P.ctrl + 1, 1u);
    }
}


// ------------------------------------------------------------------------------------------------
// Chained mode, consumer side.  A step is two functions that are deliberately not inlined: the record
// loop runs at the register limit, and the values one half keeps alive must not be in the other half's way
// (a spill inside the record loop goes to L2 here, the shared memory carve-out leaves next to no L1).
// What crosses from one to the other is a handful of integers; the sums cross through memory.

// First half: fetch the step's input row (the caller's, or the {values, tag} words the SMs wrote at the
// end of the step before), normalise it if asked to, run the set's records, and deliver the CTA's partial
// row: the second set parks its accumulators in shared memory, the first adds them to its own and stores
// the row as {partial sum, tag} words, then counts the row as written (a hint for the pollers).
// ring: stage | phase parity << 8 | exchange-buffer parity << 9 of the set's next ring item.

// Chained mode, both forms: the step's input row into packed fp32 pairs.  Either the caller's row (first
// step of a chain) or the {two 16-bit values, tag} words the CTAs wrote at the end of the step before,
// polled until every word this thread needs carries this step's tag (the row is 16 KB for all of them
// together: polling it costs the memory system little, and measured a little less time than waiting for a
// count of the CTAs that have written their columns).  With Params::prenorm the row is scaled to unit root
// mean square and rounded to the store type.  Contains a barrier over the set that also ORs `fail`.
template <int DT, int NCH, bool kFull>
__device__ __forceinline__ bool chain_input(const Params &P, Smem *sm, int step, int q, int t, unsigned long long (&xr)[NCH][4],
                                            uint32_t &recs, bool fail, uint64_t *hint_bar = nullptr, unsigned hint_target = 0) {
    constexpr int kSetWarps = 8, kSetThreads = 256;
    const int d = P.d_model, chunks = P.chunks, b = blockIdx.x, lane = t & 31, sw = t >> 5;
    volatile int *cta_abort = &sm->cta_abort;
    const long long wait_limit = P.wait_cycles;
    if (step % P.chain_len == 0) {
        const uint4 *xs = reinterpret_cast<const uint4 *>(P.x + (size_t)(step / P.chain_len) * d);
#pragma unroll
        for (int i = 0; i < NCH; ++i) {
            const int c = t + kSetThreads * i;
            if (kFull || c < chunks) unpack8p<DT>(__ldg(xs + c), xr[i]);
        }
        if (hint_bar && q == 0 && t == 0) mbar_arrive(hint_bar);      // (nothing to wait for: keeps the barrier's phase in step)
    } else {
        // 8-byte words {two 16-bit values, tag = this step}, polled until every word this thread needs carries
        // the tag (the row is 16 KB for all of them together: polling it costs the memory system little, and
        // measured a little less time than waiting for a count of the CTAs that have written their columns)
        const uint4 *lx = reinterpret_cast<const uint4 *>(P.ll_x + (size_t)(step & 1) * (d / 2));
        // split form: one thread of the CTA waits for the count of CTAs that have written their columns (a hint),
        // so that the row's few lines are read once instead of being polled by every thread of the GPU
        if (hint_bar)
            fail |= !hint_wait_cta(P.counters + (size_t)(step - 1) * kCounterStride + 32, hint_target, P.ctrl + 1, cta_abort, wait_limit,
                                   q == 0 && t == 0, hint_bar, (uint32_t)(step & 1));
        const long long t0 = clock64();
        uint32_t spins = 0;
        while (!fail) {
            bool good = true;
            uint4 w[NCH][2];
#pragma unroll
            for (int i = 0; i < NCH; ++i)
                if (kFull || t + kSetThreads * i < chunks) {
                    w[i][0] = ld_relaxed_gpu_v4(lx + (size_t)(t + kSetThreads * i) * 2);
                    w[i][1] = ld_relaxed_gpu_v4(lx + (size_t)(t + kSetThreads * i) * 2 + 1);
                }
#pragma unroll
            for (int i = 0; i < NCH; ++i)
                if (kFull || t + kSetThreads * i < chunks) {
                    good &= w[i][0].y == (uint32_t)step && w[i][0].w == (uint32_t)step && w[i][1].y == (uint32_t)step && w[i][1].w == (uint32_t)step;
                    xr[i][0] = pair_of<DT>(w[i][0].x); xr[i][1] = pair_of<DT>(w[i][0].z);
                    xr[i][2] = pair_of<DT>(w[i][1].x); xr[i][3] = pair_of<DT>(w[i][1].z);
                }
            if (good) break;
            if ((++spins & 63u) == 0 && (*cta_abort || ld_relaxed_gpu(P.ctrl + 1) || clock64() - t0 > wait_limit)) fail = true;
        }
    }
    if (P.prenorm) {
        // sum of squares of the row: thread slice, warp butterfly, then (after the barrier below) the set's
        // warps in warp order -- the same order in every set of every CTA.  The warp sums use the exchange
        // buffer the next record would use; the record after it uses the other one.
        float ss = 0.f;
#pragma unroll
        for (int i = 0; i < NCH; ++i)
#pragma unroll
            for (int e = 0; e < 4; ++e) {
                float lo, hi;
                unpack2(xr[i][e], lo, hi);
                ss = fmaf(lo, lo, ss); ss = fmaf(hi, hi, ss);
            }
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) ss += __shfl_xor_sync(0xFFFFFFFFu, ss, o);
        if (lane == 0) sm->setpart[q][recs & 1][sw].x = ss;
    }
    fail = set_barrier_or<kSetThreads>(q, fail);          // one answer for the whole set (and the warp sums are in place)
    if (fail) return true;
    if (P.prenorm) {
        float ss = 0.f;
#pragma unroll
        for (int w = 0; w < kSetWarps; ++w) ss += sm->setpart[q][recs & 1][w].x;
        recs ^= 1u;
        const float scale = rsqrtf(ss / (float)d + P.norm_eps);
        const bool emit = P.xn_out != nullptr && b == 0 && q == 0;
#pragma unroll
        for (int i = 0; i < NCH; ++i) {
            uint32_t w4[4];
#pragma unroll
            for (int e = 0; e < 4; ++e) {
                float lo, hi;
                unpack2(xr[i][e], lo, hi);
                w4[e] = (uint32_t)si_cvt<DT>::from_float(lo * scale) | ((uint32_t)si_cvt<DT>::from_float(hi * scale) << 16);
                xr[i][e] = pair_of<DT>(w4[e]);        // the dot products see the rounded values
            }
            const int c = t + kSetThreads * i;
            if (emit && (kFull || c < chunks))
                reinterpret_cast<uint4 *>(P.xn_out + (size_t)step * d)[c] = make_uint4(w4[0], w4[1], w4[2], w4[3]);
        }
    }
    return false;
}

// optional phase profile of the chained steps: thread 0 of each set adds the cycles since its last stamp to a slot
#define SI_CPROF(slot) do { if (cprof) { const long long now_ = clock64(); atomicAdd((unsigned long long *)(P.prof + (size_t)blockIdx.x * kProfSlots + (slot) + 8 * q_), (unsigned long long)(now_ - pt_)); pt_ = now_; } } while (0)

template <int DT, int NCH, bool kFull>
__device__ __noinline__ bool chain_step_records(const Params &P, uint8_t *smem, int step, unsigned &ring) {
    constexpr int kSets = 2, kSetWarps = 8, kSetThreads = 256;
    const int d = P.d_model, chunks = P.chunks, rec_bytes = d * 6, S = P.nstage / kSets;
    const int G = gridDim.x, b = blockIdx.x;
    Smem *sm = reinterpret_cast<Smem *>(smem + P.sm_off);
    float *comb = reinterpret_cast<float *>(smem + (size_t)P.nstage * rec_bytes);      // [d_model] second set's accumulators
    volatile int *cta_abort = &sm->cta_abort;
    const long long wait_limit = P.wait_cycles;
    const int ct = threadIdx.x - 32, lane = ct & 31;
    const int q = ct / kSetThreads, t = ct & (kSetThreads - 1), sw = t >> 5;
    uint64_t *sfull = sm->full + q * S, *sempty = sm->empty + q * S;
    const int *smeta = sm->meta + q * S;
    const uint8_t *sring = smem + (size_t)q * S * rec_bytes;
    int st = (int)(ring & 0xFFu); uint32_t ph = (ring >> 8) & 1u, recs = (ring >> 9) & 1u;
    bool fail = false;
    const uint32_t tag = (uint32_t)step + 1u;
    const bool cprof = P.prof != nullptr && t == 0;
    const int q_ = q;
    long long pt_ = cprof ? clock64() : 0;

    unsigned long long xr[NCH][4], acc[NCH][4];   // packed fp32 pairs
#pragma unroll
    for (int i = 0; i < NCH; ++i)
#pragma unroll
        for (int e = 0; e < 4; ++e) { acc[i][e] = 0ull; xr[i][e] = 0ull; }
    const int cnt = step_geom(P, step, G * kSets, kSets * b + q).cnt;
    // ---- the input row
    fail = chain_input<DT, NCH, kFull>(P, sm, step, q, t, xr, recs, fail);
    SI_CPROF(0);                                          // the input row has arrived (and is normalised)
    if (fail) return true;
    // ---- the set's records (the loop of the unchained kernel)
    const bool noarith = (P.stream_only & 1) != 0;
    for (int i = 0; i < cnt; ++i) {
        fail |= !mbar_wait_bounded(&sfull[st], ph, cta_abort, wait_limit);
        const bool okr = !fail && smeta[st] != 0 && !noarith;   // else: h = 0 and no accumulate
        const uint4 *rr = reinterpret_cast<const uint4 *>(sring + (size_t)st * rec_bytes);
        uint4 ga[NCH], up[NCH], dn[NCH];
#pragma unroll
        for (int k2 = 0; k2 < NCH; ++k2) {
            const int c = t + kSetThreads * k2;
            if (kFull) {
                ga[k2] = rr[c]; up[k2] = rr[chunks + c]; dn[k2] = rr[2 * chunks + c];
            } else {
                const bool in = c < chunks;
                ga[k2] = in ? rr[c] : make_uint4(0, 0, 0, 0);
                up[k2] = in ? rr[chunks + c] : make_uint4(0, 0, 0, 0);
                dn[k2] = in ? rr[2 * chunks + c] : make_uint4(0, 0, 0, 0);
            }
        }
        __syncwarp();
        if (lane == 0) mbar_arrive(&sempty[st]);
        if (++st == S) { st = 0; ph ^= 1; }
        float g, u;
        {
            unsigned long long g2 = 0ull, u2 = 0ull;
#pragma unroll
            for (int k2 = 0; k2 < NCH; ++k2) { g2 = dot8p<DT>(ga[k2], xr[k2], g2); u2 = dot8p<DT>(up[k2], xr[k2], u2); }
            float lo, hi;
            unpack2(g2, lo, hi); g = lo + hi;
            unpack2(u2, lo, hi); u = lo + hi;
        }
        {
            const bool hi16 = (lane & 16) != 0;
            float keep = (hi16 ? u : g) + __shfl_xor_sync(0xFFFFFFFFu, hi16 ? g : u, 16);
            keep += __shfl_xor_sync(0xFFFFFFFFu, keep, 8);
            keep += __shfl_xor_sync(0xFFFFFFFFu, keep, 4);
            keep += __shfl_xor_sync(0xFFFFFFFFu, keep, 2);
            keep += __shfl_xor_sync(0xFFFFFFFFu, keep, 1);
            g = keep;
        }
        const uint32_t buf = recs & 1;
        if ((lane & 15) == 0) reinterpret_cast<float *>(&sm->setpart[q][buf][sw])[lane >> 4] = g;
        fail = set_barrier_or<kSetThreads>(q, fail);       // also orders the partials for the whole set
        recs ^= 1u;
        if (fail) return true;
        float gs = 0.f, us = 0.f;
        {
            const float4 *pp = reinterpret_cast<const float4 *>(sm->setpart[q][buf]);
#pragma unroll
            for (int w = 0; w < kSetWarps / 2; ++w) {
                const float4 v4 = pp[w];
                gs += v4.x; us += v4.y; gs += v4.z; us += v4.w;
            }
        }
        if (okr) {
            const float h = si_silu_mul(gs, us);
            const unsigned long long hh = pack2(h, h);
#pragma unroll
            for (int k2 = 0; k2 < NCH; ++k2) {
                unsigned long long f[4];
                unpack8p<DT>(dn[k2], f);
#pragma unroll
                for (int e = 0; e < 4; ++e) acc[k2][e] = fma2(hh, f[e], acc[k2][e]);
            }
        }
    }
    ring = (unsigned)st | (ph << 8) | ((recs & 1u) << 9);
    SI_CPROF(1);                                          // normalisation + the set's records
    // ---- the CTA's partial row
    if (q == 1) {
#pragma unroll
        for (int k2 = 0; k2 < NCH; ++k2) {
            const int c = t + kSetThreads * k2;
            if (kFull || c < chunks) {
                ulonglong2 *o = reinterpret_cast<ulonglong2 *>(comb + (size_t)c * 8);   // pairs are consecutive columns
                o[0] = make_ulonglong2(acc[k2][0], acc[k2][1]);
                o[1] = make_ulonglong2(acc[k2][2], acc[k2][3]);
            }
        }
        __syncwarp();
        if (lane == 0) mbar_arrive(&sm->accfull[0][kChainCmb]);
        SI_CPROF(2);                                      // accumulators parked
        return false;
    }
    fail |= !mbar_wait_bounded(&sm->accfull[0][kChainCmb], (uint32_t)(step & 1), cta_abort, wait_limit);
    fail = set_barrier_or<kSetThreads>(q, fail);       // all of the row or none of it
    if (fail) return true;
    SI_CPROF(2);                                          // waited for the second set
    // the sums of the two sets meet in shared memory, in column order ...
#pragma unroll
    for (int k2 = 0; k2 < NCH; ++k2) {
        const int c = t + kSetThreads * k2;
        if (kFull || c < chunks) {
            float v[8];
#pragma unroll
            for (int e = 0; e < 4; ++e) unpack2(acc[k2][e], v[2 * e], v[2 * e + 1]);
            float4 *pc = reinterpret_cast<float4 *>(comb + (size_t)c * 8);
            const float4 o0 = pc[0], o1 = pc[1];
            pc[0] = make_float4(v[0] + o0.x, v[1] + o0.y, v[2] + o0.z, v[3] + o0.w);
            pc[1] = make_float4(v[4] + o1.x, v[5] + o1.y, v[6] + o1.z, v[7] + o1.w);
        }
    }
    set_barrier_or<kSetThreads>(q, false);
    // ... and leave as {sum, tag} words, each warp instruction writing 512 consecutive bytes (a thread storing
    // the eight words of its own chunk would touch 32 lines with every instruction)
    uint4 *row = reinterpret_cast<uint4 *>(P.ll_partial + (size_t)b * d);
    for (int u = t; u < d / 2; u += kSetThreads) {
        const float2 f = reinterpret_cast<const float2 *>(comb)[u];
        st_relaxed_gpu_v4(row + u, make_uint4(__float_as_uint(f.x), tag, __float_as_uint(f.y), tag));
    }
    SI_CPROF(3);                                          // row words issued
    // every thread of the set has issued its stores: count this CTA's row as written (a hint)
    set_barrier_or<kSetThreads>(q, false);
    if (t == 0) red_add_relaxed_gpu(P.counters + (size_t)step * kCounterStride, 1u);
    SI_CPROF(7);                                          // (set 0, shares the last slot) barrier + count
    return false;
}

// Second half: all 512 consumer threads gather this CTA's columns of every CTA's row (thread = two
// columns x a class of rows, all of its rows in one round of loads, summed in row order), the class sums
// meet in shared memory and are added in a fixed order -- deterministic, whatever arrives first -- and the
// column owners add the residual, round once, write y and the {values, tag} words of the next input row.
template <int DT, int LLR>
__device__ __noinline__ bool chain_step_exchange(const Params &P, uint8_t *smem, int step) {
    const int d = P.d_model, G = gridDim.x, b = blockIdx.x;
    Smem *sm = reinterpret_cast<Smem *>(smem + P.sm_off);
    float *csum = reinterpret_cast<float *>(smem + P.csum_off);          // [columns][classes] class sums
    volatile int *cta_abort = &sm->cta_abort;
    const long long wait_limit = P.wait_cycles;
    const int ct = threadIdx.x - 32, lane = ct & 31;
    const uint32_t tag = (uint32_t)step + 1u, par = (uint32_t)(step & 1);
    const int gpc = (d / 4 + G - 1) / G, pieces = gpc * 2, classes = kConsumers / pieces;
    bool fail = false;
    const bool cprof = P.prof != nullptr && (ct & 255) == 0;
    const int q_ = ct >> 8;
    long long pt_ = cprof ? clock64() : 0;
    {
        const int piece = ct % pieces, rc = ct / pieces;
        const int col0 = b * gpc * 4 + piece * 2;
        const int n_mine = (rc < classes && col0 < d) ? (G - rc + classes - 1) / classes : 0;     // rows rc, rc + classes, ...
        const uint4 *src = reinterpret_cast<const uint4 *>(P.ll_partial + (size_t)rc * d + col0);
        const size_t stride = (size_t)classes * d / 2;             // uint4 units between this thread's rows
        fail |= !hint_wait_cta(P.counters + (size_t)step * kCounterStride, (unsigned)G, P.ctrl + 1, cta_abort, wait_limit,
                               ct == 0, &sm->accfull[0][kChainRows], par);
        SI_CPROF(4);                                      // every CTA's row counted as written
        float sx = 0.f, sy = 0.f;
        const long long t0 = clock64();
        uint32_t spins = 0;
        while (!fail) {
            // the sum counts only if every word carried this step's tag (after the hint that is the rule)
            float ax = 0.f, ay = 0.f;
            bool good = true;
            uint4 w[LLR];
#pragma unroll
            for (int i = 0; i < LLR; ++i)
                if (i < n_mine) w[i] = ld_relaxed_gpu_v4(src + stride * i);
#pragma unroll
            for (int i = 0; i < LLR; ++i)
                if (i < n_mine) {
                    good &= w[i].y == tag && w[i].w == tag;
                    ax += __uint_as_float(w[i].x); ay += __uint_as_float(w[i].z);
                }
            if (good) { sx = ax; sy = ay; break; }
            if ((++spins & 63u) == 0 && (*cta_abort || ld_relaxed_gpu(P.ctrl + 1) || clock64() - t0 > wait_limit)) fail = true;
        }
        if (rc < classes) {
            csum[(piece * 2) * classes + rc] = sx;
            csum[(piece * 2 + 1) * classes + rc] = sy;
        }
        __syncwarp();
        if (lane == 0) mbar_arrive(&sm->accfull[0][kChainXch]);
        SI_CPROF(5);                                      // rows gathered
    }
    fail |= !mbar_wait_bounded(&sm->accfull[0][kChainXch], par, cta_abort, wait_limit);
    SI_CPROF(6);                                          // all class sums in place
    const int col = ct >> 2, p4 = ct & 3, per = (classes + 3) / 4;
    const int gcol = b * gpc * 4 + col;
    const bool owner = col < pieces * 2 && gcol < d;
    float v = 0.f;
    if (owner && !fail)
        for (int c2 = p4 * per; c2 < (p4 + 1) * per && c2 < classes; ++c2) v += csum[col * classes + c2];
    v += __shfl_xor_sync(0xFFFFFFFFu, v, 1);
    v += __shfl_xor_sync(0xFFFFFFFFu, v, 2);
    uint32_t o16 = 0;
    if (owner && p4 == 0) {
        uint32_t *prev = reinterpret_cast<uint32_t *>(csum + 1024) + col;      // this thread's output of the step before
        if (P.residual) {
            const uint32_t xin = step % P.chain_len != 0 ? *prev : (uint32_t)P.x[(size_t)(step / P.chain_len) * d + gcol];
            v += si_cvt<DT>::lo(xin);
        }
        o16 = si_cvt<DT>::from_float(v);
        *prev = o16;
        if (!fail) reinterpret_cast<uint16_t *>(P.y)[(size_t)step * d + gcol] = (uint16_t)o16;
    }
    const uint32_t odd = __shfl_down_sync(0xFFFFFFFFu, o16, 4);      // the neighbouring column's value
    const bool feeds = step + 1 < P.n_steps && (step + 1) % P.chain_len != 0;       // the next step reads this row
    if (feeds && owner && p4 == 0 && (col & 1) == 0 && !fail)
        st_relaxed_gpu_v2(P.ll_x + (size_t)((step + 1) & 1) * (d / 2) + gcol / 2, make_uint2(o16 | (odd << 16), tag));
    SI_CPROF(7);                                          // column sums, y, next input row
    return fail;
}


// ------------------------------------------------------------------------------------------------
// Chained mode, split form (CH == 2): the step is cut at the activations.
//   first half   every set: h of its records from their gate and up rows (the ring carries only those),
//                each h published as one {h, tag} word;
//   second half  every CTA: all h of the step gathered (k words), then the output columns this CTA owns,
//                sum over the step's records of h x (16-byte slices of their down rows), the slices copied
//                into shared memory by two loader warps while the first half and the exchanges ran; residual,
//                rounding, y, and the {values, tag} words of the next input row.
// Column ownership: the d_model / 8 groups of eight columns (16 bytes of a down row) are dealt to the CTAs
// in order, the first (groups mod CTAs) of them getting one more; a CTA owns at most four groups.
struct SplitCols { int g0, ng; };
__device__ __forceinline__ SplitCols split_cols(int d, int G, int b) {
    const int ngrp = d / 8, base = ngrp / G, rem = ngrp % G;
    SplitCols c;
    c.ng = base + (b < rem ? 1 : 0);
    c.g0 = b * base + (b < rem ? b : rem);
    return c;
}
__device__ __forceinline__ void cp_async16(void *dst_smem, const void *src) {
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(smem_u32(dst_smem)), "l"(src) : "memory");
}
// arrival that happens by itself once every cp.async this thread has issued so far has landed (counts as
// one of the barrier's expected arrivals)
__device__ __forceinline__ void cp_async_arrive_when_landed(uint64_t *bar) {
    asm volatile("cp.async.mbarrier.arrive.noinc.shared::cta.b64 [%0];" ::"r"(smem_u32(bar)) : "memory");
}
__device__ __forceinline__ uint64_t *split_bar(Smem *sm, int which) { return &sm->accfull[0][0] + which; }

struct SplitList { int base, k, layer; };
__device__ __forceinline__ SplitList split_list(const Params &P, int step) {
    SplitList l;
    l.layer = P.step_layers ? __ldg(P.step_layers + step) : (P.n_few ? (int)P.few_layers[step] : step % P.n_layers);
    if (P.idx_offsets) {
        const int o0 = __ldg(P.idx_offsets + step), o1 = __ldg(P.idx_offsets + step + 1);
        l.base = o0; l.k = o1 - o0 < 0 ? 0 : o1 - o0;
    } else {
        l.base = P.per_layer_lists ? l.layer * P.k_fixed : step * P.k_fixed; l.k = P.k_fixed;
    }
    l.k += P.n_static;
    if (l.k > P.k_cap) l.k = P.k_cap;       // (a longer list is reported by the first half; nothing is read beyond the buffers)
    return l;
}

// The loader warps: for every step, once the second half of the step before has read the slice buffer, copy
// this CTA's 16-byte column groups of every listed record's down row into it (slice p at p * 64 bytes).
__device__ __forceinline__ void split_slice_loader(const Params &P, uint8_t *smem, Smem *sm, int lw, int lane) {
    const int d = P.d_model, G = gridDim.x;
    const SplitCols cols = split_cols(d, G, blockIdx.x);
    uint8_t *sbuf = smem + P.sbuf_off;
    bool ok = true;
    for (int step = 0; step < P.n_steps && ok; ++step) {
        if (step > 0) ok = mbar_wait_bounded(split_bar(sm, kSplitSlicesFree), (uint32_t)((step - 1) & 1), &sm->cta_abort, P.wait_cycles);
        if (!ok) break;
        const SplitList l = split_list(P, step);
        if (cols.ng > 0) {
            const char *rec = P.store_base + P.rec_off[l.layer] + (size_t)d * 4 + (size_t)cols.g0 * 16;   // down row, this CTA's columns
            const int n_loaded = P.n_loaded[l.layer];
            // A warp takes 32 list entries at a time: one coalesced load of their slots (all of a lane's loads in one
            // round first: a load per copy would put a trip to L2 in front of every copy), then four copy
            // instructions in which four neighbouring lanes fetch the (up to) 64 bytes of one record's slice, so
            // that an instruction asks for eight whole pieces instead of 32 scattered 16-byte ones.
            constexpr int kPer = kSplitKCapMax / (32 * kSplitLoaderWarps);
            int slot[kPer];
#pragma unroll
            for (int j = 0; j < kPer; ++j) {
                const int p = (j * kSplitLoaderWarps + lw) * 32 + lane;
                slot[j] = p < l.k ? (p < P.n_static ? p : __ldg(P.idx + l.base + (p - P.n_static))) : -1;
            }
            const int g = lane & 3, sub = lane >> 2;
#pragma unroll
            for (int j = 0; j < kPer; ++j) {
                const int p0 = (j * kSplitLoaderWarps + lw) * 32;
                if (p0 < l.k) {                              // (uniform over the warp)
#pragma unroll
                    for (int r = 0; r < 4; ++r) {
                        const int sl = __shfl_sync(0xFFFFFFFFu, slot[j], r * 8 + sub);
                        const int p = p0 + r * 8 + sub;
                        if (p < l.k && g < cols.ng && !(P.stream_only & 16)) {
                            const char *src = rec + (size_t)((sl >= 0 && sl < n_loaded) ? sl : 0) * ((size_t)d * 6);   // (a bad slot's h is zero)
                            cp_async16(sbuf + (size_t)p * 64 + g * 16, src + g * 16);
                        }
                    }
                }
            }
        }
        cp_async_arrive_when_landed(split_bar(sm, kSplitSlicesFull));
    }
    asm volatile("cp.async.wait_all;" ::: "memory");      // nothing of this thread may be in flight when the CTA ends
    if (!ok && lane == 0) raise_abort(P, sm, SI_ERR_TIMEOUT);
}

// First half of a step (not inlined, like the halves of the other form): input row, then for each of the
// set's records the two dot products, SiLU(g) * u, and the {h, tag} word of the record's list position.
template <int DT, int NCH, bool kFull>
__device__ __noinline__ bool split_step_gateup(const Params &P, uint8_t *smem, int step, unsigned &ring) {
    constexpr int kSets = 2, kSetWarps = 8, kSetThreads = 256;
    const int chunks = P.chunks, S = P.nstage / kSets;
    const int G = gridDim.x, b = blockIdx.x;
    Smem *sm = reinterpret_cast<Smem *>(smem + P.sm_off);
    volatile int *cta_abort = &sm->cta_abort;
    const long long wait_limit = P.wait_cycles;
    const int ct = threadIdx.x - 32, lane = ct & 31;
    const int q = ct / kSetThreads, t = ct & (kSetThreads - 1), sw = t >> 5;
    uint64_t *sfull = sm->full + q * S, *sempty = sm->empty + q * S;
    const int *smeta = sm->meta + q * S;
    const uint8_t *sring = smem + (size_t)q * S * P.stage_bytes;
    int st = (int)(ring & 0xFFu); uint32_t ph = (ring >> 8) & 1u, recs = (ring >> 9) & 1u;
    bool fail = false;
    const uint32_t tag = (uint32_t)step + 1u;
    const bool cprof = P.prof != nullptr && t == 0;
    const int q_ = q;
    long long pt_ = cprof ? clock64() : 0;

    unsigned long long xr[NCH][4];   // packed fp32 pairs
#pragma unroll
    for (int i = 0; i < NCH; ++i)
#pragma unroll
        for (int e = 0; e < 4; ++e) xr[i][e] = 0ull;
    const StepGeom geo = step_geom(P, step, G * kSets, kSets * b + q);
    if (geo.k > P.k_cap && t == 0 && P.status) atomicCAS(P.status, 0, SI_ERR_OUT_OF_RANGE);   // a list longer than the call was sized for
    fail = chain_input<DT, NCH, kFull>(P, sm, step, q, t, xr, recs, fail, split_bar(sm, kSplitInput), (unsigned)G);
    SI_CPROF(0);                                          // the input row has arrived (and is normalised)
    if (fail) return true;
    uint2 *hrow = P.ll_h + (size_t)(step & 1) * P.k_cap;
    const bool noarith = (P.stream_only & 1) != 0;
    for (int i = 0; i < geo.cnt; ++i) {
        fail |= !mbar_spin_bounded(&sfull[st], ph, cta_abort, wait_limit);
        const bool okr = !fail && smeta[st] != 0 && !noarith;   // else: h = 0
        const uint4 *rr = reinterpret_cast<const uint4 *>(sring + (size_t)st * P.stage_bytes);
        uint4 ga[NCH], up[NCH];
#pragma unroll
        for (int k2 = 0; k2 < NCH; ++k2) {
            const int c = t + kSetThreads * k2;
            const bool in = kFull || c < chunks;
            ga[k2] = in ? rr[c] : make_uint4(0, 0, 0, 0);
            up[k2] = in ? rr[chunks + c] : make_uint4(0, 0, 0, 0);
        }
        __syncwarp();
        if (lane == 0) mbar_arrive(&sempty[st]);
        if (++st == S) { st = 0; ph ^= 1; }
        float g, u;
        {
            unsigned long long g2 = 0ull, u2 = 0ull;
#pragma unroll
            for (int k2 = 0; k2 < NCH; ++k2) { g2 = dot8p<DT>(ga[k2], xr[k2], g2); u2 = dot8p<DT>(up[k2], xr[k2], u2); }
            float lo, hi;
            unpack2(g2, lo, hi); g = lo + hi;
            unpack2(u2, lo, hi); u = lo + hi;
        }
        {
            const bool hi16 = (lane & 16) != 0;
            float keep = (hi16 ? u : g) + __shfl_xor_sync(0xFFFFFFFFu, hi16 ? g : u, 16);
            keep += __shfl_xor_sync(0xFFFFFFFFu, keep, 8);
            keep += __shfl_xor_sync(0xFFFFFFFFu, keep, 4);
            keep += __shfl_xor_sync(0xFFFFFFFFu, keep, 2);
            keep += __shfl_xor_sync(0xFFFFFFFFu, keep, 1);
            g = keep;
        }
        const uint32_t buf = recs & 1;
        if ((lane & 15) == 0) reinterpret_cast<float *>(&sm->setpart[q][buf][sw])[lane >> 4] = g;
        fail = set_barrier_or<kSetThreads>(q, fail);       // also orders the partials for the whole set
        recs ^= 1u;
        if (fail) return true;
        if (t == ((i & (kSetWarps - 1)) << 5)) {             // the set's warps take turns: the sums of a record are off the other records' path
            float gs = 0.f, us = 0.f;
            const float4 *pp = reinterpret_cast<const float4 *>(sm->setpart[q][buf]);
#pragma unroll
            for (int w = 0; w < kSetWarps / 2; ++w) {
                const float4 v4 = pp[w];
                gs += v4.x; us += v4.y; gs += v4.z; us += v4.w;
            }
            const float h = okr ? si_silu_mul(gs, us) : 0.f;
            const int p = geo.first + i * (G * kSets);
            if (p < P.k_cap) st_relaxed_gpu_v2(hrow + p, make_uint2(__float_as_uint(h), tag));
        }
    }
    ring = (unsigned)st | (ph << 8) | ((recs & 1u) << 9);
    // this set's h words are on their way: count the set (a hint for the one polling thread of every CTA)
    if (t == 0) red_add_relaxed_gpu(P.counters + (size_t)step * kCounterStride, 1u);
    SI_CPROF(1);                                          // the set's records
    return false;
}

// Second half: gather every h of the step, form this CTA's output columns from the slices, finish the step.
template <int DT>
__device__ __noinline__ bool split_step_down(const Params &P, uint8_t *smem, int step) {
    const int d = P.d_model, G = gridDim.x, b = blockIdx.x;
    Smem *sm = reinterpret_cast<Smem *>(smem + P.sm_off);
    volatile int *cta_abort = &sm->cta_abort;
    const long long wait_limit = P.wait_cycles;
    const int ct = threadIdx.x - 32, lane = ct & 31;
    const uint32_t tag = (uint32_t)step + 1u, par = (uint32_t)(step & 1);
    float *hbuf = reinterpret_cast<float *>(smem + P.hbuf_off);
    const uint8_t *sbuf = smem + P.sbuf_off;
    float2 *red = reinterpret_cast<float2 *>(smem + P.red_off);           // [32 record classes][16 column pairs]
    const SplitList l = split_list(P, step);
    const SplitCols cols = split_cols(d, G, b);
    bool fail = false;
    const bool cprof = P.prof != nullptr && (ct & 255) == 0;
    const int q_ = ct >> 8;
    long long pt_ = cprof ? clock64() : 0;
    // the buffers of the step before are free once every warp (the last: the one that finishes the step) has said so
    if (step > 0) fail |= !mbar_spin_bounded(split_bar(sm, kSplitSlicesFree), (uint32_t)((step - 1) & 1), cta_abort, wait_limit);
    {
        // ---- all h of the step: two {h, tag} words per 16-byte load, polled until tagged
        const uint4 *src = reinterpret_cast<const uint4 *>(P.ll_h + (size_t)(step & 1) * P.k_cap);
        const int units = (l.k + 1) / 2;
        // (thousands of threads polling the few lines of the h row would queue up in front of the stores they
        // wait for: one thread waits for the count of sets, then every word is read once, tags checked)
        fail |= !hint_wait_cta(P.counters + (size_t)step * kCounterStride, (unsigned)(2 * G), P.ctrl + 1, cta_abort, wait_limit,
                               ct == 0, split_bar(sm, kSplitHint), par);
        const long long t0 = clock64();
        uint32_t spins = 0;
        while (!fail) {
            bool good = true;
            uint4 w[2];
#pragma unroll
            for (int i = 0; i < 2; ++i) {
                const int u = ct + kConsumers * i;
                if (u < units) w[i] = ld_relaxed_gpu_v4(src + u);
            }
#pragma unroll
            for (int i = 0; i < 2; ++i) {
                const int u = ct + kConsumers * i;
                if (u < units) {
                    good &= w[i].y == tag && (2 * u + 1 >= l.k || w[i].w == tag);
                    hbuf[2 * u] = __uint_as_float(w[i].x);
                    if (2 * u + 1 < l.k) hbuf[2 * u + 1] = __uint_as_float(w[i].z);
                }
            }
            if (good) break;
            if ((++spins & 63u) == 0 && (*cta_abort || ld_relaxed_gpu(P.ctrl + 1) || clock64() - t0 > wait_limit)) fail = true;
        }
        __syncwarp();
        if (lane == 0) mbar_arrive(split_bar(sm, kSplitH));
    }
    SI_CPROF(4);                                          // this thread's share of h gathered
    fail |= !mbar_spin_bounded(split_bar(sm, kSplitH), par, cta_abort, wait_limit);
    fail |= !mbar_spin_bounded(split_bar(sm, kSplitSlicesFull), par, cta_abort, wait_limit);
    SI_CPROF(5);                                          // all h and all slices in shared memory
    {
        // ---- lane (column group cg of eight, record class nc of 128): records nc, nc + 128, ... in ascending order,
        // one 16-byte load per record; then the eight classes of the warp by a butterfly, and one row of 32 column
        // sums per warp for the first warp to add up (all in a fixed order)
        // (four neighbouring lanes read the 64 bytes of one slice, the next four the next slice: no bank conflicts)
        const int cg = lane & 3, nc = (ct >> 5) * 8 + (lane >> 2);
        float a[8] = {0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f};
        if (cg < cols.ng && !fail) {
            const uint8_t *sp = sbuf + cg * 16;
            for (int p = nc; p < l.k; p += 128) {
                const float h = hbuf[p];
                const uint4 w = *reinterpret_cast<const uint4 *>(sp + (size_t)p * 64);
                a[0] = fmaf(h, si_cvt<DT>::lo(w.x), a[0]); a[1] = fmaf(h, si_cvt<DT>::hi(w.x), a[1]);
                a[2] = fmaf(h, si_cvt<DT>::lo(w.y), a[2]); a[3] = fmaf(h, si_cvt<DT>::hi(w.y), a[3]);
                a[4] = fmaf(h, si_cvt<DT>::lo(w.z), a[4]); a[5] = fmaf(h, si_cvt<DT>::hi(w.z), a[5]);
                a[6] = fmaf(h, si_cvt<DT>::lo(w.w), a[6]); a[7] = fmaf(h, si_cvt<DT>::hi(w.w), a[7]);
            }
        }
#pragma unroll
        for (int o = 4; o < 32; o <<= 1)
#pragma unroll
            for (int e = 0; e < 8; ++e) a[e] += __shfl_xor_sync(0xFFFFFFFFu, a[e], o);
        if (lane < 4) {
            float4 *dst = reinterpret_cast<float4 *>(reinterpret_cast<float *>(red) + (ct >> 5) * 32 + cg * 8);
            dst[0] = make_float4(a[0], a[1], a[2], a[3]);
            dst[1] = make_float4(a[4], a[5], a[6], a[7]);
        }
        __syncwarp();
        if (lane == 0) mbar_arrive(split_bar(sm, kSplitRed));
    }
    SI_CPROF(6);                                          // partial sums
    if (ct >= 32) {                                       // fifteen warps are done with the step's buffers
        if (lane == 0) mbar_arrive(split_bar(sm, kSplitSlicesFree));
        return fail;
    }
    // ---- the first warp finishes the step: the 32 record classes in ascending order, residual, rounding
    fail |= !mbar_spin_bounded(split_bar(sm, kSplitRed), par, cta_abort, wait_limit);
    // lane = column (32 of them): the sixteen warps' sums in warp order, all loads at once; even lanes then take
    // their neighbour's value and finish a pair of columns
    float vx = 0.f, vy;
    {
        const float *rf = reinterpret_cast<const float *>(red);
        float r[kConsumerWarps];
#pragma unroll
        for (int w = 0; w < kConsumerWarps; ++w) r[w] = rf[w * 32 + lane];
#pragma unroll
        for (int w = 0; w < kConsumerWarps; ++w) vx += r[w];
        vy = __shfl_down_sync(0xFFFFFFFFu, vx, 1);
    }
    const int pair = lane >> 1;
    if ((lane & 1) == 0 && pair < 4 * cols.ng && !fail) {
        const int gcol = cols.g0 * 8 + pair * 2;
        uint32_t *prev = reinterpret_cast<uint32_t *>(smem + P.prev_off) + pair;     // this thread's output of the step before
        if (P.residual) {
            const uint32_t xin = step % P.chain_len != 0 ? *prev
                                                         : *reinterpret_cast<const uint32_t *>(P.x + (size_t)(step / P.chain_len) * d + gcol);
            vx += si_cvt<DT>::lo(xin); vy += si_cvt<DT>::hi(xin);
        }
        const uint32_t o = (uint32_t)si_cvt<DT>::from_float(vx) | ((uint32_t)si_cvt<DT>::from_float(vy) << 16);
        *prev = o;
        *reinterpret_cast<uint32_t *>(reinterpret_cast<uint16_t *>(P.y) + (size_t)step * d + gcol) = o;
        if (step + 1 < P.n_steps && (step + 1) % P.chain_len != 0)       // the next step reads this row
            st_relaxed_gpu_v2(P.ll_x + (size_t)((step + 1) & 1) * (d / 2) + gcol / 2, make_uint2(o, tag));
    }
    __syncwarp();
    if (lane == 0) {
        // this CTA's words of the next input row are on their way: count the CTA (a hint), free the step's buffers
        if (step + 1 < P.n_steps && (step + 1) % P.chain_len != 0) red_add_relaxed_gpu(P.counters + (size_t)step * kCounterStride + 32, 1u);
        mbar_arrive(split_bar(sm, kSplitSlicesFree));
    }
    SI_CPROF(7);                                          // column sums, y, next input row
    return fail;
}

template <int DT, int NCH, bool kFull>
__device__ __forceinline__ void split_consumers(const Params &P, uint8_t *smem, Smem *sm) {
    unsigned ring = 0;
    bool fail = false;
    for (int step = 0; step < P.n_steps && !fail; ++step) {
        fail = split_step_gateup<DT, NCH, kFull>(P, smem, step, ring);
        if (!fail) fail = split_step_down<DT>(P, smem, step);
    }
    if (fail && (threadIdx.x & 31) == 0) raise_abort(P, sm, SI_ERR_TIMEOUT);
}

#undef SI_CPROF

template <int DT, int NCH, bool kFull, int LLR>
__device__ __forceinline__ void chained_consumers(const Params &P, uint8_t *smem, Smem *sm) {
    unsigned ring = 0;
    bool fail = false;
    for (int step = 0; step < P.n_steps && !fail; ++step) {
        fail = chain_step_records<DT, NCH, kFull>(P, smem, step, ring);
        if (!fail) fail = chain_step_exchange<DT, LLR>(P, smem, step);
    }
    if (fail && (threadIdx.x & 31) == 0) raise_abort(P, sm, SI_ERR_TIMEOUT);
}

// kProf: phase profile compiled in; kFull: every thread of a set owns NCH chunks of every row (chunks == NCH * 256);
// GRP: float4 column groups a reducer warp covers at once (its 32 lanes = GRP groups x 32/GRP row classes);
// SETW: warps per consumer set -- 8: two sets of 256 threads; 16: one set of 512 threads (rows too long for
// two rings and two hand-over buffers: thread t then owns chunks t, t + 512)
// CH: 0 = every step's input is given; 1, 2 = chained mode (every step reads the output of the step before it;
// the consumers themselves run the exchanges between the SMs and there are no reducer warps): 1 = the SMs
// exchange partial output rows, 2 = the split form that exchanges the activations (two more warps load slices)
// LLR (CH == 1): partial rows one consumer thread gathers per step (all in flight at once)
template <int DT, int NCH, bool kFull, bool kProf, int GRP, int SETW = 8, int CH = 0, int LLR = 5>
__global__ void __launch_bounds__(CH == 0 ? kThreads : (CH == 1 ? kThreadsChained : kThreadsSplit), 1)   // at most 20 warps: 96 registers per thread
si_decode_persistent_kernel(const __grid_constant__ Params P) {
    extern __shared__ __align__(128) uint8_t smem[];
    constexpr int kSets = 16 / SETW, kSetWarps = SETW, kSetThreads = SETW * 32;   // shadow the two-set defaults
    const int rec_bytes = P.d_model * 6;
    const int nstage = P.nstage;               // total over both sets (even)
    const int S = nstage / kSets;              // ring stages per consumer set
    uint8_t *ring = smem;
    float *accbuf = reinterpret_cast<float *>(smem + (size_t)nstage * rec_bytes);   // [set][d_model] hand-over to the reducers
    Smem *sm = reinterpret_cast<Smem *>(smem + P.sm_off);
    uint64_t *full = sm->full, *empty = sm->empty;
    int *meta = sm->meta;
    volatile int *cta_abort = &sm->cta_abort;

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    // Step groups: the CTAs of group `grp` run the steps grp, grp + NG, ... among themselves (their v-th
    // step is step v * NG + grp of the launch).  With short lists this divides the per-step fixed work --
    // the x copy, the hand-over, the partial rows and their reduction -- by NG for the same records.
    const int NG = P.n_groups, grp = blockIdx.x % NG;
    const int G = gridDim.x / NG, b = blockIdx.x / NG;      // CTAs of this group, index within it
    const int nv = P.n_steps > grp ? (P.n_steps - grp + NG - 1) / NG : 0;   // steps of this group
    const int Gv = G * kSets;                  // consumer sets act as virtual CTAs 2b, 2b+1 of 2G
    const int d = P.d_model, chunks = P.chunks;
    const long long wait_limit = P.wait_cycles;
    constexpr bool chained = CH != 0;          // (one step group then: the launch code sees to it)
    constexpr int xi = CH ? 0 : 1;             // ring items per step that carry the input row (chained: none, the consumers fetch it)

    if (tid == 0) {
        for (int s = 0; s < nstage; ++s) { mbar_init(&full[s], 1); mbar_init(&empty[s], kSetWarps); }
        for (int q = 0; q < kSets; ++q)
            for (int w = 0; w < kReducerWarps; ++w) { mbar_init(&sm->accfull[q][w], kSetWarps); mbar_init(&sm->accempty[q][w], 1); }
        if (CH == 1) {     // chained mode has no hand-over to reducers: three of those barriers serve its consumers
            mbar_init(&sm->accfull[0][kChainCmb], kSetWarps);               // second set's accumulators parked
            mbar_init(&sm->accfull[0][kChainXch], kConsumerWarps);          // every warp's class sums written
            mbar_init(&sm->accfull[0][kChainRows], 1);                      // the polling thread's news: every CTA's row is written
        }
        if (CH == 2) {
            mbar_init(split_bar(sm, kSplitSlicesFull), 32 * kSplitLoaderWarps);   // every loader lane's copies of the step landed
            mbar_init(split_bar(sm, kSplitSlicesFree), kConsumerWarps);           // every consumer warp done with the step's buffers
            mbar_init(split_bar(sm, kSplitH), kConsumerWarps);                    // every warp's share of h in shared memory
            mbar_init(split_bar(sm, kSplitRed), kConsumerWarps);                  // every warp's partial sums in shared memory
            mbar_init(split_bar(sm, kSplitHint), 1);                              // the polling thread's news: every set's h is written
            mbar_init(split_bar(sm, kSplitInput), 1);                             // the same for the next input row
        }
        sm->cta_abort = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncthreads();

    if (warp == 0) {
        // ------------------------------------------------------------------ producer warp
        // Each consumer set has its own ring of S stages and its own item stream: per step one
        // x item, then the records of virtual CTA 2b+set.  Two jobs share this warp.
        //  (1) Descriptor walk: half-warp h walks set h's items in order, 16 at a time (lane l
        //      takes item wn + l), loads the slot indices with one round of loads issued a
        //      full window early, and writes {source address, bytes, meta} into the set's
        //      shared-memory descriptor ring.
        //  (2) Issue: lane j < 2S owns ring stage j and issues that stage's items at its own
        //      pace: in each polling pass every lane whose stage is free arms the barrier and
        //      starts its bulk copy.
        const uint64_t policy = l2_policy_evict_first();
        const unsigned FULL = 0xFFFFFFFFu;
        const int hq = lane >> 4, hl = lane & 15;      // walker role
        const bool mine = lane < kSets * S;            // issue role
        const int iq = mine ? lane / S : 0, is = lane % S;   // (iq < kSets)
        uint32_t n = is;                               // set-ring item index this lane issues next
        uint32_t iph = 0;                              // phase parity of that item's round through the ring
        uint32_t issued = 0;
        // walker (uniform within a half-warp): item wn is item wt of step wstep (t = 0 is x)
        uint32_t wn = 0, desc_ready = 0, total = 0xFFFFFFFFu;
        int wstep = 0, wt = 0;
        unsigned long long pf_src = 0; uint32_t pf_bytes = 0; int pf_meta = 0; bool pf_valid = false;
        bool pf_pending = false;
        const int vb = kSets * b + hq;
        const int nvw = hq < kSets ? nv : 0;           // a half-warp without a set has nothing to walk
        auto prefetch_window = [&](bool doit) {
            int step = wstep, t = wt + hl;
            bool in = false;
            if (doit) {
                StepGeom g;
                in = step < nvw;
                if (in) g = step_geom(P, step * NG + grp, Gv, vb);
                while (in && t >= g.cnt + xi) {
                    t -= g.cnt + xi; ++step;
                    in = step < nvw;
                    if (in) g = step_geom(P, step * NG + grp, Gv, vb);
                }
                pf_valid = in;
                if (in) {
                    const int rs = step * NG + grp;               // step of the launch
                    const int layer = P.step_layers ? __ldg(P.step_layers + rs) : (P.n_few ? (int)P.few_layers[rs] : rs % P.n_layers);
                    if (t < xi) {
                        pf_src = (unsigned long long)(P.x + (size_t)rs * d);
                        pf_bytes = (uint32_t)d * 2; pf_meta = g.cnt;
                    } else {
                        const int lbase = P.per_layer_lists ? layer * P.k_fixed : g.base;
                        const long long pos = g.first + (long long)(t - xi) * Gv;       // position in the step: static prefix, then the list
                        const int slot = pos < P.n_static ? (int)pos : __ldg(P.idx + lbase + (pos - P.n_static));
                        const bool valid = slot >= 0 && slot < P.n_loaded[layer];
                        pf_src = (unsigned long long)(P.store_base + P.rec_off[layer] + (size_t)(valid ? slot : 0) * rec_bytes);
                        pf_bytes = valid ? P.copy_bytes : 0u; pf_meta = valid ? 1 : 0;
                    }
                }
            }
            // the walker moves on by the 16 items of this window: continue after lane 15's item
            const int s15 = __shfl_sync(FULL, step, (lane & 16) | 15), t15 = __shfl_sync(FULL, t, (lane & 16) | 15);
            const unsigned vmask = (__ballot_sync(FULL, doit && pf_valid) >> (hq * 16)) & 0xFFFFu;
            if (doit) {
                if (vmask != 0xFFFFu) total = wn + __popc(vmask);     // the item list ends in this window
                wstep = s15; wt = t15 + 1;
                pf_pending = true;
            }
        };
        auto commit_window = [&](bool doit) {
            if (doit) {
                if (pf_valid) {
                    uint4 dsc;
                    dsc.x = (uint32_t)pf_src; dsc.y = (uint32_t)(pf_src >> 32); dsc.z = pf_bytes; dsc.w = (uint32_t)pf_meta;
                    sm->desc[hq][(wn + hl) % kDescRing] = dsc;
                }
                wn += 16;
                desc_ready = wn < total ? wn : total;
                pf_pending = false;
            }
            __syncwarp();
        };
        prefetch_window(true); commit_window(true);
        prefetch_window(desc_ready < total);

        bool ok = true;
        long long t_last = clock64();
        while (true) {
            // issue lanes need their set's walker state
            const uint32_t i_ready = __shfl_sync(FULL, desc_ready, iq * 16);
            const uint32_t i_total = __shfl_sync(FULL, total, iq * 16);
            const bool have = mine && n < i_total;
            if (!__any_sync(FULL, have)) break;
            // keep each descriptor ring ahead of its set's slowest issue lane by at least a window
            uint32_t n_min = 0xFFFFFFFFu;
            for (int k = 0; k < S; ++k) {
                const uint32_t v = __shfl_sync(FULL, n, (hq < kSets ? hq : 0) * S + k);
                n_min = v < n_min ? v : n_min;
            }
            const bool do_commit = pf_pending && desc_ready - n_min <= (uint32_t)(kDescRing - 16 - kMaxStages);
            commit_window(do_commit);
            prefetch_window(do_commit && desc_ready < total);
            bool progressed = false;
            if (have && n < i_ready && !(P.withhold && blockIdx.x == 0 && iq == 0 && n == 1)) {
                const int st = iq * S + is;
                if (mbar_test_wait(&empty[st], iph ^ 1)) {
                    const uint4 dsc = sm->desc[iq][n % kDescRing];
                    meta[st] = (int)dsc.w;
                    if (dsc.z != 0 && (P.stream_only & 8)) {
                        mbar_arrive(&full[st]);
                    } else if (dsc.z != 0) {
                        mbar_arrive_expect_tx(&full[st], dsc.z);
                        bulk_g2s(ring + (size_t)st * P.stage_bytes,
                                 (const void *)(((unsigned long long)dsc.y << 32) | dsc.x), dsc.z, &full[st], policy);
                    } else {
                        if (P.status) atomicCAS(P.status, 0, SI_ERR_OUT_OF_RANGE);
                        mbar_arrive(&full[st]);
                    }
                    ++issued;
                    n += S; iph ^= 1;
                    progressed = true;
                    if (CH && n < i_ready) {
                        // chained: between two steps the ring stands still while the SMs exchange their sums;
                        // the record that will follow this one through the stage is asked into L2 meanwhile
                        const uint4 nx = sm->desc[iq][n % kDescRing];
                        if (nx.z != 0)
                            asm volatile("cp.async.bulk.prefetch.L2.global [%0], %1;"
                                         ::"l"(((unsigned long long)nx.y << 32) | nx.x), "r"(nx.z) : "memory");
                    }
                }
            }
            if (__any_sync(FULL, progressed)) {
                t_last = clock64();
            } else {
                if (*cta_abort || clock64() - t_last > wait_limit) { ok = false; break; }
                __nanosleep(100);       // nothing to issue: do not burn issue slots and power
            }
        }
        if (!ok && lane == 0) raise_abort(P, sm, SI_ERR_TIMEOUT);
        // never leave the CTA while a copy into its shared memory is still in flight
        if (mine && issued > 0) {
            const uint32_t last = n - S;           // set-ring index of this lane's last issued item
            const uint32_t ph = (last / S) & 1;
            long long t0 = clock64();
            const long long drain = wait_limit > kDrainCycles ? wait_limit : kDrainCycles;
            while (!mbar_try_wait(&full[iq * S + is], ph) && clock64() - t0 < drain) {}
        }
        return;
    }

    // Warp w runs on scheduler partition w mod 4.  The service warps (producer 0, reducers 4, 8, 12)
    // share partition 0 with one consumer warp, so that their rarely executed code does not compete
    // with four consumer warps for the partition's instruction cache and issue slots.
    const bool is_reducer = (warp & 3) == 0 && warp >= 4 && warp <= 4 * kReducerWarps;
    if constexpr (CH == 1) {
        chained_consumers<DT, NCH, kFull, LLR>(P, smem, sm);
        return;
    }
    if constexpr (CH == 2) {
        if (warp > kConsumerWarps) split_slice_loader(P, smem, sm, warp - kConsumerWarps - 1, lane);
        else split_consumers<DT, NCH, kFull>(P, smem, sm);
        return;
    }
    if (!is_reducer) {
        // ------------------------------------------------------------------ consumers
        // Two independent sets of 8 warps; set q consumes ring q.  A landed record is copied
        // into registers (3*NCH 16-byte chunks per thread) and its stage handed back at once;
        // the arithmetic then runs out of registers, so the ring is refilled while the set
        // computes.  Thread t of a set owns chunks t, t+256 of every row.
        const int cw = warp < 16 ? warp - (warp / 4 + 1) : warp - 4;   // consumer warp index 0..15
        const int ct = cw * 32 + lane;           // 0..511
        const int q = ct / kSetThreads;          // consumer set
        const int t = ct & (kSetThreads - 1);    // thread within the set
        const int sw = t >> 5;                   // warp within the set
        uint64_t *sfull = full + q * S, *sempty = empty + q * S;
        int *smeta = meta + q * S;
        uint8_t *sring = ring + (size_t)q * S * rec_bytes;
        int st = 0; uint32_t ph = 0;             // ring stage and phase parity of the set's next item
        uint32_t recs = 0;                       // records this set has handed to its barrier
        bool fail = false;
        const bool prof = kProf && P.prof != nullptr && t == 0;
        long long pf[8] = {0, 0, 0, 0, 0, 0, 0, 0}, pt = prof ? clock64() : 0;
#define SI_PROF(slot) do { if (prof) { long long now_ = clock64(); pf[slot] += now_ - pt; pt = now_; } } while (0)

        const bool noarith = (P.stream_only & 1) != 0;  // diagnostics: drain only

        for (int step = 0; step < nv && !fail; ++step) {         // the group's steps, in its own numbering
            unsigned long long xr[NCH][4], acc[NCH][4];   // packed fp32 pairs
#pragma unroll
            for (int i = 0; i < NCH; ++i)
#pragma unroll
                for (int e = 0; e < 4; ++e) { acc[i][e] = 0ull; xr[i][e] = 0ull; }
            {
                int cnt;
                {   // x item
                    fail |= !mbar_wait_bounded(&sfull[st], ph, cta_abort, wait_limit);
                    cnt = fail ? 0 : smeta[st];
                    const uint4 *xs = reinterpret_cast<const uint4 *>(sring + (size_t)st * rec_bytes);
#pragma unroll
                    for (int i = 0; i < NCH; ++i) {
                        const int c = t + kSetThreads * i;
                        if (kFull || c < chunks) unpack8p<DT>(xs[c], xr[i]);
                    }
                    __syncwarp();
                    if (lane == 0) mbar_arrive(&sempty[st]);
                    if (++st == S) { st = 0; ph ^= 1; }
                }
                // the record count steers the set's barriers: agree on it (and on failure) first
                fail = set_barrier_or<kSetThreads>(q, fail);
                if (fail) break;
                SI_PROF(0);                               // wait for x
                for (int i = 0; i < cnt; ++i) {
                    fail |= !mbar_wait_bounded(&sfull[st], ph, cta_abort, wait_limit);
                    const bool okr = !fail && smeta[st] != 0 && !noarith;   // else: h = 0 and no accumulate
                    // ---- copy this thread's chunks of the record into registers, free the stage
                    const uint4 *rr = reinterpret_cast<const uint4 *>(sring + (size_t)st * rec_bytes);
                    uint4 ga[NCH], up[NCH], dn[NCH];
#pragma unroll
                    for (int k2 = 0; k2 < NCH; ++k2) {
                        const int c = t + kSetThreads * k2;
                        if (kFull) {
                            ga[k2] = rr[c]; up[k2] = rr[chunks + c]; dn[k2] = rr[2 * chunks + c];
                        } else {
                            const bool in = c < chunks;
                            ga[k2] = in ? rr[c] : make_uint4(0, 0, 0, 0);
                            up[k2] = in ? rr[chunks + c] : make_uint4(0, 0, 0, 0);
                            dn[k2] = in ? rr[2 * chunks + c] : make_uint4(0, 0, 0, 0);
                        }
                    }
                    __syncwarp();
                    if (lane == 0) mbar_arrive(&sempty[st]);
                    if (++st == S) { st = 0; ph ^= 1; }
                    SI_PROF(1);                           // wait for the record + copy out
                    // ---- dot products: thread slice, warp butterfly (lane 0 <- gate, lane 16 <- up)
                    float g, u;
                    {
                        unsigned long long g2 = 0ull, u2 = 0ull;
#pragma unroll
                        for (int k2 = 0; k2 < NCH; ++k2) { g2 = dot8p<DT>(ga[k2], xr[k2], g2); u2 = dot8p<DT>(up[k2], xr[k2], u2); }
                        float lo, hi;
                        unpack2(g2, lo, hi); g = lo + hi;
                        unpack2(u2, lo, hi); u = lo + hi;
                    }
                    {
                        const bool hi16 = (lane & 16) != 0;
                        float keep = (hi16 ? u : g) + __shfl_xor_sync(0xFFFFFFFFu, hi16 ? g : u, 16);
                        keep += __shfl_xor_sync(0xFFFFFFFFu, keep, 8);
                        keep += __shfl_xor_sync(0xFFFFFFFFu, keep, 4);
                        keep += __shfl_xor_sync(0xFFFFFFFFu, keep, 2);
                        keep += __shfl_xor_sync(0xFFFFFFFFu, keep, 1);
                        g = keep;
                    }
                    SI_PROF(5);                           // dots + butterfly
                    // ---- exchange among the set's 8 warps (double-buffered, one barrier per record)
                    const uint32_t buf = recs & 1;
                    if ((lane & 15) == 0) reinterpret_cast<float *>(&sm->setpart[q][buf][sw])[lane >> 4] = g;
                    fail = set_barrier_or<kSetThreads>(q, fail);       // also orders the partials for the whole set
                    SI_PROF(6);                           // 8-warp exchange
                    ++recs;
                    if (fail) break;
                    float gs = 0.f, us = 0.f;
                    {
                        const float4 *pp = reinterpret_cast<const float4 *>(sm->setpart[q][buf]);
#pragma unroll
                        for (int w = 0; w < kSetWarps / 2; ++w) {
                            const float4 v4 = pp[w];
                            gs += v4.x; us += v4.y; gs += v4.z; us += v4.w;
                        }
                    }
                    if (okr) {         // a record that was not copied (slot out of range) holds stale bytes
                        const float h = si_silu_mul(gs, us);
                        const unsigned long long hh = pack2(h, h);
#pragma unroll
                        for (int k2 = 0; k2 < NCH; ++k2) {
                            unsigned long long f[4];
                            unpack8p<DT>(dn[k2], f);
#pragma unroll
                            for (int e = 0; e < 4; ++e) acc[k2][e] = fma2(hh, f[e], acc[k2][e]);
                        }
                    }
                    SI_PROF(2);                           // record arithmetic
                }
                if (fail) break;
            }

            // ---- hand this set's accumulators of the step to the reducer warps (shared memory);
            // the set is then free for the next step: it never touches global synchronisation
            {
                if (step > 0) {      // the buffer was last handed over at step - 1
                    const int ps = step - 1;
                    fail |= !mbar_wait_bounded(&sm->accempty[q][ps % kReducerWarps], (uint32_t)((ps / kReducerWarps) & 1), cta_abort, wait_limit);
                }
                if (fail) break;
                SI_PROF(4);                               // wait for the hand-over buffer
                float *ab = accbuf + (size_t)q * d;
#pragma unroll
                for (int k2 = 0; k2 < NCH; ++k2) {
                    const int c = t + kSetThreads * k2;
                    if (kFull || c < chunks) {
                        ulonglong2 *o = reinterpret_cast<ulonglong2 *>(ab + (size_t)c * 8);   // pairs are consecutive columns
                        o[0] = make_ulonglong2(acc[k2][0], acc[k2][1]);
                        o[1] = make_ulonglong2(acc[k2][2], acc[k2][3]);
                    }
                }
                __syncwarp();
                if (lane == 0) mbar_arrive(&sm->accfull[q][step % kReducerWarps]);
            }
            SI_PROF(3);                                   // accumulator hand-over
        }
#undef SI_PROF
        if (prof && q == 0) {
            for (int i = 0; i < 5; ++i) P.prof[(size_t)blockIdx.x * kProfSlots + i] = pf[i];
            P.prof[(size_t)blockIdx.x * kProfSlots + 5] = pf[5] + pf[6];
        }
        if (prof && q == 1) { P.prof[(size_t)blockIdx.x * kProfSlots + 6] = pf[4]; P.prof[(size_t)blockIdx.x * kProfSlots + 7] = pf[1]; }
        if (fail && lane == 0) raise_abort(P, sm, SI_ERR_TIMEOUT);
        return;
    }

    // -------------------------------------------------------------------------- reducer warps
    // Everything that needs other SMs lives here, off the consumers' path.  Reducer warp r handles
    // steps s = r (mod 3), in two phases:
    //  (A) when both consumer sets have handed over their accumulators of step s: add the two,
    //      store the CTA's partial y into slot s mod D of the global ring (after every CTA has
    //      finished reading the step that used the slot before), give the hand-over buffers back,
    //      and publish "partial of step s stored" (grid-scope fence + atomic);
    //  (B) reduce step sr = s - kLag, which every CTA published long ago: each lane loads rows
    //      lane, lane+32, ... of this CTA's column groups and sums them in
    //      ascending order; a warp butterfly combines the lanes (fixed order: deterministic
    //      split-K); y is written once; "partials of step sr consumed" is published.
    {
        const int r = warp / 4 - 1;                            // 0 .. kReducerWarps-1
        const bool nosync = (P.stream_only & 4) != 0;
        const int ngroups = d / 4;
        const int gpc = (ngroups + G - 1) / G;                 // <= GRP (launch check)
        const int g_valid = ngroups - b * gpc < gpc ? (ngroups - b * gpc < 0 ? 0 : ngroups - b * gpc) : gpc;
        const bool rprof = kProf && P.prof != nullptr && r == 0 && lane == 0;
        long long rp[6] = {0, 0, 0, 0, 0, 0}, rt = rprof ? clock64() : 0;
#define SI_RPROF(slot) do { if (rprof) { long long now_ = clock64(); rp[slot] += now_ - rt; rt = now_; } } while (0)
        const int bg = lane & (GRP - 1);                       // phase B: this lane's column group ...
        const int brc = lane / GRP;                            // ... and row class (rows brc, brc + kRowClasses, ...)
        constexpr int kRowClasses = 32 / GRP;
        float *const gpartial = P.partial + (size_t)grp * kPartialDepth * G * d;   // this group's ring of partial rows
        auto ctr_of = [&](int v) { return P.counters + ((size_t)v * NG + grp) * kCounterStride; };   // counters of the group's step v
        constexpr int kRowBatch = 13;                          // partial rows in flight per lane
        for (int step = r; step < nv + kLag; step += kReducerWarps) {
            int ok = 1;
            if (step < nv) {
                // ---- phase A: take each set's accumulators as soon as that set hands them over.  The
                // first set's row is stored, the second set's is added with vector reductions at L2
                // (a + b is the same whichever arrives first, so y stays bit-reproducible).
                const uint32_t par = (uint32_t)((step / kReducerWarps) & 1);
                float4 *dst = reinterpret_cast<float4 *>(gpartial + ((size_t)(step % kPartialDepth) * G + b) * d);
                const int n4 = d / 4;
                int taken = 0;                            // bit q: set q's accumulators already consumed
                // has every SM finished reading the step that used this ring slot before?  Asked
                // now, while nothing is waiting for this warp; the answer is needed after the idle wait.
                unsigned freed = (unsigned)G;
                if (lane == 0 && !nosync && step >= kPartialDepth)
                    freed = ld_acquire_gpu(ctr_of(step - kPartialDepth) + 32);
                for (int sub = 0; sub < kSets && ok; ++sub) {
                    int q = 0;
                    if (lane == 0) {
                        q = -1;
                        long long t0 = clock64();
                        while (q < 0) {
                            if (!(taken & 1) && mbar_test_wait(&sm->accfull[0][r], par)) q = 0;
                            else if (kSets > 1 && !(taken & 2) && mbar_test_wait(&sm->accfull[kSets - 1][r], par)) q = 1;
                            else {
                                if (*cta_abort || clock64() - t0 > wait_limit) break;
                                __nanosleep(200);
                            }
                        }
                        ok = q >= 0;
                        SI_RPROF(0);                      // idle: waiting for a set's hand-over
                        if (ok && sub == 0 && freed < (unsigned)G)
                            ok = counter_wait_bounded(ctr_of(step - kPartialDepth) + 32, (unsigned)G, P.ctrl + 1, cta_abort, wait_limit);
                    }
                    ok = __shfl_sync(0xFFFFFFFFu, ok, 0);
                    q = __shfl_sync(0xFFFFFFFFu, q, 0);
                    SI_RPROF(1);                          // ring slot of the partial buffer free again
                    if (!ok) break;
                    const float4 *a = reinterpret_cast<const float4 *>(accbuf + (size_t)q * d);
                    for (int i0 = 0; i0 < n4; i0 += 32 * 8) {
                        float4 u0[8];
#pragma unroll
                        for (int j = 0; j < 8; ++j) {
                            const int i = i0 + lane + 32 * j;
                            u0[j] = i < n4 ? a[i] : make_float4(0.f, 0.f, 0.f, 0.f);
                        }
#pragma unroll
                        for (int j = 0; j < 8; ++j) {
                            const int i = i0 + lane + 32 * j;
                            if (i < n4 && !nosync) {
                                if (sub == 0) st_relaxed_gpu_f4(dst + i, u0[j]);
                                else red_add_gpu_f4(dst + i, u0[j]);
                            }
                        }
                    }
                    __syncwarp();
                    if (lane == 0) mbar_arrive(&sm->accempty[q][r]);
                    taken |= 1 << q;
                    SI_RPROF(2);                          // copy the accumulators out
                }
            }
            const int sr = step - kLag;
            if (ok && sr >= 0 && !nosync) {
                // ---- phase B: lane (group bg, row class brc) sums rows brc, brc + 4, ... of its column
                // group in ascending order, kRowBatch loads in flight; two butterfly steps combine the
                // four row classes (fixed order: deterministic split-K)
                if (lane == 0)
                    ok = counter_wait_bounded(ctr_of(sr), (unsigned)G, P.ctrl + 1, cta_abort, wait_limit);
                ok = __shfl_sync(0xFFFFFFFFu, ok, 0);
                SI_RPROF(4);                              // every SM has published the step
                if (ok) {
                    float4 v = make_float4(0.f, 0.f, 0.f, 0.f);
                    const float4 *base = reinterpret_cast<const float4 *>(
                        gpartial + (size_t)(sr % kPartialDepth) * G * d + (size_t)b * gpc * 4) + bg;
                    const size_t row_stride = (size_t)d / 4;
                    if (bg < g_valid && (P.stream_only & 2) == 0) {
                        for (int r0 = brc; r0 < G; r0 += kRowClasses * kRowBatch) {
                            float4 t0[kRowBatch];
#pragma unroll
                            for (int j = 0; j < kRowBatch; ++j) {
                                const int row = r0 + kRowClasses * j;
                                t0[j] = row < G ? __ldcg(base + (size_t)row * row_stride) : make_float4(0.f, 0.f, 0.f, 0.f);
                            }
#pragma unroll
                            for (int j = 0; j < kRowBatch; ++j) { v.x += t0[j].x; v.y += t0[j].y; v.z += t0[j].z; v.w += t0[j].w; }
                        }
                    }
#pragma unroll
                    for (int o = GRP; o < 32; o <<= 1) {
                        v.x += __shfl_xor_sync(0xFFFFFFFFu, v.x, o); v.y += __shfl_xor_sync(0xFFFFFFFFu, v.y, o);
                        v.z += __shfl_xor_sync(0xFFFFFFFFu, v.z, o); v.w += __shfl_xor_sync(0xFFFFFFFFu, v.w, o);
                    }
                    if (brc == 0 && bg < g_valid) {
                        const size_t col = ((size_t)sr * NG + grp) * d + (size_t)(b * gpc + bg) * 4;
                        if (P.residual) {
                            uint2 xw = __ldg(reinterpret_cast<const uint2 *>(P.x + col));
                            v.x += si_cvt<DT>::lo(xw.x); v.y += si_cvt<DT>::hi(xw.x);
                            v.z += si_cvt<DT>::lo(xw.y); v.w += si_cvt<DT>::hi(xw.y);
                        }
                        if (P.y_f32) {
                            *reinterpret_cast<float4 *>(reinterpret_cast<float *>(P.y) + col) = v;
                        } else {
                            uint2 o;
                            o.x = (uint32_t)si_cvt<DT>::from_float(v.x) | ((uint32_t)si_cvt<DT>::from_float(v.y) << 16);
                            o.y = (uint32_t)si_cvt<DT>::from_float(v.z) | ((uint32_t)si_cvt<DT>::from_float(v.w) << 16);
                            *reinterpret_cast<uint2 *>(reinterpret_cast<uint16_t *>(P.y) + col) = o;
                        }
                    }
                }
                SI_RPROF(5);                              // load + sum the partial rows, write y
            }
            if (!ok) {
                if (lane == 0) raise_abort(P, sm, SI_ERR_TIMEOUT);
                break;
            }
            // ---- publish with one fence: "partial of this step stored" and "partials of step sr
            // consumed" (its ring slot may be overwritten once every SM has said so)
            __syncwarp();
            if (lane == 0 && !nosync) {
                __threadfence();
                if (step < nv) atomicAdd(ctr_of(step), 1u);
                if (sr >= 0 && sr + kPartialDepth < nv) atomicAdd(ctr_of(sr) + 32, 1u);
            }
            SI_RPROF(3);                                  // publish (fence + atomics)
        }
        if (rprof)
            for (int i = 0; i < 6; ++i) P.prof[(size_t)blockIdx.x * kProfSlots + 8 + i] = rp[i];
#undef SI_RPROF
    }
}

// Step groups on n_sms SMs (1 = none).  Four groups were the fastest or within noise of it for every list
// length measured (215 .. 7168 entries at d_model 4096): a step's fixed work -- the x copy, two hand-overs,
// a partial row per CTA and its share of the reduction -- is paid by a quarter of the SMs for the same
// records.  More groups would give a CTA more column groups to reduce than a warp has lanes.
inline int pick_groups(int n_sms) { return n_sms % 4 == 0 ? 4 : (n_sms % 2 == 0 ? 2 : 1); }

inline size_t smem_bytes(int d_model, int nstage, int sets = kSets) {
    return (size_t)nstage * d_model * 6 + (size_t)sets * d_model * 4 + sizeof(Smem) + 64;
}
inline int pick_stages(int d_model, int sets = kSets) {
    const size_t budget = 227 * 1024;
    if (smem_bytes(d_model, 0, sets) >= budget) return 0;
    int n = (int)((budget - smem_bytes(d_model, 0, sets)) / ((size_t)d_model * 6));
    if (n > kMaxStages) n = kMaxStages;
    return sets == 2 ? n & ~1 : n;       // split evenly between the consumer sets
}
// Rows too long for two sets (more than three chunks per thread of a 256-thread set, or no room for two
// stages per ring): one consumer set of 512 threads, thread t owning chunks t and t + 512.
inline bool wide_rows(int d_model) {
    return d_model / 8 > kSetThreads * 3 || pick_stages(d_model) < 4;
}

}  // namespace si_persist

#ifndef SI_PERSIST_KERNEL_ONLY      // (a build of single kernel instantiations, to read their register use, leaves the host side out)
inline bool si_persistent_supported(const si_store *s) {
    // thread t of a 256-thread set owns chunks t, t + 256 (, t + 512) of a row (d_model <= 6144); the
    // rings need at least two stages per consumer set beside the two hand-over buffers; a reducer warp's
    // lanes cover the float4 column groups of a CTA
    const int chunks = s->d_model / 8, G = s->num_sms;
    const int gpc = (s->d_model / 4 + G - 1) / G;
    if (s->n_layers > SI_MAX_LAYERS || gpc > si_persist::kMaxGroups) return false;
    if (si_persist::wide_rows(s->d_model))      // one set of 512 threads, two chunks per thread, at least three ring stages
        return chunks <= si_persist::kSetThreads * 4 && si_persist::pick_stages(s->d_model, 1) >= 3;
    return si_persist::pick_stages(s->d_model) >= 4 && chunks <= si_persist::kSetThreads * 3;
}

// Bytes of the partial-y ring.
inline size_t si_persistent_partial_bytes(const si_store *s) {
    return (size_t)si_persist::kPartialDepth * s->num_sms * s->d_model * 4;
}

// total_smem: dynamic shared memory of the launch when it is not the unchained layout's (0: that layout's)
template <int DT, int NCH, bool FULL, bool PROF, int GRP, int SETW = 8, int CH = 0, int LLR = 5>
inline int si_decode_persistent_launch_t(const si_persist::Params &P, int G, cudaStream_t stream, size_t extra_smem = 0,
                                         size_t total_smem = 0) {
    auto kern = si_persist::si_decode_persistent_kernel<DT, NCH, FULL, PROF, GRP, SETW, CH, LLR>;
    size_t smem = total_smem ? total_smem : si_persist::smem_bytes(P.d_model, P.nstage, 16 / SETW) + extra_smem;
    // the limit is raised to the most any instance needs (setting it is cheap, a host-side call, and
    // keeps no state here that threads or devices could disagree about)
    SI_CUDA_TRY(cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
    void *args[] = {(void *)&P};
    SI_CUDA_TRY(cudaLaunchCooperativeKernel((void *)kern, dim3(G),
                                            dim3(CH == 0 ? si_persist::kThreads : (CH == 1 ? si_persist::kThreadsChained : si_persist::kThreadsSplit)),
                                            args, smem, stream));
    return SI_OK;
}

inline int si_decode_persistent_launch(const si_store *s, int n_steps, const int32_t *layers_host,
                                       const void *x, const int32_t *idx, const int32_t *idx_offsets,
                                       int k_fixed, void *y, int y_dtype, unsigned flags, char *wsb,
                                       const si_ws_layout &ws, int32_t *status_dev, cudaStream_t stream,
                                       const si_decode_extra *ex) {
    static const si_decode_extra no_extra;
    if (!ex) ex = &no_extra;
    si_persist::Params P;
    P.store_base = s->mem;
    for (int l = 0; l < s->n_layers; ++l) { P.rec_off[l] = s->rec_off[l]; P.n_loaded[l] = s->n_loaded[l]; }
    P.n_layers = s->n_layers; P.n_steps = n_steps; P.k_fixed = k_fixed; P.d_model = s->d_model;
    const bool wide = si_persist::wide_rows(s->d_model);
    P.chunks = s->d_model / 8; P.nstage = si_persist::pick_stages(s->d_model, wide ? 1 : 2);
    P.stage_bytes = P.copy_bytes = (unsigned)s->d_model * 6;
    P.sbuf_off = P.hbuf_off = P.red_off = P.prev_off = 0; P.k_cap = 0; P.ll_h = nullptr;
    P.step_layers = nullptr; P.n_few = 0;
    // steps region: [n_steps] layer ids | control words (256 bytes) | [n_steps][64] counters
    int32_t *steps = (int32_t *)(wsb + ws.steps_off);
    if (layers_host && n_steps <= si_persist::kFewSteps) {
        P.n_few = n_steps;                      // short launch: no copy, the ids travel with the arguments
        for (int i = 0; i < n_steps; ++i) P.few_layers[i] = (unsigned char)layers_host[i];
    } else if (layers_host) {
        SI_CUDA_TRY(cudaMemcpyAsync(steps, layers_host, (size_t)n_steps * 4, cudaMemcpyHostToDevice, stream));
        P.step_layers = steps;
    }
    P.ctrl = (unsigned int *)(wsb + ws.steps_off + si_align_up((size_t)n_steps * 4, 256));
    P.counters = P.ctrl + 64;
    P.x = (const uint16_t *)x; P.idx = idx; P.idx_offsets = idx_offsets; P.y = y;
    P.y_f32 = y_dtype == SI_F32; P.residual = (flags & SI_FLAG_RESIDUAL) != 0;
    P.per_layer_lists = (flags & SI_FLAG_LIST_PER_LAYER) != 0 && !idx_offsets;
    P.n_static = ex->n_static;
    const int k_total = k_fixed + ex->n_static;       // most positions of a step
    P.partial = (float *)(wsb + ws.partial_off);
    P.status = status_dev;
    P.prof = ex->profile;
    P.stream_only = ex->skip_mask & 31;
    if (ex->ring_stages > 0 && !wide && 2 * ex->ring_stages <= P.nstage) P.nstage = 2 * ex->ring_stages;   // diagnostics: shallower rings
    P.wait_cycles = ex->wait_cycles > 0 ? ex->wait_cycles : si_persist::kWaitCycles;
    P.withhold = ex->withhold;
    P.chain_len = ex->chain_len; P.prenorm = ex->prenorm; P.norm_eps = ex->norm_eps; P.xn_out = (uint16_t *)ex->xn_out;
    int G = s->num_sms;
    if (!idx_offsets && k_total < G) G = k_total < 1 ? 1 : k_total;
    // every CTA reduces at most kMaxGroups float4 column groups
    const int g_min = (s->d_model / 4 + si_persist::kMaxGroups - 1) / si_persist::kMaxGroups;
    if (G < g_min) G = g_min;
    // Step groups: the SMs are split into groups that each take every n-th step on their own (launches of at
    // least two steps per group; a launch that uses fewer CTAs than SMs keeps one group).  The steps of a
    // stack call are independent of one another by its contract (every step's input is given), so how many
    // SMs share a step is a question of what keeps them busy: a step's fixed work -- the input row into both
    // rings, two hand-overs, a partial row per CTA and its share of the cross-SM sum -- costs about 3.4 us on all
    // SMs whatever the list's length, about 1.8 us on half and 1.0 us on a quarter of them.  Lists of up to 600
    // entries (at most four records per SM otherwise) therefore go to a quarter of the SMs, lists of up to 1100
    // to half, longer ones to all SMs, every SM working through its steps in their order; a caller who passes
    // SI_FLAG_STEPS_ANY_ORDER gets four groups whatever the length.
    int ng = 1;
    if (G == s->num_sms && ex->chain_len == 0) {
        const int forced = ex->step_groups;   // diagnostics: force a group count
        const int by_length = k_total <= 600 ? 4 : (k_total <= 1100 ? 2 : 1);
        ng = forced ? forced : ((flags & SI_FLAG_STEPS_ANY_ORDER) ? si_persist::pick_groups(s->num_sms) : by_length);
        while (ng > 1 && (s->num_sms % ng != 0 || n_steps < 2 * ng ||
                          (s->d_model / 4 + s->num_sms / ng - 1) / (s->num_sms / ng) > si_persist::kMaxGroups))
            ng >>= 1;
    }
    P.n_groups = ng;
    const int gpc = (s->d_model / 4 + G / ng - 1) / (G / ng);       // column groups per CTA -> lanes of a reducer warp
    SI_CUDA_TRY(cudaMemsetAsync(P.ctrl, 0, 256 + (size_t)n_steps * si_persist::kCounterStride * 4, stream));   // control words + counters
    P.sm_off = (unsigned)((size_t)P.nstage * s->d_model * 6 + (size_t)(wide ? 1 : 2) * s->d_model * 4);
    P.ll_partial = nullptr; P.ll_x = nullptr; P.csum_off = 0;
    // chained, split form: fixed-size slices need a CTA to own at most four groups of eight columns, every SM
    // must take part (a CTA without records still owns columns), and the step's slices must fit shared memory
    if (ex->chain_len > 0 && ex->chain_form != 1 && !wide && P.chunks <= 2 * si_persist::kSetThreads &&
        s->d_model / 8 <= 4 * s->num_sms && k_total >= 1) {
        const int Gs = s->num_sms;
        const int k_cap = (int)si_align_up((size_t)k_total, 64);
        const size_t tail = (size_t)k_cap * 64 + si_align_up((size_t)k_cap * 4, 16) + 4096 + 64 + sizeof(si_persist::Smem) + 64;
        const size_t budget = 227 * 1024;
        int nst = tail < budget ? (int)((budget - tail) / ((size_t)s->d_model * 4)) : 0;
        nst = (nst > si_persist::kMaxStages ? si_persist::kMaxStages : nst) & ~1;
        if (ex->ring_stages > 0 && 2 * ex->ring_stages <= nst) nst = 2 * ex->ring_stages;
        const size_t ll_bytes = (size_t)s->d_model * 8 + (size_t)2 * k_cap * 8;       // input-row words, then the h words
        if (nst >= 4 && k_cap <= si_persist::kSplitKCapMax && ll_bytes <= ws.partial_bytes) {
            P.nstage = nst; P.stage_bytes = P.copy_bytes = (unsigned)s->d_model * 4; P.k_cap = k_cap;
            size_t off = (size_t)nst * P.stage_bytes;
            P.sbuf_off = (unsigned)off; off += (size_t)k_cap * 64;
            P.hbuf_off = (unsigned)off; off += si_align_up((size_t)k_cap * 4, 16);
            P.red_off = (unsigned)off; off += 4096;
            P.prev_off = (unsigned)off; off += 64;
            P.sm_off = (unsigned)off; off += sizeof(si_persist::Smem) + 64;
            P.ll_x = (uint2 *)(wsb + ws.partial_off);
            P.ll_h = P.ll_x + s->d_model;
            SI_CUDA_TRY(cudaMemsetAsync(P.ll_x, 0, ll_bytes, stream));
            const bool full_s = P.chunks == ((P.chunks + 255) / 256) * 256;
#define SI_PLS(DT, N, F) si_decode_persistent_launch_t<DT, N, F, false, 8, 8, 2>(P, Gs, stream, 0, off)
#define SI_PLS2(DT) (P.chunks <= 256 ? (full_s ? SI_PLS(DT, 1, true) : SI_PLS(DT, 1, false)) : (full_s ? SI_PLS(DT, 2, true) : SI_PLS(DT, 2, false)))
            return s->dtype == SI_BF16 ? SI_PLS2(SI_BF16) : SI_PLS2(SI_F16);
#undef SI_PLS2
#undef SI_PLS
        }
        if (ex->chain_form == 2) return SI_ERR_UNSUPPORTED;       // the split form was asked for and does not fit
    }
    if (ex->chain_len > 0) {
        // chained: two consumer sets only; the tagged exchange words live in the partial-row area and start at zero
        if (wide) return SI_ERR_UNSUPPORTED;
        const int pieces = gpc * 2, classes = si_persist::kConsumers / pieces;
        const int rpt = classes < 1 ? si_persist::kLLRows + 1 : (G + classes - 1) / classes;   // partial rows a consumer thread gathers
        if (rpt > si_persist::kLLRows) return SI_ERR_UNSUPPORTED;
        const size_t ll_bytes = (size_t)G * s->d_model * 8 + (size_t)s->d_model * 8;
        if (ll_bytes > ws.partial_bytes) return SI_ERR_NOMEM;
        P.ll_partial = (uint2 *)(wsb + ws.partial_off);
        P.ll_x = P.ll_partial + (size_t)G * s->d_model;
        SI_CUDA_TRY(cudaMemsetAsync(P.ll_partial, 0, ll_bytes, stream));
        // class sums (at most 4 KB) and the column owners' last outputs (512 B): in the second hand-over buffer where that
        // is large enough, else behind everything
        const size_t base = (size_t)P.nstage * s->d_model * 6;
        size_t extra = 0;
        if ((size_t)s->d_model * 4 >= 4096 + 512) P.csum_off = (unsigned)(base + (size_t)s->d_model * 4);
        else { P.csum_off = (unsigned)si_align_up(si_persist::smem_bytes(s->d_model, P.nstage), 16); extra = 4096 + 512 + 16; }
        const int set_threads_c = si_persist::kSetThreads;
        const int nch_c = (P.chunks + set_threads_c - 1) / set_threads_c;
        const bool full_c = P.chunks == nch_c * set_threads_c;
#define SI_PLC(DT, N, F) (rpt <= 2 ? si_decode_persistent_launch_t<DT, N, F, false, 8, 8, 1, 2>(P, G, stream, extra)   \
                          : rpt <= 5 ? si_decode_persistent_launch_t<DT, N, F, false, 8, 8, 1, 5>(P, G, stream, extra) \
                                     : si_decode_persistent_launch_t<DT, N, F, false, 8, 8, 1, si_persist::kLLRows>(P, G, stream, extra))
#define SI_PLC2(DT) (nch_c <= 1 ? (full_c ? SI_PLC(DT, 1, true) : SI_PLC(DT, 1, false))   \
                     : nch_c <= 2 ? (full_c ? SI_PLC(DT, 2, true) : SI_PLC(DT, 2, false)) \
                                  : (full_c ? SI_PLC(DT, 3, true) : SI_PLC(DT, 3, false)))
        return s->dtype == SI_BF16 ? SI_PLC2(SI_BF16) : SI_PLC2(SI_F16);
#undef SI_PLC2
#undef SI_PLC
    }
    // NCH: 16-byte chunks per thread and row (256 threads per consumer set)
    const int set_threads = wide ? 2 * si_persist::kSetThreads : si_persist::kSetThreads;
    const int nch = (P.chunks + set_threads - 1) / set_threads;
    const bool full = P.chunks == nch * set_threads;
    // the phase profile is a separate instantiation: the production kernel carries no clock reads
#define SI_PL3(DT, N, F, PR) (gpc <= 8 ? si_decode_persistent_launch_t<DT, N, F, PR, 8>(P, G, stream)    \
                              : gpc <= 16 ? si_decode_persistent_launch_t<DT, N, F, PR, 16>(P, G, stream) \
                                          : si_decode_persistent_launch_t<DT, N, F, PR, 32>(P, G, stream))
#define SI_PL2(DT, N, F) (P.prof ? SI_PL3(DT, N, F, true) : SI_PL3(DT, N, F, false))
    // three chunks per thread (d_model 4104 .. 6144): no phase profile, 16 or 32 column groups per warp
#define SI_PL_W(DT, F) (gpc <= 16 ? si_decode_persistent_launch_t<DT, 3, F, false, 16>(P, G, stream) \
                                  : si_decode_persistent_launch_t<DT, 3, F, false, 32>(P, G, stream))
#define SI_PL(DT) (nch <= 1 ? (full ? SI_PL2(DT, 1, true) : SI_PL2(DT, 1, false))     \
                   : nch <= 2 ? (full ? SI_PL2(DT, 2, true) : SI_PL2(DT, 2, false)) \
                              : (full ? SI_PL_W(DT, true) : SI_PL_W(DT, false)))
    // wide rows: one set of 16 warps, two chunks per thread, no phase profile
#define SI_PL_X(DT, F) (gpc <= 16 ? si_decode_persistent_launch_t<DT, 2, F, false, 16, 16>(P, G, stream) \
                                  : si_decode_persistent_launch_t<DT, 2, F, false, 32, 16>(P, G, stream))
    if (wide) return s->dtype == SI_BF16 ? (full ? SI_PL_X(SI_BF16, true) : SI_PL_X(SI_BF16, false))
                                         : (full ? SI_PL_X(SI_F16, true) : SI_PL_X(SI_F16, false));
#undef SI_PL_X
    return s->dtype == SI_BF16 ? SI_PL(SI_BF16) : SI_PL(SI_F16);
#undef SI_PL2
#undef SI_PL3
#undef SI_PL_W
#undef SI_PL
}
#endif  // SI_PERSIST_KERNEL_ONLY
