// Persistent batch-1 selective decode for sm_100a.
//
// One CTA per SM runs any number of (token, layer) steps in a single launch.  Each CTA has
// three roles:
//   * warp 0 (producer) walks the CTA's share of every step's active list and streams each
//     selected neuron record -- 6*d_model contiguous bytes: gate row | up row | down row --
//     from HBM into a shared-memory ring with one bulk async copy (cp.async.bulk, completion
//     on an mbarrier).  Each lane owns one ring stage and issues that stage's items on its
//     own, so there are as many independent issue streams as stages.  The ring runs ahead
//     across step boundaries, so HBM never waits for the arithmetic or for the cross-SM
//     reduction;
//   * warps 1..16 (consumers, 512 threads) take records four at a time.  For the dot
//     products warp (r, q) handles record r of the batch over column quarter q with its
//     slice of x in registers (five shuffles per warp, no CTA-wide exchange beyond 32
//     floats); the warps meet on a split-phase mbarrier and -- one batch later, so the
//     barrier latency is hidden -- every thread combines the quarters, applies SiLU(g)*u and
//     accumulates h * down for its 8*NCH output columns into fp32 registers.  At the end of
//     a step the CTA stores its partial y into a ring of D partial buffers and goes
//     straight on to the next step;
//   * warps 17..18 (reducers, alternating steps) publish "step s written" on a per-step counter, wait until all
//     CTAs have done so, and reduce this CTA's slice of columns over the partials in CTA
//     order (deterministic split-K), writing y once.  The reduction of step s overlaps the
//     record stream of steps s+1.. ; a second per-step counter lets a partial buffer be
//     reused only after every CTA has finished reading it.
// List position p of step s goes to CTA (p + rot_s) mod G, rot_s = (number of list entries
// before step s) mod G, so records are dealt round-robin across steps and no SM is
// persistently the one with an extra record.
//
// Every wait is bounded: on expiry the kernel records SI_ERR_TIMEOUT, raises a grid-wide
// abort flag, lets its outstanding copies land and returns.
#pragma once

#include "si_common.cuh"

#define SI_MAX_LAYERS 128

namespace si_persist {

constexpr int kConsumers = 512;
constexpr int kConsumerWarps = kConsumers / 32;
static_assert(kConsumerWarps == 16, "consumer warps are arranged as 4 records x 4 column quarters");
constexpr int kThreads = 32 + kConsumers + 64;    // producer warp, consumers, signalling warp, watcher warp
constexpr int kFlagRing = 8;                      // per-step shared-memory flags kept for this many steps
constexpr int kCounterStride = 64;                // uint32 per step: written at +0, reduced at +32 (own 128-byte lines)
constexpr int kMaxStages = 16;
constexpr int kDescRing = 128;                    // copy descriptors kept ahead of the issue lanes
constexpr int kPartialDepth = 6;                  // D: partial-y buffers in flight
constexpr int kLag = 2;                           // a step's cross-SM reduction starts this many steps later
constexpr long long kWaitCycles = 4000000000ll;   // ~2 s at 1.9 GHz

struct Params {
    const char *store_base;
    unsigned long long rec_off[SI_MAX_LAYERS];
    int n_loaded[SI_MAX_LAYERS];
    int n_layers, n_steps, k_fixed, d_model, chunks, nstage;
    const int32_t *step_layers;   // device int32 [n_steps] or nullptr (step mod n_layers)
    const uint16_t *x;            // [n_steps, d_model]
    const int32_t *idx;           // [n_steps, k_fixed] or CSR payload
    const int32_t *idx_offsets;   // CSR [n_steps + 1] or nullptr
    void *y;
    int y_f32, residual;
    float *partial;               // [D][G][d_model]
    unsigned int *ctrl;           // [1] abort flag (zero at launch)
    unsigned int *counters;       // [n_steps][kCounterStride], zero at launch: +0 "written" = CTAs that
                                  // stored their partial of the step, +32 "reduced" = CTAs that finished
                                  // reading the step's partials
    int32_t *status;
    long long *prof;              // optional phase profile: int64 [G][8] cycle counters, or nullptr
    int stream_only;              // diagnostics bit mask (see si_debug_decode_stream_only)
    int prefetch_rounds;          // L2 prefetch distance in ring rounds (0 = off)
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
__device__ __forceinline__ bool mbar_wait_bounded(uint64_t *bar, uint32_t parity, volatile int *cta_abort) {
    if (mbar_try_wait(bar, parity)) return true;
    long long t0 = clock64();
    while (true) {
        for (int i = 0; i < 64; ++i)
            if (mbar_try_wait(bar, parity)) return true;
        if (*cta_abort) return false;
        if (clock64() - t0 > kWaitCycles) return false;
    }
}
// Warp-level wait: only lane 0 polls the barrier (32 lanes polling one barrier word cost 32
// shared-memory barrier operations per probe), the warp then reconverges; the shuffle orders the
// other lanes' subsequent reads after lane 0's acquire.
__device__ __forceinline__ bool mbar_wait_warp(uint64_t *bar, uint32_t parity, volatile int *cta_abort, int lane) {
    int ok = 1;
    if (lane == 0) ok = mbar_wait_bounded(bar, parity, cta_abort) ? 1 : 0;
    return __shfl_sync(0xFFFFFFFFu, ok, 0) != 0;
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
                                                     volatile int *cta_abort) {
    if (ld_acquire_gpu(ctr) >= target) return true;
    long long t0 = clock64();
    while (true) {
        for (int i = 0; i < 16; ++i) {
            if (ld_acquire_gpu(ctr) >= target) return true;
            __nanosleep(64);
        }
        if (*cta_abort || ld_relaxed_gpu(grid_abort)) return false;
        if (clock64() - t0 > kWaitCycles) return false;
    }
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

// Warp reduction of four values with six shuffles: afterwards lane 0 holds sum(v0), lane 8
// sum(v1), lane 16 sum(v2), lane 24 sum(v3).  Fixed order, hence deterministic.
__device__ __forceinline__ float warp_sum4(float v0, float v1, float v2, float v3, int lane) {
    const bool hi16 = (lane & 16) != 0;
    float s0 = hi16 ? v0 : v2, s1 = hi16 ? v1 : v3;
    float k0 = hi16 ? v2 : v0, k1 = hi16 ? v3 : v1;
    k0 += __shfl_xor_sync(0xFFFFFFFFu, s0, 16);
    k1 += __shfl_xor_sync(0xFFFFFFFFu, s1, 16);
    const bool hi8 = (lane & 8) != 0;
    float s = hi8 ? k0 : k1, k = hi8 ? k1 : k0;
    k += __shfl_xor_sync(0xFFFFFFFFu, s, 8);
    k += __shfl_xor_sync(0xFFFFFFFFu, k, 4);
    k += __shfl_xor_sync(0xFFFFFFFFu, k, 2);
    k += __shfl_xor_sync(0xFFFFFFFFu, k, 1);
    return k;
}

// Per-step list geometry, identical in producer and consumers.
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
    int rot = (int)(before % G);
    g.first = (b - rot + G) % G;
    g.cnt = g.k > g.first ? (g.k - g.first + G - 1) / G : 0;
    return g;
}

struct Smem {
    uint64_t full[kMaxStages];
    uint64_t empty[kMaxStages];
    uint64_t redbar[2];            // consumer warps' partial dot products are in part[buf]
    uint64_t stepbar[kPartialDepth];   // consumers stored the partial y of step s (slot s mod D)
    int meta[kMaxStages];
    uint4 desc[kDescRing];         // {src lo, src hi, bytes (0: nothing to copy), meta}
    float part[2][2 * kConsumerWarps];   // [buf][record*8 + quarter*2 + (gate|up)]
    uint64_t ybar[2];              // redy[buf] is complete
    uint64_t pubbar[kFlagRing];    // every CTA has published its partial of step s (slot s mod ring)
    uint64_t freebar[kFlagRing];   // every CTA has finished reading the partials of step s
    float4 redy[2][64];            // warp-level sums of a step's column groups
    volatile int cta_abort;
};

__device__ __forceinline__ void raise_abort(const Params &P, Smem *sm, int code) {
    if (!sm->cta_abort) {
        sm->cta_abort = 1;
        if (P.status) atomicCAS(P.status, 0, code);
        atomicExch(P.ctrl + 1, 1u);
    }
}

template <int DT, int NCH, int NQ, int NRL>
__global__ void __launch_bounds__(kThreads, 1)   // 18 warps: at most 96 registers per thread
si_decode_persistent_kernel(const __grid_constant__ Params P) {
    extern __shared__ __align__(128) uint8_t smem[];
    const int rec_bytes = P.d_model * 6;
    const int nstage = P.nstage;
    uint8_t *ring = smem;
    Smem *sm = reinterpret_cast<Smem *>(smem + (size_t)nstage * rec_bytes);
    uint64_t *full = sm->full, *empty = sm->empty;
    int *meta = sm->meta;
    volatile int *cta_abort = &sm->cta_abort;

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int G = gridDim.x, b = blockIdx.x;
    const int d = P.d_model, chunks = P.chunks;

    if (tid == 0) {
        for (int s = 0; s < nstage; ++s) { mbar_init(&full[s], 1); mbar_init(&empty[s], kConsumerWarps); }
        mbar_init(&sm->redbar[0], kConsumerWarps); mbar_init(&sm->redbar[1], kConsumerWarps);
        for (int s = 0; s < kPartialDepth; ++s) mbar_init(&sm->stepbar[s], kConsumerWarps);
        mbar_init(&sm->ybar[0], kConsumerWarps); mbar_init(&sm->ybar[1], kConsumerWarps);
        for (int s = 0; s < kFlagRing; ++s) { mbar_init(&sm->pubbar[s], 1); mbar_init(&sm->freebar[s], 1); }
        sm->cta_abort = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncthreads();

    if (warp == 0) {
        // ------------------------------------------------------------------ producer warp
        // Two jobs share this warp.
        //  (1) Descriptor walk: the warp walks the CTA's items in order, 32 at a time (lane l
        //      takes item wn + l), loads the slot indices with one coalesced round of loads
        //      issued a full window early, and writes {source address, bytes, meta} into a
        //      shared-memory descriptor ring.
        //  (2) Issue: lane j < nstage owns ring stage j and issues every item n = j (mod
        //      nstage) at its own pace: in each polling pass every lane whose stage is free
        //      arms the barrier and starts its bulk copy.  One thread issuing alone cannot keep
        //      an SM's share of HBM busy; here as many lanes issue together as stages are free.
        const uint64_t policy = l2_policy_evict_first();
        const bool mine = lane < nstage;
        uint32_t n = lane;             // ring item index this lane issues next
        uint32_t issued = 0;
        // walker: item wn is item wt of step wstep (t = 0 is x, t >= 1 is record t - 1)
        uint32_t wn = 0, desc_ready = 0, total = 0xFFFFFFFFu;
        int wstep = 0, wt = 0;
        // per-lane prefetched descriptor of item wn + lane
        unsigned long long pf_src = 0; uint32_t pf_bytes = 0; int pf_meta = 0; bool pf_valid = false;
        bool pf_pending = false;       // a window has been prefetched and not yet committed
        auto prefetch_window = [&]() {
            // lane l: locate item (wstep, wt + l)
            int step = wstep, t = wt + lane;
            StepGeom g;
            bool in = step < P.n_steps;
            if (in) g = step_geom(P, step, G, b);
            while (in && t > g.cnt) {
                t -= g.cnt + 1; ++step;
                in = step < P.n_steps;
                if (in) g = step_geom(P, step, G, b);
            }
            pf_valid = in;
            if (in) {
                const int layer = P.step_layers ? __ldg(P.step_layers + step) : step % P.n_layers;
                if (t == 0) {
                    pf_src = (unsigned long long)(P.x + (size_t)step * d);
                    pf_bytes = (uint32_t)d * 2; pf_meta = g.cnt;
                } else {
                    const int slot = __ldg(P.idx + g.base + g.first + (long long)(t - 1) * G);
                    const bool valid = slot >= 0 && slot < P.n_loaded[layer];
                    pf_src = (unsigned long long)(P.store_base + P.rec_off[layer] + (size_t)(valid ? slot : 0) * rec_bytes);
                    pf_bytes = valid ? (uint32_t)rec_bytes : 0u; pf_meta = valid ? 1 : 0;
                }
            }
            // the walker moves on by the 32 items of this window: continue after lane 31's item
            const int s31 = __shfl_sync(0xFFFFFFFFu, step, 31), t31 = __shfl_sync(0xFFFFFFFFu, t, 31);
            const unsigned vmask = __ballot_sync(0xFFFFFFFFu, pf_valid);
            if (vmask != 0xFFFFFFFFu) total = wn + __popc(vmask);     // the list of items ends in this window
            wstep = s31; wt = t31 + 1;
            pf_pending = true;
        };
        auto commit_window = [&]() {
            if (pf_valid) {
                uint4 dsc;
                dsc.x = (uint32_t)pf_src; dsc.y = (uint32_t)(pf_src >> 32); dsc.z = pf_bytes; dsc.w = (uint32_t)pf_meta;
                sm->desc[(wn + lane) % kDescRing] = dsc;
            }
            __syncwarp();
            wn += 32;
            desc_ready = wn < total ? wn : total;
            pf_pending = false;
        };
        prefetch_window(); commit_window();
        if (desc_ready < total) prefetch_window();

        bool ok = true;
        long long t_last = clock64();
        while (true) {
            const bool have = mine && n < total;
            if (!__any_sync(0xFFFFFFFFu, have)) break;
            // keep the descriptor ring ahead of the slowest lane by at least one window
            const uint32_t n_min = __reduce_min_sync(0xFFFFFFFFu, mine ? n : 0xFFFFFFFFu);
            if (pf_pending && desc_ready - n_min <= kDescRing - 32 - kMaxStages) {
                commit_window();
                if (desc_ready < total) prefetch_window();
            }
            bool progressed = false;
            if (have && n < desc_ready) {
                const int st = lane; const uint32_t ph = (n / nstage) & 1;
                if (mbar_test_wait(&empty[st], ph ^ 1)) {
                    const uint4 dsc = sm->desc[n % kDescRing];
                    meta[st] = (int)dsc.w;
                    if (dsc.z != 0) {
                        mbar_arrive_expect_tx(&full[st], dsc.z);
                        const void *src = (const void *)(((unsigned long long)dsc.y << 32) | dsc.x);
                        if (P.stream_only & 8) {   // diagnostics: uniformly random records of layer 0
                            unsigned long long r = ((unsigned long long)n * 2654435761ull + (unsigned long long)b * 40503ull) % (unsigned long long)P.n_loaded[0];
                            src = P.store_base + P.rec_off[0] + r * rec_bytes;
                        }
                        if (P.stream_only & 16)
                            asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                                         ::"r"(smem_u32(ring + (size_t)st * rec_bytes)), "l"(src), "r"(dsc.z), "r"(smem_u32(&full[st])) : "memory");
                        else
                        bulk_g2s(ring + (size_t)st * rec_bytes, src, dsc.z, &full[st], policy);
                    } else {
                        if (P.status) atomicCAS(P.status, 0, SI_ERR_OUT_OF_RANGE);
                        mbar_arrive(&full[st]);
                    }
                    ++issued;
                    // pull a later item of this lane from HBM into L2 now, so that its copy into
                    // shared memory later pays the L2 latency rather than the loaded-HBM latency
                    const uint32_t npf = n + (uint32_t)(P.prefetch_rounds * nstage);
                    if (P.prefetch_rounds > 0 && npf < desc_ready) {
                        const uint4 pd = sm->desc[npf % kDescRing];
                        if (pd.z != 0)
                            asm volatile("cp.async.bulk.prefetch.L2.global [%0], %1;"
                                         ::"l"(((unsigned long long)pd.y << 32) | pd.x), "r"(pd.z) : "memory");
                    }
                    n += nstage;
                    progressed = true;
                }
            }
            if (__any_sync(0xFFFFFFFFu, progressed)) {
                t_last = clock64();
            } else if (*cta_abort || clock64() - t_last > kWaitCycles) {
                ok = false;
                break;
            }
        }
        if (!ok && lane == 0) raise_abort(P, sm, SI_ERR_TIMEOUT);
        // never leave the CTA while a copy into its shared memory is still in flight
        if (mine && issued > 0) {
            const uint32_t last = n - nstage;      // ring index of this lane's last issued item
            const uint32_t ph = (last / nstage) & 1;
            long long t0 = clock64();
            while (!mbar_try_wait(&full[lane], ph) && clock64() - t0 < kWaitCycles) {}
        }
        return;
    }

    if (warp <= kConsumerWarps) {
        // ------------------------------------------------------------------ consumers
        // Records are taken in batches of four.  Dot products: consumer warp (wr, wq) handles
        // record wr of the batch over column quarter wq, with its slice of x in registers,
        // so the four records' dots run in independent warps and need no CTA-wide exchange
        // beyond 32 floats.  Down projection: thread ct owns output columns of chunk
        // ct + 512*q and accumulates all four records.
        const int ct = tid - 32;                 // 0..511
        const int cw = ct >> 5;                  // consumer warp 0..15
        const int wr = cw >> 2, wq = cw & 3;
        const int cq = chunks >> 2;              // 16-byte chunks per column quarter
        uint32_t n = 0;                          // ring item counter
        uint32_t batches = 0;                    // batches handed to the split-phase barrier so far
        bool fail = false;
        if (P.stream_only & 32) {   // diagnostics: drain the ring item by item, nothing else
            for (int step = 0; step < P.n_steps; ++step) {
                int st = n % nstage; uint32_t ph = (n / nstage) & 1;
                if (!mbar_wait_bounded(&full[st], ph, cta_abort)) return;
                const int cnt = meta[st];
                __syncwarp();
                if (lane == 0) mbar_arrive(&empty[st]);
                ++n;
                for (int i = 0; i < cnt; ++i) {
                    st = n % nstage; ph = (n / nstage) & 1;
                    if (!mbar_wait_bounded(&full[st], ph, cta_abort)) return;
                    __syncwarp();
                    if (lane == 0) mbar_arrive(&empty[st]);
                    ++n;
                }
            }
            return;
        }
        const bool prof = P.prof != nullptr && ct == 0;
        long long pf[8] = {0, 0, 0, 0, 0, 0, 0, 0}, pt = prof ? clock64() : 0;
#define SI_PROF(slot) do { if (prof) { long long now_ = clock64(); pf[slot] += now_ - pt; pt = now_; } } while (0)

        // split-K reduction geometry: this CTA reduces column groups [b*gpc, (b+1)*gpc) of
        // every step; TPG threads share one group, thread pl of them sums partials pl, pl+TPG, ...
        const int ngroups = d / 4;                 // float4 column groups
        const int gpc = (ngroups + G - 1) / G;     // groups per CTA
        int GP = 1; while (GP < gpc) GP <<= 1;     // padded to a power of two (<= 512 by the launch check)
        const int TPG = kConsumers / GP;
        const int WL = TPG < 32 ? TPG : 32;        // lanes of one warp that share a group
        const int rgi = ct / TPG, rpl = ct % TPG;
        const int rgrp = b * gpc + rgi;
        const bool ractive = rgi < gpc && rgrp < ngroups;
        const bool nosync = (P.stream_only & 4) != 0;   // diagnostics: no cross-CTA exchange at all

        // Steps n_steps .. n_steps + kLag - 1 are flush iterations: no records, they only finish
        // the reductions that are still in flight.
        for (int step = 0; step <= P.n_steps + kLag && !fail; ++step) {
            const bool real = step < P.n_steps;
            // ---- [A0] write y of step (step-1-kLag): its group sums are in redy[(step-1) & 1]
            if (step - 1 >= kLag && !(P.stream_only & 128)) {
                const int sy = step - 1 - kLag, yb = (step - 1 - kLag) & 1;
                fail |= !mbar_wait_warp(&sm->ybar[yb], (uint32_t)(((step - 1 - kLag) >> 1) & 1), cta_abort, lane);
                if (!fail && ct < GP && ct < gpc && b * gpc + ct < ngroups) {
                    const int W = TPG / WL;
                    float4 v = sm->redy[yb][ct * W];
                    for (int w = 1; w < W; ++w) {
                        const float4 t4 = sm->redy[yb][ct * W + w];
                        v.x += t4.x; v.y += t4.y; v.z += t4.z; v.w += t4.w;
                    }
                    const size_t col = (size_t)sy * d + (size_t)(b * gpc + ct) * 4;
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
            if (step == P.n_steps + kLag || fail) break;

            // ---- [A1] start the reduction of step sr = step - kLag: every CTA has published its
            // partial of that step long ago; the loads fly while this step's records are processed
            float4 rv[NRL];
#pragma unroll
            for (int j = 0; j < NRL; ++j) rv[j] = make_float4(0.f, 0.f, 0.f, 0.f);
            if (step >= kLag && !(P.stream_only & 128)) {
                const int sr = step - kLag;
                if (!nosync) fail |= !mbar_wait_warp(&sm->pubbar[sr % kFlagRing], (sr / kFlagRing) & 1, cta_abort, lane);
                if (fail) break;
                if (ractive && (P.stream_only & 6) == 0) {
                    const float *col = P.partial + (size_t)(sr % kPartialDepth) * G * d + (size_t)rgrp * 4;
#pragma unroll
                    for (int j = 0; j < NRL; ++j) {
                        const int gg = rpl + TPG * j;
                        if (gg < G) rv[j] = __ldcg(reinterpret_cast<const float4 *>(col + (size_t)gg * d));
                    }
                }
            }
            SI_PROF(5);                                   // reduction: wait for publication, issue loads

            float xr[NQ][8], acc[NCH][8];
            int cnt = 0;
#pragma unroll
            for (int q = 0; q < NCH; ++q)
#pragma unroll
                for (int e = 0; e < 8; ++e) acc[q][e] = 0.f;
            if (real) {
                int st = n % nstage; uint32_t ph = (n / nstage) & 1;
                fail |= !mbar_wait_warp(&full[st], ph, cta_abort, lane);
                cnt = fail ? 0 : meta[st];
                const uint4 *xs = reinterpret_cast<const uint4 *>(ring + (size_t)st * rec_bytes) + wq * cq;
#pragma unroll
                for (int j = 0; j < NQ; ++j) {
                    int c = lane + 32 * j;
                    uint4 v = c < cq ? xs[c] : make_uint4(0, 0, 0, 0);
                    unpack8<DT>(v, xr[j]);
                }
                __syncwarp();
                if (lane == 0) mbar_arrive(&empty[st]);
                ++n;
            }
            SI_PROF(0);                                   // wait for x

            // software pipeline over batches: the dot products of batch i are handed to the
            // warps' barrier and finished (summed, SiLU, down accumulate) while batch i+1 loads
            uint4 dnp[4][NCH];                            // down chunks of the pending batch
            bool pend = false;
            uint32_t pbatch = 0;
            auto finish_pending = [&]() {
                const uint32_t buf = pbatch & 1, par = (pbatch >> 1) & 1;
                fail |= !mbar_wait_warp(&sm->redbar[buf], par, cta_abort, lane);
                // part[buf] holds 32 floats, index r*8 + quarter*2 + (0: gate, 1: up)
                float v = reinterpret_cast<const float *>(sm->part[buf])[lane];
                v += __shfl_xor_sync(0xFFFFFFFFu, v, 2);
                v += __shfl_xor_sync(0xFFFFFFFFu, v, 4);
                const float u = __shfl_xor_sync(0xFFFFFFFFu, v, 1);
                const float hh = si_silu_mul(v, u);       // meaningful on lanes 0, 8, 16, 24
                float h[4];
#pragma unroll
                for (int r = 0; r < 4; ++r) h[r] = __shfl_sync(0xFFFFFFFFu, hh, r * 8);
#pragma unroll
                for (int q = 0; q < NCH; ++q) {
#pragma unroll
                    for (int r = 0; r < 4; ++r) {
                        float f[8];
                        unpack8<DT>(dnp[r][q], f);
#pragma unroll
                        for (int e = 0; e < 8; ++e) acc[q][e] = fmaf(h[r], f[e], acc[q][e]);
                    }
                }
            };

            for (int i = 0; i < cnt && !fail; i += 4) {
                const int nb = cnt - i < 4 ? cnt - i : 4;
                // the previous batch's warps have all published their dot products by now (or
                // will within a few cycles): finish it before its down chunks are overwritten
                if (pend && !(P.stream_only & 64)) finish_pending();
                // ---- take the batch's records one by one as they land; a stage is handed
                // back as soon as this warp has what it needs from it, so the ring refills early
                float g = 0.f, u = 0.f;
#pragma unroll
                for (int r = 0; r < 4; ++r) {
                    const uint32_t m = n + r;
                    const int st = m % nstage; const uint32_t ph = (m / nstage) & 1;
                    bool okr = false;
                    if (r < nb) {
                        fail |= !mbar_wait_warp(&full[st], ph, cta_abort, lane);
                        okr = !fail && meta[st] != 0 && (P.stream_only & 1) == 0;
                    }
                    const uint4 *rr = reinterpret_cast<const uint4 *>(ring + (size_t)st * rec_bytes);
                    if (r == wr && okr) {
                        // dot products of this warp's record over this warp's column quarter
                        const uint4 *r0 = rr + wq * cq;
#pragma unroll
                        for (int j = 0; j < NQ; ++j) {
                            int c = lane + 32 * j;
                            if (c < cq) {
                                uint4 a = r0[c], bb = r0[chunks + c];
                                g += dot8<DT>(a, xr[j]); u += dot8<DT>(bb, xr[j]);
                            }
                        }
                    }
                    // down row of the record for this thread's columns
#pragma unroll
                    for (int q = 0; q < NCH; ++q) {
                        int c = ct + kConsumers * q;
                        dnp[r][q] = (okr && c < chunks) ? rr[2 * chunks + c] : make_uint4(0, 0, 0, 0);
                    }
                    if (r < nb) {
                        __syncwarp();
                        if (lane == 0) mbar_arrive(&empty[st]);
                    }
                }
                SI_PROF(1);                               // records: wait, dots, down loads
                n += nb;
                if (P.stream_only & 64) continue;
                // lane 0 <- sum(g), lane 16 <- sum(u): five shuffles, fixed order
                {
                    const bool hi16 = (lane & 16) != 0;
                    float keep = (hi16 ? u : g) + __shfl_xor_sync(0xFFFFFFFFu, hi16 ? g : u, 16);
                    keep += __shfl_xor_sync(0xFFFFFFFFu, keep, 8);
                    keep += __shfl_xor_sync(0xFFFFFFFFu, keep, 4);
                    keep += __shfl_xor_sync(0xFFFFFFFFu, keep, 2);
                    keep += __shfl_xor_sync(0xFFFFFFFFu, keep, 1);
                    g = keep;
                }
                const uint32_t buf = batches & 1;
                if ((lane & 15) == 0) reinterpret_cast<float *>(sm->part[buf])[cw * 2 + (lane >> 4)] = g;
                __syncwarp();
                if (lane == 0) mbar_arrive(&sm->redbar[buf]);
                pend = true; pbatch = batches;
                ++batches;
                SI_PROF(2);                               // publish dot products
            }
            if (pend && !fail && !(P.stream_only & 64)) finish_pending();
            SI_PROF(2);
            if (fail) break;

            // ---- [C1] finish the reduction of step sr: thread sum, warp butterfly over the WL
            // lanes that share a group (fixed order), warp-level sums to shared memory
            if (step >= kLag && !(P.stream_only & 128)) {
                float4 v = rv[0];
#pragma unroll
                for (int j = 1; j < NRL; ++j) { v.x += rv[j].x; v.y += rv[j].y; v.z += rv[j].z; v.w += rv[j].w; }
                for (int o = WL >> 1; o > 0; o >>= 1) {
                    v.x += __shfl_xor_sync(0xFFFFFFFFu, v.x, o); v.y += __shfl_xor_sync(0xFFFFFFFFu, v.y, o);
                    v.z += __shfl_xor_sync(0xFFFFFFFFu, v.z, o); v.w += __shfl_xor_sync(0xFFFFFFFFu, v.w, o);
                }
                const int sr = step - kLag;
                if ((ct % WL) == 0) sm->redy[sr & 1][ct / WL] = v;
            }
            SI_PROF(3);                                   // reduction: sums

            // ---- [C2] store the partial y of this step into the ring of D buffers
            if (real) {
                if (step >= kPartialDepth && !nosync) {
                    const int q = step - kPartialDepth;
                    fail |= !mbar_wait_warp(&sm->freebar[q % kFlagRing], (q / kFlagRing) & 1, cta_abort, lane);
                    if (fail) break;
                }
                float *mine = P.partial + ((size_t)(step % kPartialDepth) * G + b) * d;
#pragma unroll
                for (int q = 0; q < NCH; ++q) {
                    int c = ct + kConsumers * q;
                    if (c < chunks && !nosync) {
                        float4 *o = reinterpret_cast<float4 *>(mine + (size_t)c * 8);
                        __stcg(o, make_float4(acc[q][0], acc[q][1], acc[q][2], acc[q][3]));
                        __stcg(o + 1, make_float4(acc[q][4], acc[q][5], acc[q][6], acc[q][7]));
                    }
                }
            }
            // ---- [C3] this warp is done with the step: its partial is stored and its loads of
            // step sr have been consumed
            __syncwarp();
            if (lane == 0) {
                if (step >= kLag && !(P.stream_only & 128)) mbar_arrive(&sm->ybar[(step - kLag) & 1]);
                if (real) mbar_arrive(&sm->stepbar[step % kPartialDepth]);
            }
            SI_PROF(4);                                   // partial store
        }
#undef SI_PROF
        if (prof) {
            for (int i = 0; i < 6; ++i) P.prof[(size_t)b * 8 + i] = pf[i];
        }
        if (fail && lane == 0) raise_abort(P, sm, SI_ERR_TIMEOUT);
        return;
    }

    // -------------------------------------------------------------------------- signalling warp
    // Keeps the grid-scope fences and atomics off the consumers' path: once all consumer warps
    // are done with step s (partial stored, loads of step s - kLag consumed) it publishes
    // written[s] and reduced[s - kLag].
    if (warp == 1 + kConsumerWarps) {
        if (lane == 0 && (P.stream_only & 4) == 0) {
            for (int step = 0; step < P.n_steps; ++step) {
                if (!mbar_wait_bounded(&sm->stepbar[step % kPartialDepth], (step / kPartialDepth) & 1, cta_abort)) {
                    raise_abort(P, sm, SI_ERR_TIMEOUT);
                    break;
                }
                __threadfence();
                atomicAdd(P.counters + (size_t)step * kCounterStride, 1u);
                if (step >= kLag) atomicAdd(P.counters + (size_t)(step - kLag) * kCounterStride + 32, 1u);
            }
        }
        return;
    }
    // -------------------------------------------------------------------------- watcher warp
    // The only thread of the CTA that polls global memory: it turns "all G CTAs have published
    // step s" / "all G CTAs have finished reading step s" into shared-memory barriers the
    // consumers wait on.  It cannot run more than kFlagRing steps ahead of the consumers: a
    // step's counters only fill up after this CTA's own consumers have passed that step.
    if (lane == 0 && (P.stream_only & 4) == 0) {
        int pw = 0, pr = 0;                   // next step whose written / reduced counter is awaited
        const int n_red = P.n_steps - kLag;   // reduced[] is signalled for steps 0 .. n_steps-kLag-1
        long long t_last = clock64();
        while (pw < P.n_steps || pr < n_red) {
            bool progressed = false;
            if (pw < P.n_steps && ld_acquire_gpu(P.counters + (size_t)pw * kCounterStride) >= (unsigned)G) {
                mbar_arrive(&sm->pubbar[pw % kFlagRing]); ++pw; progressed = true;
            }
            if (pr < n_red && ld_acquire_gpu(P.counters + (size_t)pr * kCounterStride + 32) >= (unsigned)G) {
                mbar_arrive(&sm->freebar[pr % kFlagRing]); ++pr; progressed = true;
            }
            if (progressed) { t_last = clock64(); continue; }
            if (*cta_abort || ld_relaxed_gpu(P.ctrl + 1)) break;
            if (clock64() - t_last > kWaitCycles) { raise_abort(P, sm, SI_ERR_TIMEOUT); break; }
            __nanosleep(100);
        }
    }
}

inline size_t smem_bytes(int d_model, int nstage) {
    return (size_t)nstage * d_model * 6 + sizeof(Smem) + 128;
}
inline int pick_stages(int d_model) {
    const size_t budget = 227 * 1024 - 1024;
    int n = (int)((budget - smem_bytes(d_model, 0)) / ((size_t)d_model * 6));
    if (n > kMaxStages) n = kMaxStages;
    return n;
}

}  // namespace si_persist

// Diagnostics: when set, every persistent launch writes per-CTA cycle counts of the consumer
// phases (wait x, wait records, arithmetic, wait partial buffer, partial store).
long long *&si_decode_profile_buffer();
// Diagnostics: when non-zero, persistent launches only stream the records (practical HBM ceiling).
int &si_decode_stream_only();

inline bool si_persistent_supported(const si_store *s) {
    // the split-K reduction lets 512 / pow2ceil(groups per SM) threads share a column group and
    // gives each of them at most 3 / 5 / 10 partials (d_model <= 4096 / 8192 / 16384)
    const int chunks = s->d_model / 8, G = s->num_sms;
    const int gpc = (s->d_model / 4 + G - 1) / G;
    int gp = 1; while (gp < gpc) gp <<= 1;
    if (gp > 64) return false;
    const int tpg = si_persist::kConsumers / gp;
    const int nrl_max = chunks <= 512 ? 3 : chunks <= 1024 ? 5 : 10;
    return s->n_layers <= SI_MAX_LAYERS && si_persist::pick_stages(s->d_model) >= 3 &&
           chunks <= si_persist::kConsumers * 4 && (G + tpg - 1) / tpg <= nrl_max;
}

// Bytes of the partial-y ring.
inline size_t si_persistent_partial_bytes(const si_store *s) {
    return (size_t)si_persist::kPartialDepth * s->num_sms * s->d_model * 4;
}

template <int DT, int NCH, int NQ, int NRL>
inline int si_decode_persistent_launch_t(const si_persist::Params &P, int G, cudaStream_t stream) {
    auto kern = si_persist::si_decode_persistent_kernel<DT, NCH, NQ, NRL>;
    size_t smem = si_persist::smem_bytes(P.d_model, P.nstage);
    SI_CUDA_TRY(cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
    void *args[] = {(void *)&P};
    SI_CUDA_TRY(cudaLaunchCooperativeKernel((void *)kern, dim3(G), dim3(si_persist::kThreads), args, smem, stream));
    return SI_OK;
}

inline int si_decode_persistent_launch(const si_store *s, int n_steps, const int32_t *layers_host,
                                       const void *x, const int32_t *idx, const int32_t *idx_offsets,
                                       int k_fixed, void *y, int y_dtype, unsigned flags, char *wsb,
                                       const si_ws_layout &ws, int32_t *status_dev, cudaStream_t stream) {
    si_persist::Params P;
    P.store_base = s->mem;
    for (int l = 0; l < s->n_layers; ++l) { P.rec_off[l] = s->rec_off[l]; P.n_loaded[l] = s->n_loaded[l]; }
    P.n_layers = s->n_layers; P.n_steps = n_steps; P.k_fixed = k_fixed; P.d_model = s->d_model;
    P.chunks = s->d_model / 8; P.nstage = si_persist::pick_stages(s->d_model);
    P.step_layers = nullptr;
    // steps region: [n_steps] layer ids | [n_steps][64] counters
    int32_t *steps = (int32_t *)(wsb + ws.steps_off);
    if (layers_host) {
        SI_CUDA_TRY(cudaMemcpyAsync(steps, layers_host, (size_t)n_steps * 4, cudaMemcpyHostToDevice, stream));
        P.step_layers = steps;
    }
    P.counters = (unsigned int *)(wsb + ws.steps_off + si_align_up((size_t)n_steps * 4, 256));
    P.x = (const uint16_t *)x; P.idx = idx; P.idx_offsets = idx_offsets; P.y = y;
    P.y_f32 = y_dtype == SI_F32; P.residual = (flags & SI_FLAG_RESIDUAL) != 0;
    P.partial = (float *)(wsb + ws.partial_off);
    P.ctrl = (unsigned int *)(wsb + ws.ctrl_off);
    P.status = status_dev;
    P.prof = si_decode_profile_buffer();
    P.stream_only = si_decode_stream_only() & 0xFF;
    P.prefetch_rounds = (si_decode_stream_only() >> 8) & 0xF;
    int G = s->num_sms;
    if (!idx_offsets && k_fixed < G) G = k_fixed < 1 ? 1 : k_fixed;
    SI_CUDA_TRY(cudaMemsetAsync(P.ctrl, 0, 256, stream));
    SI_CUDA_TRY(cudaMemsetAsync(P.counters, 0, (size_t)n_steps * si_persist::kCounterStride * 4, stream));
    // NCH: 16-byte column chunks per thread in the down projection (512 threads);
    // NQ : chunks per lane in the dot products (a warp covers a quarter of the columns)
    const int nch = (P.chunks + si_persist::kConsumers - 1) / si_persist::kConsumers;
    const int nq = (P.chunks / 4 + 31) / 32;
    // NRL: partial-y loads per thread in the split-K reduction (see the kernel)
#define SI_PL(DT)                                                                     \
    (nq <= 1 ? si_decode_persistent_launch_t<DT, 1, 1, 3>(P, G, stream)               \
     : nq <= 2 ? si_decode_persistent_launch_t<DT, 1, 2, 3>(P, G, stream)             \
     : nq <= 4 ? si_decode_persistent_launch_t<DT, 1, 4, 3>(P, G, stream)             \
     : nq <= 8 ? si_decode_persistent_launch_t<DT, 2, 8, 5>(P, G, stream)             \
               : si_decode_persistent_launch_t<DT, 4, 16, 10>(P, G, stream))
    (void)nch;
    return s->dtype == SI_BF16 ? SI_PL(SI_BF16) : SI_PL(SI_F16);
#undef SI_PL
}
