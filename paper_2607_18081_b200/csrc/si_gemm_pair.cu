// Prefill contractions on pairs of SMs (more than 128 tokens in a call).
//
// With hundreds of tokens the two contractions of a multi-token call are bound by how fast an SM can fill
// its shared memory, not by HBM: a 128 x 128 tile needs 48 KB of operands for 512 tensor-pipe cycles.  Here a
// thread-block cluster of two CTAs works on one tile with tcgen05.mma.cta_group::2 (M = 256: the tokens, 128
// per CTA; N = 256 or 128 store columns, each CTA holding half of them in its shared memory), so every CTA
// loads its own 128 tokens and only HALF of the weight tile the pair multiplies them with:
//
//   gate/up   D[256 tokens x (W gate | W up)] = X[tokens, k] . W[U tile, k]^T         (K = d_model; W = 128 or 96)
//             CTA 0 of the pair loads the tile's gate rows, CTA 1 its up rows; a thread of the epilogue owns
//             one token and finds gate and up of a neuron in its own registers: H = member . SiLU(g) . u
//   down      D[256 tokens x N columns] = H[tokens, U_k] . Wd[U_k, columns]           (K = |U|)
//             CTA r loads columns r * N/2 .. of the 64 down rows of a chunk (MN-major operand)
//
// No partial tiles in global memory: H and y are written straight from tensor memory (with a long K, two pairs
// share a down tile, half of K each, and exchange their accumulators through distributed shared memory).  Each CTA tracks the
// stages of its own shared memory with local mbarriers, exactly as the one-CTA kernels do; the pair is coupled
// by two signals only: the second CTA's MMA warp relays "my half of stage s has landed" to a barrier of the
// first (the one that issues the MMAs), and the commit that frees a stage (or declares the accumulators
// complete) arrives on the barriers of both.  All waits are bounded; both CTAs stay until a last cluster
// barrier, so neither is signalled after it has gone.
#include "si_tc.cuh"

using namespace si_tc;

namespace {

constexpr int kPairMaxStages = 8;
constexpr int kPrefetchAhead = 16;               // chunks between a weight tile's L2 prefetch and its copy into shared memory
constexpr int kPairTokens = 256;                 // tokens of a pair's tile (M of the MMA), 128 per CTA

__device__ __forceinline__ void mbar_arrive_remote(uint32_t cluster_addr) {
    asm volatile("mbarrier.arrive.relaxed.cluster.shared::cluster.b64 _, [%0];" ::"r"(cluster_addr) : "memory");
}
// wait on a barrier that a thread of the other CTA arrives on (cluster-scope acquire); bounded like mbar_wait
__device__ __forceinline__ bool mbar_wait_cluster(uint64_t *bar, uint32_t parity, long long limit) {
    for (long long i = 0; i < limit; ++i) {
        uint32_t ok;
        asm volatile(
            "{\n\t.reg .pred p;\n\t"
            "mbarrier.try_wait.parity.acquire.cluster.shared::cta.b64 p, [%1], %2;\n\t"
            "selp.u32 %0, 1, 0, p;\n\t}"
            : "=r"(ok) : "r"(smem_u32(bar)), "r"(parity) : "memory");
        if (ok) return true;
    }
    return false;
}
// D[256 x N] (+)= A . B over the pair: A rows and B rows of either CTA are read from its own shared memory at
// the descriptors' offsets; issued by one thread of the pair's first CTA
__device__ __forceinline__ void umma_pair(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc, uint32_t accumulate) {
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::2.kind::f16 [%0], %1, %2, %3, p;\n\t}"
        ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate) : "memory");
}
// arrives on the barrier at this offset in BOTH CTAs of the pair (mask: their ranks in the cluster) once the MMAs issued
// so far have completed
__device__ __forceinline__ void umma_commit_pair(uint64_t *bar, uint16_t mask) {
    asm volatile("tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.multicast::cluster.b64 [%0], %1;"
                 ::"r"(smem_u32(bar)), "h"(mask) : "memory");
}

// One pipeline stage of the pair's MMA thread as a single instruction sequence: probe the NEXT stage's barrier,
// issue this stage's four MMAs (K = 16 each), commit them to this stage's "empty" barriers of both CTAs, and only
// then read the probe's answer.  A probe takes a couple of hundred cycles to answer; issued first, it is answered
// while the MMAs are being issued instead of ahead of them.  Returns whether the next stage had already landed.
__device__ __forceinline__ bool pair_issue_stage(uint32_t d_tmem, const uint64_t (&a)[4], const uint64_t (&b)[4], uint32_t idesc,
                                                 uint32_t accumulate_first, uint64_t *empty_bar, uint64_t *next_full, uint32_t next_parity, uint16_t mask) {
    uint32_t landed;
    asm volatile(
        "{\n\t.reg .pred q, p, t;\n\t"
        "mbarrier.try_wait.parity.acquire.cluster.shared::cta.b64 q, [%12], %13;\n\t"
        "setp.ne.b32 p, %10, 0;\n\t"
        "setp.eq.b32 t, 0, 0;\n\t"
        "tcgen05.mma.cta_group::2.kind::f16 [%1], %2, %6, %11, p;\n\t"
        "tcgen05.mma.cta_group::2.kind::f16 [%1], %3, %7, %11, t;\n\t"
        "tcgen05.mma.cta_group::2.kind::f16 [%1], %4, %8, %11, t;\n\t"
        "tcgen05.mma.cta_group::2.kind::f16 [%1], %5, %9, %11, t;\n\t"
        "tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.multicast::cluster.b64 [%14], %15;\n\t"
        "selp.u32 %0, 1, 0, q;\n\t}"
        : "=r"(landed)
        : "r"(d_tmem), "l"(a[0]), "l"(a[1]), "l"(a[2]), "l"(a[3]), "l"(b[0]), "l"(b[1]), "l"(b[2]), "l"(b[3]), "r"(accumulate_first),
          "r"(idesc), "r"(smem_u32(next_full)), "r"(next_parity), "r"(smem_u32(empty_bar)), "h"(mask)
        : "memory");
    return landed != 0;
}

// Two stages in one sequence: the probes of the two stages after them come first and are read last, so that they
// have the time of eight MMAs to be answered (under load a probe takes several hundred cycles -- more than the four
// MMAs of one stage when these are narrow).  bit 0 / 1 of the result: stage c + 2 / c + 3 had already landed.
__device__ __forceinline__ uint32_t pair_issue_two_stages(uint32_t d_tmem, const uint64_t (&a)[8], const uint64_t (&b)[8], uint32_t idesc,
                                                          uint32_t accumulate_first, uint64_t *empty0, uint64_t *empty1,
                                                          uint64_t *next_full0, uint32_t next_parity0, uint64_t *next_full1, uint32_t next_parity1,
                                                          uint16_t mask) {
    uint32_t landed;
    asm volatile(
        "{\n\t.reg .pred q0, q1, p, t;\n\t.reg .b32 r0, r1;\n\t"
        "mbarrier.try_wait.parity.acquire.cluster.shared::cta.b64 q0, [%20], %21;\n\t"
        "mbarrier.try_wait.parity.acquire.cluster.shared::cta.b64 q1, [%22], %23;\n\t"
        "setp.ne.b32 p, %18, 0;\n\t"
        "setp.eq.b32 t, 0, 0;\n\t"
        "tcgen05.mma.cta_group::2.kind::f16 [%1], %2, %10, %19, p;\n\t"
        "tcgen05.mma.cta_group::2.kind::f16 [%1], %3, %11, %19, t;\n\t"
        "tcgen05.mma.cta_group::2.kind::f16 [%1], %4, %12, %19, t;\n\t"
        "tcgen05.mma.cta_group::2.kind::f16 [%1], %5, %13, %19, t;\n\t"
        "tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.multicast::cluster.b64 [%24], %26;\n\t"
        "tcgen05.mma.cta_group::2.kind::f16 [%1], %6, %14, %19, t;\n\t"
        "tcgen05.mma.cta_group::2.kind::f16 [%1], %7, %15, %19, t;\n\t"
        "tcgen05.mma.cta_group::2.kind::f16 [%1], %8, %16, %19, t;\n\t"
        "tcgen05.mma.cta_group::2.kind::f16 [%1], %9, %17, %19, t;\n\t"
        "tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.multicast::cluster.b64 [%25], %26;\n\t"
        "selp.u32 r0, 1, 0, q0;\n\t"
        "selp.u32 r1, 2, 0, q1;\n\t"
        "or.b32 %0, r0, r1;\n\t}"
        : "=r"(landed)
        : "r"(d_tmem), "l"(a[0]), "l"(a[1]), "l"(a[2]), "l"(a[3]), "l"(a[4]), "l"(a[5]), "l"(a[6]), "l"(a[7]),
          "l"(b[0]), "l"(b[1]), "l"(b[2]), "l"(b[3]), "l"(b[4]), "l"(b[5]), "l"(b[6]), "l"(b[7]),
          "r"(accumulate_first), "r"(idesc), "r"(smem_u32(next_full0)), "r"(next_parity0), "r"(smem_u32(next_full1)), "r"(next_parity1),
          "r"(smem_u32(empty0)), "r"(smem_u32(empty1)), "h"(mask)
        : "memory");
    return landed;
}

// One stage of a tile that is two sub-tiles wide (two accumulators, one A operand): the probe of the next stage, the
// four MMAs of the first sub-tile, the four of the second (same A descriptors, B descriptors b[4..7], accumulator d1),
// one commit, the probe's answer.
__device__ __forceinline__ bool pair_issue_wide_stage(uint32_t d0, uint32_t d1, const uint64_t (&a)[4], const uint64_t (&b)[8], uint32_t idesc,
                                                      uint32_t accumulate_first, uint64_t *empty_bar, uint64_t *next_full, uint32_t next_parity,
                                                      uint16_t mask) {
    uint32_t landed;
    asm volatile(
        "{\n\t.reg .pred q, p, t;\n\t"
        "mbarrier.try_wait.parity.acquire.cluster.shared::cta.b64 q, [%17], %18;\n\t"
        "setp.ne.b32 p, %15, 0;\n\t"
        "setp.eq.b32 t, 0, 0;\n\t"
        "tcgen05.mma.cta_group::2.kind::f16 [%1], %3, %7, %16, p;\n\t"
        "tcgen05.mma.cta_group::2.kind::f16 [%2], %3, %11, %16, p;\n\t"
        "tcgen05.mma.cta_group::2.kind::f16 [%1], %4, %8, %16, t;\n\t"
        "tcgen05.mma.cta_group::2.kind::f16 [%2], %4, %12, %16, t;\n\t"
        "tcgen05.mma.cta_group::2.kind::f16 [%1], %5, %9, %16, t;\n\t"
        "tcgen05.mma.cta_group::2.kind::f16 [%2], %5, %13, %16, t;\n\t"
        "tcgen05.mma.cta_group::2.kind::f16 [%1], %6, %10, %16, t;\n\t"
        "tcgen05.mma.cta_group::2.kind::f16 [%2], %6, %14, %16, t;\n\t"
        "tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.multicast::cluster.b64 [%19], %20;\n\t"
        "selp.u32 %0, 1, 0, q;\n\t}"
        : "=r"(landed)
        : "r"(d0), "r"(d1), "l"(a[0]), "l"(a[1]), "l"(a[2]), "l"(a[3]), "l"(b[0]), "l"(b[1]), "l"(b[2]), "l"(b[3]),
          "l"(b[4]), "l"(b[5]), "l"(b[6]), "l"(b[7]), "r"(accumulate_first), "r"(idesc), "r"(smem_u32(next_full)), "r"(next_parity),
          "r"(smem_u32(empty_bar)), "h"(mask)
        : "memory");
    return landed != 0;
}

struct PairBars {
    // stage landed.  In the pair's first CTA one arrival more is expected: the second CTA's word that ITS half has landed
    uint64_t full_t[kPairMaxStages];     // ... tensor copies only (one arrival: the thread that starts them)
    uint64_t full_g[kPairMaxStages];     // ... gathered rows + the dense tile (all loader threads + 1)
    uint64_t empty[kPairMaxStages];      // the MMAs have read the stage (both CTAs are told)
    uint64_t accbar;                     // accumulators complete (both CTAs are told)
    uint64_t xbar;                       // (K split) the other pair's partial accumulators have arrived
    uint32_t tmem_slot;
    int failed;
};

// set-up common to both kernels: barriers, tensor memory of the pair, cluster barrier.  Returns the tensor-memory base.
__device__ __forceinline__ uint32_t pair_setup(PairBars *B, int nstage, uint32_t ncols, uint32_t rank) {
    const int tid = threadIdx.x, warp = tid >> 5;
    if (tid == 0) {
        const uint32_t from_peer = rank == 0 ? 1u : 0u;
        for (int s = 0; s < nstage; ++s) {
            mbar_init(&B->full_t[s], 1 + from_peer); mbar_init(&B->full_g[s], kLoaderThreads + 1 + from_peer);
            mbar_init(&B->empty[s], 1);
        }
        mbar_init(&B->accbar, 1);
        mbar_init(&B->xbar, 1);
        B->failed = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == kLoaderWarps) {
        asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&B->tmem_slot)), "r"(ncols) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    cluster_sync_all();                  // the other CTA's barriers exist before anything is signalled across
    tc_fence_after();
    return *reinterpret_cast<volatile uint32_t *>(&B->tmem_slot);
}

__device__ __forceinline__ void pair_teardown(uint32_t tmem, uint32_t ncols) {
    tc_fence_before();
    __syncthreads();
    cluster_sync_all();                  // nobody reads this CTA's shared or tensor memory any more, nobody signals it
    if ((threadIdx.x >> 5) == kLoaderWarps)
        asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(ncols) : "memory");
}

// The MMA warp's loop.  First CTA: wait until both halves of a stage have landed (its own copies and the second
// CTA's word arrive on the same barrier), issue, free the stage in both CTAs.  Second CTA: pass the completion of
// its own stage barrier on to the first CTA's.  `gathered`: the stage holds rows written by cp.async (generic
// proxy), which need a proxy fence before the MMAs read them.  a0 / b0: the operand descriptors of the four MMAs
// of stage 0; those of stage s follow by adding s * stage_bytes to the address field.  The MMAs of a stage are
// issued back to back with as little as possible in between: an MMA instruction is not handed over before the
// one ahead of it is nearly done, so whatever the thread does between two stages the tensor pipe waits for.
__device__ __forceinline__ void pair_mma_loop(PairBars *B, uint64_t *full, bool gathered, int n_chunks, int nstage, long long limit,
                                              uint32_t rank, uint32_t tmem, uint32_t idesc, const uint64_t (&a0)[4], const uint64_t (&b0)[4],
                                              uint32_t stage_bytes, uint32_t leader = 0, uint32_t wide_b_bytes = 0,
                                              uint32_t wide_d_cols = 0) {
    // rank: this CTA's place in its pair (0 issues the MMAs); leader: the cluster rank of the pair's first CTA;
    // wide_b_bytes != 0: the tile is two sub-tiles wide -- the second sub-tile's B rows lie wide_b_bytes further on
    // in a stage, its accumulator wide_d_cols columns further on in tensor memory
    const uint16_t mask = (uint16_t)(3u << leader);
    volatile int *failed = &B->failed;
    bool ok = true;
    if (rank == 0 && wide_b_bytes) {
        bool landed = false;
        int st = 0; uint32_t ph = 0;
        const uint64_t step = (uint64_t)(stage_bytes >> 4), sub = (uint64_t)(wide_b_bytes >> 4);
        for (int c = 0; c < n_chunks; ++c) {
            if (!landed) ok = mbar_wait_cluster(&full[st], ph, limit);
            if (!ok) break;
            if (gathered) { fence_async_proxy(); tc_fence_after(); }
            const uint64_t o = step * (uint64_t)st;
            const uint64_t a[4] = {a0[0] + o, a0[1] + o, a0[2] + o, a0[3] + o};
            const uint64_t b[8] = {b0[0] + o, b0[1] + o, b0[2] + o, b0[3] + o, b0[0] + o + sub, b0[1] + o + sub, b0[2] + o + sub, b0[3] + o + sub};
            int s1 = st; uint32_t p1 = ph;
            if (++s1 == nstage) { s1 = 0; p1 ^= 1u; }
            landed = pair_issue_wide_stage(tmem, tmem + wide_d_cols, a, b, idesc, c ? 1u : 0u, &B->empty[st], &full[s1], p1, mask);
            st = s1; ph = p1;
        }
        if (!ok) *failed = 1;
        umma_commit_pair(&B->accbar, mask);
    } else if (rank == 0) {
        // stages are issued two at a time; `landed` bit 0 / 1: the probe of the first / second of the two was answered "yes"
        uint32_t landed = 0;
        int st = 0; uint32_t ph = 0;
        const uint64_t step = (uint64_t)(stage_bytes >> 4);     // (the address field holds bytes / 16 and never overflows: shared memory is < 256 KB)
        auto next = [&](int &s_, uint32_t &p_) { if (++s_ == nstage) { s_ = 0; p_ ^= 1u; } };
        int c = 0;
        for (; c + 1 < n_chunks; c += 2) {
            int s1 = st; uint32_t p1 = ph; next(s1, p1);
            if (!(landed & 1u)) ok = mbar_wait_cluster(&full[st], ph, limit);
            if (ok && !(landed & 2u)) ok = mbar_wait_cluster(&full[s1], p1, limit);
            if (!ok) break;
            if (gathered) { fence_async_proxy(); tc_fence_after(); }
            const uint64_t o0 = step * (uint64_t)st, o1 = step * (uint64_t)s1;
            const uint64_t a[8] = {a0[0] + o0, a0[1] + o0, a0[2] + o0, a0[3] + o0, a0[0] + o1, a0[1] + o1, a0[2] + o1, a0[3] + o1};
            const uint64_t b[8] = {b0[0] + o0, b0[1] + o0, b0[2] + o0, b0[3] + o0, b0[0] + o1, b0[1] + o1, b0[2] + o1, b0[3] + o1};
            int s2 = s1; uint32_t p2 = p1; next(s2, p2);
            int s3 = s2; uint32_t p3 = p2; next(s3, p3);
            // (probes past the last chunk look at stages that nothing refills: they answer "no" and are not used)
            landed = pair_issue_two_stages(tmem, a, b, idesc, c ? 1u : 0u, &B->empty[st], &B->empty[s1], &full[s2], p2, &full[s3], p3, mask);
            st = s2; ph = p2;
        }
        if (ok && c < n_chunks) {              // an odd chunk is left
            if (!(landed & 1u)) ok = mbar_wait_cluster(&full[st], ph, limit);
            if (ok) {
                if (gathered) { fence_async_proxy(); tc_fence_after(); }
                const uint64_t o0 = step * (uint64_t)st;
                const uint64_t a[4] = {a0[0] + o0, a0[1] + o0, a0[2] + o0, a0[3] + o0};
                const uint64_t b[4] = {b0[0] + o0, b0[1] + o0, b0[2] + o0, b0[3] + o0};
                int s1 = st; uint32_t p1 = ph; next(s1, p1);
                pair_issue_stage(tmem, a, b, idesc, c ? 1u : 0u, &B->empty[st], &full[s1], p1, mask);
            }
        }
        if (!ok) *failed = 1;
        umma_commit_pair(&B->accbar, mask);    // accumulators complete (or nothing was issued): told to both CTAs
    } else {
        const uint32_t remote0 = map_to_cta(smem_u32(&full[0]), leader);
        for (int c = 0; c < n_chunks; ++c) {
            const int st = c % nstage; const uint32_t ph = (c / nstage) & 1;
            ok = mbar_wait(&full[st], ph, limit);
            if (!ok) break;
            if (gathered) fence_async_proxy();   // this CTA's gathered rows are visible to the MMAs before the first CTA is told
            mbar_arrive_remote(remote0 + (uint32_t)st * 8u);
        }
        if (!ok) *failed = 1;
    }
}

// H for this CTA's 128 tokens x the tile's S * W neurons, straight from tensor memory: thread = token (lane of the
// tensor memory); sub-tile s has its gate values in columns [s * 2W, s * 2W + W) and its up values in the W columns
// after them.  Warps w and w + 4 share the lanes: with one sub-tile they take W / 2 neurons each, with two a sub-tile
// each.  Written without a branch per element: SiLU(g) * u is formed for every element and kept or zeroed by a select.
template <int DT, int W, int S>
__device__ __forceinline__ void gateup_epilogue(const GemmParams &P, uint32_t tmem, int warp, int lane, int tok0, int nt, int n_u) {
    const int q = warp & 3, half = warp >> 2;
    const int t = tok0 + q * 32 + lane;
    constexpr int kCount = S == 1 ? W / 2 : W;                    // neurons of this thread
    const int sub = S == 1 ? 0 : half, r0 = S == 1 ? (W / 2) * half : 0;
    const uint32_t trow = tmem + ((uint32_t)(q * 32) << 16) + (uint32_t)(sub * 2 * W + r0);
    const int i0 = nt * S * W + sub * W + r0;                     // union position of this thread's first neuron
    uint16_t *hrow = P.h_out + (size_t)t * P.nu_pad + i0;
    const bool has_row = t < P.t_pad_total;                       // H has rows for the tokens padded to 16 only (no early
                                                                  // return: the tensor-memory loads below are warp-wide)
    const int lim = t < P.T ? n_u - i0 : 0;                       // positions below lim are real entries of a real token
    const bool own = P.tokbits != nullptr;                        // (uniform) every token keeps to its own list
    const uint32_t *tb = own ? P.tokbits + (size_t)(t < P.T ? t : 0) * P.mask_words : nullptr;
    for (int n0 = 0; n0 < kCount; n0 += 16) {
        if (i0 + n0 >= P.nu_pad) break;                           // (a last tile may reach past the padded union)
        uint32_t g[16], u[16];
        tmem_ld16(trow + (uint32_t)n0, g);
        tmem_ld16(trow + (uint32_t)(W + n0), u);
        uint32_t member = 0xFFFFu;                                // bit j: the token selected neuron n0 + j
        if (own) {
            member = 0;
#pragma unroll
            for (int jj = 0; jj < 16; ++jj) {
                const int slot = P.union_slots[i0 + n0 + jj];     // the same address in every lane
                member |= ((tb[slot >> 5] >> (slot & 31)) & 1u) << jj;
            }
        }
        uint32_t w[8];
#pragma unroll
        for (int jj = 0; jj < 16; ++jj) {
            const uint32_t bits = si_cvt<DT>::from_float(si_silu_mul(__uint_as_float(g[jj]), __uint_as_float(u[jj])));
            const uint32_t b = (n0 + jj < lim && ((member >> jj) & 1u)) ? bits : 0u;
            if (jj & 1) w[jj >> 1] |= b << 16; else w[jj >> 1] = b;
        }
        if (has_row) {
            *reinterpret_cast<uint4 *>(hrow + n0) = make_uint4(w[0], w[1], w[2], w[3]);
            *reinterpret_cast<uint4 *>(hrow + n0 + 8) = make_uint4(w[4], w[5], w[6], w[7]);
        }
    }
}

// Gate/up contraction: one pair per (union tile of S * W neurons, 256 tokens).  N of an MMA = 2 W: the gate rows and
// the up rows of W neurons; S = 2: the tile is two such sub-tiles with an accumulator each, which share the X tile
// (less operand traffic per MMA cycle, and half as many tiles: large unions in one wave instead of two).  The host
// picks (W, S) by cost: waves of pair tiles over the SM pairs x the MMA time of a tile's chunk.
template <int W, int S>
__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(kGemmThreads, 1)
si_pair_gateup_kernel(const __grid_constant__ GemmParams P, const __grid_constant__ CUtensorMap x_map,
                      const __grid_constant__ CUtensorMap rec_map) {
    extern __shared__ __align__(1024) uint8_t smem[];
    constexpr int R = S * W;                                      // weight rows of a tile (per CTA: the gate rows, or the up rows)
    constexpr int stage_bytes = 128 * 128 + R * 128;              // this CTA's X tile, this CTA's R weight rows
    uint8_t *tiles = smem;
    PairBars *B = reinterpret_cast<PairBars *>(smem + (size_t)P.nstage * stage_bytes);
    volatile int *failed = &B->failed;
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const uint32_t rank = cluster_ctarank();
    constexpr uint32_t ncols = S == 1 ? 256 : 512;                // per sub-tile W gate + W up accumulator columns
    const uint32_t tmem = pair_setup(B, P.nstage, ncols, rank);

    pdl_wait();                                 // the union kernel's results
    pdl_launch();
    const int pair = blockIdx.x >> 1;
    const int n_tiles = (P.nu_pad + R - 1) / R;
    const int nt = pair % n_tiles, tp = pair / n_tiles;
    const int n_u = *P.n_union;
    // tiles past the real union have nothing to do (the down contraction reads H in chunks of 64 entries: up to there
    // H must be written)
    const bool active = nt * R < (n_u + kChunkK - 1) / kChunkK * kChunkK;
    const int n_chunks = active ? P.d_model / kChunkK : 0;
    const int tok0 = tp * kPairTokens + (int)rank * 128;          // this CTA's tokens
    // union entry of tile row r (a last tile may reach past the padded union: its surplus rows repeat the last entry)
    auto entry = [&](int r) { const int e = nt * R + r; return e < P.nu_pad ? e : P.nu_pad - 1; };
    // a tile of R consecutive slots needs no gather: its rows are one tensor copy out of the record matrix
    const int slot_first = P.union_slots[entry(0)];
    const bool run = nt * R + R <= P.nu_pad && P.union_slots[nt * R + R - 1] - slot_first == R - 1;
    uint64_t *full = run ? B->full_t : B->full_g;
    const bool withhold = P.withhold && blockIdx.x == 0;

    if (warp < kLoaderWarps) {
        int armed = 0;                       // (a thread that starts tensor copies) 1 + the last chunk whose copies it has started
        if (run) {
            // two threads (of different warps) start the copies of alternate chunks: one thread's round of probe,
            // expect and two tensor copies takes longer than the MMAs of a chunk
            if (lane == 0 && warp < 2) {
                for (int c = warp; c < n_chunks; c += 2) {
                    const int st = c % P.nstage; const uint32_t ph = (c / P.nstage) & 1;
                    if (!mbar_wait(&B->empty[st], ph ^ 1, P.spin_limit)) { *failed = 1; break; }
                    if (withhold && c == 0) continue;
                    uint8_t *stage = tiles + (size_t)st * stage_bytes;
                    armed = c + 1;
                    mbar_arrive_expect_tx(&full[st], (uint32_t)stage_bytes);
                    tma_load_tile(stage, &x_map, c * kChunkK, tok0, &full[st]);
                    tma_load_tile(stage + 128 * 128, &rec_map, (int)rank * P.d_model + c * kChunkK, slot_first, &full[st]);
                    // the weights come from HBM: ask for the tile of a later chunk now, so that its copy finds it in L2
                    // (the ring alone holds too few bytes for that latency); one of the token tiles asks for all
                    if (tp == 0 && c + kPrefetchAhead < n_chunks)
                        tma_prefetch_tile(&rec_map, (int)rank * P.d_model + (c + kPrefetchAhead) * kChunkK, slot_first);
                }
            }
        } else {
            // copy j of a thread covers 16-byte piece (tid & 7) of tile row 32*j + (tid >> 3): a warp instruction
            // reads four whole 128-byte row segments
            const int q8 = tid & 7, r32 = tid >> 3;
            const char *wrow[R / 32];
#pragma unroll
            for (int j = 0; j < R / 32; ++j)
                wrow[j] = P.rec_base + (size_t)P.union_slots[entry(32 * j + r32)] * P.rec_bytes + (size_t)rank * P.d_model * 2 + q8 * 16;
            const int off0 = r32 * 128 + ((q8 ^ (r32 & 7)) << 4);
            for (int c = 0; c < n_chunks; ++c) {
                const int st = c % P.nstage; const uint32_t ph = (c / P.nstage) & 1;
                if (!mbar_wait_relaxed(&B->empty[st], ph ^ 1, P.spin_limit, 32)) { *failed = 1; break; }
                uint8_t *stage = tiles + (size_t)st * stage_bytes;
                uint8_t *sw = stage + 128 * 128 + off0;
#pragma unroll
                for (int j = 0; j < R / 32; ++j) { cp_async16(sw + j * 4096, wrow[j]); wrow[j] += 128; }
                if (tid == 0 && !(withhold && c == 0)) {
                    armed = c + 1;
                    mbar_arrive_expect_tx(&full[st], 128u * 128u);
                    tma_load_tile(stage, &x_map, c * kChunkK, tok0, &full[st]);
                }
                cp_async_arrive_when_landed(&full[st]);
            }
            cp_async_wait_all();             // nothing of this thread may still be in flight when the CTA ends
        }
        // ---------------------------------------------------------------- epilogue
        bool ok = mbar_wait_relaxed(&B->accbar, 0, P.spin_limit, 256) && !*failed;
        if (!ok && armed > 0)                // a wait ran out: the tensor copies this thread started must still land before the CTA goes
            for (int c = armed - 1; c >= 0 && c > armed - 1 - P.nstage; c -= run ? 2 : 1)
                mbar_wait(&full[c % P.nstage], (c / P.nstage) & 1, P.spin_limit);
        tc_fence_after();
        if (ok && active) {
            if (P.fmt) gateup_epilogue<SI_BF16, W, S>(P, tmem, warp, lane, tok0, nt, n_u);
            else gateup_epilogue<SI_F16, W, S>(P, tmem, warp, lane, tok0, nt, n_u);
        }
        if (!ok && tid == 0 && P.status) atomicCAS(P.status, 0, SI_ERR_TIMEOUT);
    } else if (lane == 0) {
        const uint32_t idesc = make_idesc(P.fmt, 0, 0, 256, 2 * W);
        const uint32_t sx = smem_u32(tiles), sw = sx + 128 * 128;
        uint64_t a0[4], b0[4];
#pragma unroll
        for (int k4 = 0; k4 < 4; ++k4) { a0[k4] = make_desc(sx + k4 * 32, 16, 1024); b0[k4] = make_desc(sw + k4 * 32, 16, 1024); }
        pair_mma_loop(B, full, !run, n_chunks, P.nstage, P.spin_limit, rank, tmem, idesc, a0, b0, (uint32_t)stage_bytes, 0u,
                      S == 2 ? (uint32_t)(W * 128) : 0u, (uint32_t)(2 * W));
    }
    pair_teardown(tmem, ncols);
}

// Sixteen consecutive output columns of one token: residual added, rounded to the output type, written.
__device__ __forceinline__ void down_store16(const GemmParams &P, size_t o, float (&a)[16]) {
    if (P.residual) {
        const uint4 x0 = *reinterpret_cast<const uint4 *>(P.x + o), x1 = *reinterpret_cast<const uint4 *>(P.x + o + 8);
        const uint32_t xw[8] = {x0.x, x0.y, x0.z, x0.w, x1.x, x1.y, x1.z, x1.w};
#pragma unroll
        for (int j = 0; j < 8; ++j) {
            a[2 * j] += P.fmt ? si_cvt<SI_BF16>::lo(xw[j]) : si_cvt<SI_F16>::lo(xw[j]);
            a[2 * j + 1] += P.fmt ? si_cvt<SI_BF16>::hi(xw[j]) : si_cvt<SI_F16>::hi(xw[j]);
        }
    }
    if (P.y_f32) {
        float4 *yo = reinterpret_cast<float4 *>(reinterpret_cast<float *>(P.y) + o);
#pragma unroll
        for (int j = 0; j < 4; ++j) yo[j] = make_float4(a[4 * j], a[4 * j + 1], a[4 * j + 2], a[4 * j + 3]);
    } else {
        uint32_t w[8];
#pragma unroll
        for (int j = 0; j < 8; ++j)
            w[j] = P.fmt ? ((uint32_t)si_cvt<SI_BF16>::from_float(a[2 * j]) | ((uint32_t)si_cvt<SI_BF16>::from_float(a[2 * j + 1]) << 16))
                         : ((uint32_t)si_cvt<SI_F16>::from_float(a[2 * j]) | ((uint32_t)si_cvt<SI_F16>::from_float(a[2 * j + 1]) << 16));
        uint4 *yo = reinterpret_cast<uint4 *>(reinterpret_cast<uint16_t *>(P.y) + o);
        yo[0] = make_uint4(w[0], w[1], w[2], w[3]);
        yo[1] = make_uint4(w[4], w[5], w[6], w[7]);
    }
}

// y for this CTA's 128 tokens x N columns, straight from tensor memory.
template <int N>
__device__ __forceinline__ void down_epilogue(const GemmParams &P, bool ok, int n_chunks, uint32_t tmem, int warp, int lane, int tok0, int ct) {
    constexpr int kHalfCols = N / 2;
    if (!ok) return;
    // thread = token; warps w and w + 4 share the lanes and take half of the tile's columns each
    const int q = warp & 3, half = warp >> 2;
    const int t = tok0 + q * 32 + lane;
    const uint32_t trow = tmem + ((uint32_t)(q * 32) << 16);
    const size_t o0 = (size_t)t * P.d_model + (size_t)ct * N + half * kHalfCols;
    for (int n0 = 0; n0 < kHalfCols; n0 += 16) {
        uint32_t v[16];
        if (n_chunks > 0) tmem_ld16(trow + (uint32_t)(half * kHalfCols + n0), v);
        if (t >= P.T) continue;
        float a[16];
#pragma unroll
        for (int j = 0; j < 16; ++j) a[j] = n_chunks > 0 ? __uint_as_float(v[j]) : 0.f;
        down_store16(P, o0 + n0, a);
    }
}

// The same when two pairs of a cluster of four CTAs have each summed half of K into their own accumulators of the
// same 256-column tile (pair kq: K half kq): CTA (kq, r) finishes columns [kq * 128, kq * 128 + 128) of its 128 tokens.
// It stages the other 128 columns of its accumulators in its own shared memory and sends them to CTA (1 - kq, r) --
// which holds the other K half of the same tokens -- as one bulk copy through distributed shared memory (remote
// stores from every thread took five times as long), receives that CTA's values for its own columns the same way,
// and adds them in K order.  The staging areas are the pipeline stages, free once every CTA's MMAs are complete (the
// cluster barrier below); a CTA leaves only after the last cluster barrier, i.e. after its own block has been received.
__device__ __forceinline__ void down_epilogue_split(const GemmParams &P, uint8_t *smem, PairBars *B, bool ok, int n_chunks, uint32_t tmem,
                                                    int warp, int lane, int tok0, int ct, uint32_t kq, uint32_t rank) {
    constexpr int kPitch = 128 + 4;                               // floats per staged token row
    constexpr uint32_t kBlockBytes = 128 * kPitch * 4;            // 67584
    float *snd = reinterpret_cast<float *>(smem);                 // [128 tokens][kPitch]: what this CTA sends
    float *rcv = reinterpret_cast<float *>(smem + 68 * 1024);     // ... and what it receives
    const int tid = threadIdx.x;
    const int q = warp & 3, half = warp >> 2;
    const int row = q * 32 + lane, t = tok0 + row;
    const uint32_t trow = tmem + ((uint32_t)(q * 32) << 16);
    tc_fence_before();
    __syncthreads();
    cluster_sync_all();
    if (tid == 0) mbar_arrive_expect_tx(&B->xbar, kBlockBytes);
    if (warp < kLoaderWarps) {
        tc_fence_after();
        float *srow = snd + (size_t)row * kPitch + half * 64;
        for (int n0 = 0; n0 < 64; n0 += 16) {
            uint32_t v[16];
            if (n_chunks > 0) tmem_ld16(trow + (uint32_t)((1 - (int)kq) * 128 + half * 64 + n0), v);
#pragma unroll
            for (int i = 0; i < 4; ++i)
                *reinterpret_cast<uint4 *>(srow + n0 + 4 * i) = n_chunks > 0 ? make_uint4(v[4 * i], v[4 * i + 1], v[4 * i + 2], v[4 * i + 3])
                                                                              : make_uint4(0u, 0u, 0u, 0u);
        }
        tc_fence_before();
    }
    fence_async_proxy();                     // the staged block was written with ordinary stores; the copy reads it through the async proxy
    __syncthreads();
    if (tid == 0) {
        const uint32_t partner = ((1u - kq) << 1) | rank;
        bulk_copy_to_cta(map_to_cta(smem_u32(rcv), partner), snd, kBlockBytes, map_to_cta(smem_u32(&B->xbar), partner));
    }
    if (warp < kLoaderWarps) {
        const bool got = mbar_wait_cluster(&B->xbar, 0, P.spin_limit);
        if (!got && tid == 0 && P.status) atomicCAS(P.status, 0, SI_ERR_TIMEOUT);
        if (ok && got) {
            tc_fence_after();
            const size_t o0 = (size_t)t * P.d_model + (size_t)ct * 256 + kq * 128 + half * 64;
            for (int n0 = 0; n0 < 64; n0 += 16) {
                uint32_t v[16];
                if (n_chunks > 0) tmem_ld16(trow + (uint32_t)(kq * 128 + half * 64 + n0), v);
                if (t >= P.T) continue;
                const float *rv = rcv + (size_t)row * kPitch + half * 64 + n0;
                float a[16];
#pragma unroll
                for (int j = 0; j < 16; ++j) {
                    const float own = n_chunks > 0 ? __uint_as_float(v[j]) : 0.f;
                    a[j] = kq == 0 ? own + rv[j] : rv[j] + own;   // K half 0 first, whoever adds
                }
                down_store16(P, o0 + n0, a);
            }
        }
    }
}

// Down contraction: one pair per (N output columns, 256 tokens); N = 128 or 256, half of them per CTA.  KS = 2: a
// cluster of four CTAs -- two pairs -- works on a tile, each pair on half of K (N = 256 only).
template <int N, int KS>
__global__ void __cluster_dims__(2 * KS, 1, 1) __launch_bounds__(kGemmThreads, 1)
si_pair_down_kernel(const __grid_constant__ GemmParams P, const __grid_constant__ CUtensorMap h_map,
                    const __grid_constant__ CUtensorMap rec_map) {
    extern __shared__ __align__(1024) uint8_t smem[];
    constexpr int kHalfCols = N / 2;                              // output columns whose down rows this CTA loads
    constexpr int kWBytes = 64 * kHalfCols * 2;                   // 64 union entries x kHalfCols columns
    constexpr int stage_bytes = 128 * 128 + kWBytes;              // this CTA's H tile, its half of the down rows
    constexpr int kCopies = kWBytes / 16 / kLoaderThreads;        // 16-byte copies per loader thread and chunk (2 or 4)
    uint8_t *tiles = smem;
    PairBars *B = reinterpret_cast<PairBars *>(smem + (size_t)P.nstage * stage_bytes);
    volatile int *failed = &B->failed;
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    static_assert(KS == 1 || N == 256, "the K split finishes 128 columns per pair");
    const uint32_t crank = cluster_ctarank();
    const uint32_t rank = crank & 1u, kq = crank >> 1, leader = crank & ~1u;   // place in the pair, K share of the pair, first CTA of the pair
    constexpr uint32_t ncols = N;
    const uint32_t tmem = pair_setup(B, P.nstage, ncols, rank);
    bool ok = true;                             // (loader / epilogue threads) no wait of this thread ran out

    pdl_wait();                                 // H (and, through the gate/up kernel's own wait, the union)
    pdl_launch();
    const int tile = blockIdx.x / (2 * KS);
    const int col_tiles = P.d_model / N;
    const int ct = tile % col_tiles, tp = tile / col_tiles;
    const int n_u = *P.n_union;
    const int all_chunks = (n_u + kChunkK - 1) / kChunkK;         // 64 union entries per chunk
    const int per = (all_chunks + KS - 1) / KS;
    const int c_lo = (int)kq * per;                                // this pair's share of K
    const int n_chunks = all_chunks - c_lo < per ? (all_chunks > c_lo ? all_chunks - c_lo : 0) : per;
    const int tok0 = tp * kPairTokens + (int)rank * 128;
    // a union that is one run of consecutive slots (a static prefix, a whole layer) needs no gather: the down rows of
    // a chunk are tensor copies out of the record matrix (64 slots x 64 columns each)
    const int slot_first = P.union_slots[0];
    const bool run = all_chunks > 0 && P.union_slots[all_chunks * kChunkK - 1] - slot_first == all_chunks * kChunkK - 1;
    uint64_t *full = run ? B->full_t : B->full_g;

    if (warp < kLoaderWarps && run) {
        int armed = 0;
        if (lane == 0 && warp < 2) {         // two threads start the copies of alternate chunks
            const int col0 = 2 * P.d_model + ct * N + (int)rank * kHalfCols;
            for (int c = warp; c < n_chunks; c += 2) {
                const int st = c % P.nstage; const uint32_t ph = (c / P.nstage) & 1;
                if (!mbar_wait(&B->empty[st], ph ^ 1, P.spin_limit)) { *failed = 1; break; }
                uint8_t *stage = tiles + (size_t)st * stage_bytes;
                armed = c + 1;
                mbar_arrive_expect_tx(&full[st], (uint32_t)stage_bytes);
                tma_load_tile(stage, &h_map, (c_lo + c) * kChunkK, tok0, &full[st]);
#pragma unroll
                for (int hh = 0; hh < kHalfCols / 64; ++hh)
                    tma_load_tile(stage + 128 * 128 + hh * 8192, &rec_map, col0 + hh * 64, slot_first + (c_lo + c) * kChunkK, &full[st]);
                if (tp == 0 && c + kPrefetchAhead < n_chunks)
#pragma unroll
                    for (int hh = 0; hh < kHalfCols / 64; ++hh)
                        tma_prefetch_tile(&rec_map, col0 + hh * 64, slot_first + (c_lo + c + kPrefetchAhead) * kChunkK);
            }
        }
        ok = mbar_wait_relaxed(&B->accbar, 0, P.spin_limit, 256) && !*failed;
        if (!ok && armed > 0)                // a wait ran out: the tensor copies this thread started must still land before the CTA goes
            for (int c = armed - 1; c >= 0 && c > armed - 1 - P.nstage; c -= 2)
                mbar_wait(&full[c % P.nstage], (c / P.nstage) & 1, P.spin_limit);
        tc_fence_after();
        if (KS == 1) down_epilogue<N>(P, ok, n_chunks, tmem, warp, lane, tok0, ct);
        if (!ok && tid == 0 && P.status) atomicCAS(P.status, 0, SI_ERR_TIMEOUT);
    } else if (warp < kLoaderWarps) {
        // Copy j of a thread covers 16-byte piece `pc` of the down-row segment of chunk entry kk = kEntStep*j + e.
        // Entry kk, 64-column half hh, piece p land at hh*8192 + (kk >> 3)*1024 + (kk & 7)*128 + ((p ^ (kk & 7)) << 4):
        // the MN-major layout with 128-byte swizzle (8 entries x 64 columns per 1024-byte atom).
        constexpr int kPieces = kHalfCols * 2 / 16;               // 16-byte pieces per entry segment (8 or 16)
        constexpr int kEntStep = kLoaderThreads / kPieces;        // entries covered by one copy of all threads (32 or 16)
        const int pc = tid % kPieces, e = tid / kPieces;
        const int k8 = e & 7;
        const int dst0 = (pc >> 3) * 8192 + (e >> 3) * 1024 + k8 * 128 + (((pc & 7) ^ k8) << 4);
        const char *src0 = P.rec_base + (size_t)P.d_model * 4 + ((size_t)ct * N + (size_t)rank * kHalfCols) * 2 + pc * 16;
        int armed = 0;
        int slots_next[kCopies];                                   // union slots of the next chunk (fetched one chunk ahead)
#pragma unroll
        for (int j = 0; j < kCopies; ++j) slots_next[j] = n_chunks > 0 ? P.union_slots[c_lo * kChunkK + kEntStep * j + e] : 0;
        for (int c = 0; c < n_chunks; ++c) {
            const int st = c % P.nstage; const uint32_t ph = (c / P.nstage) & 1;
            int slots[kCopies];
#pragma unroll
            for (int j = 0; j < kCopies; ++j) {                     // padded entries carry a valid slot
                slots[j] = slots_next[j];
                if (c + 1 < n_chunks) slots_next[j] = P.union_slots[(c_lo + c + 1) * kChunkK + kEntStep * j + e];
            }
            if (!mbar_wait_relaxed(&B->empty[st], ph ^ 1, P.spin_limit, 32)) { *failed = 1; break; }
            uint8_t *stage = tiles + (size_t)st * stage_bytes;
#pragma unroll
            for (int j = 0; j < kCopies; ++j)
                cp_async16(stage + 128 * 128 + dst0 + j * (kEntStep / 8) * 1024, src0 + (size_t)slots[j] * P.rec_bytes);
            if (tid == 0) {
                armed = c + 1;
                mbar_arrive_expect_tx(&full[st], 128u * 128u);
                tma_load_tile(stage, &h_map, (c_lo + c) * kChunkK, tok0, &full[st]);
            }
            cp_async_arrive_when_landed(&full[st]);
        }
        cp_async_wait_all();
        ok = mbar_wait_relaxed(&B->accbar, 0, P.spin_limit, 256) && !*failed;
        if (!ok && armed > 0)                // a wait ran out: the tensor copies already started must still land before the CTA goes
            for (int c = armed - 1; c >= 0 && c > armed - 1 - P.nstage; --c)
                mbar_wait(&full[c % P.nstage], (c / P.nstage) & 1, P.spin_limit);
        tc_fence_after();
        if (KS == 1) down_epilogue<N>(P, ok, n_chunks, tmem, warp, lane, tok0, ct);
        if (!ok && tid == 0 && P.status) atomicCAS(P.status, 0, SI_ERR_TIMEOUT);
    } else if (lane == 0) {
        const uint32_t idesc = make_idesc(P.fmt, 0, 1, 256, N);
        const uint32_t sh = smem_u32(tiles), sw = sh + 128 * 128;
        uint64_t a0[4], b0[4];
#pragma unroll
        for (int k4 = 0; k4 < 4; ++k4) {       // 16 union entries per MMA = two 8-entry groups of 1024 bytes
            a0[k4] = make_desc(sh + k4 * 32, 16, 1024); b0[k4] = make_desc(sw + k4 * 2048, 8192, 1024);
        }
        pair_mma_loop(B, full, !run, n_chunks, P.nstage, P.spin_limit, rank, tmem, idesc, a0, b0, (uint32_t)stage_bytes, leader);
    }
    if (KS == 2) down_epilogue_split(P, smem, B, ok, n_chunks, tmem, warp, lane, tok0, ct, kq, rank);
    pair_teardown(tmem, ncols);
}

template <typename... KArgs, typename... Args>
cudaError_t launch_pair(void (*kern)(KArgs...), int ctas, size_t smem, cudaStream_t stream, Args... args) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(ctas); cfg.blockDim = dim3(kGemmThreads); cfg.dynamicSmemBytes = smem; cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr; cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, kern, KArgs(args)...);
}

int stages_for(size_t stage_bytes) {
    int n = (int)(((size_t)227 * 1024 - sizeof(PairBars) - 1024) / stage_bytes);
    return n > kPairMaxStages ? kPairMaxStages : n;
}

}  // namespace

// The kernel shapes of a call with T tokens (T > 128) whose union has room for nu_pad entries, on a device of num_sms
// SMs.  Host logic only.
//   gate/up: tiles of W = 128 or 96 neurons, or of two sub-tiles of 128 or 112: cost = waves of pair tiles over the SM
//            pairs x the MMA time of a tile's chunk (4 MMAs of N = 2 W per sub-tile: 4 S W cycles, plus what a stage
//            costs besides)
//   down:    256 columns per pair halve the H traffic of a column, 128 give twice the pairs.  When tiles of 256 columns
//            would leave most SM pairs without one, two pairs share a tile of 256, half of K each (a cluster of four
//            CTAs that exchanges its partial accumulators through distributed shared memory) -- as long as that is one
//            wave and K is long enough to pay for the exchange (measured at 512 tokens: 3 % ahead of the 128-column
//            tiles at 50 chunks of K, 18 % at 121); tiles of 128 columns otherwise.
void si_pair_plan(int d_model, int nu_pad, int T, int num_sms, si_pair_plan_t *plan) {
    const int tok_pairs = (T + kPairTokens - 1) / kPairTokens;
    const int slots = num_sms / 2;
    static const struct { int w, sub; } shapes[] = {{128, 1}, {96, 1}, {128, 2}, {112, 2}};
    long best_cost = -1;
    for (int i = 0; i < 4; ++i) {
        const int r = shapes[i].w * shapes[i].sub;
        const int pairs = ((nu_pad + r - 1) / r) * tok_pairs;
        const long cost = (long)((pairs + slots - 1) / slots) * (4 * r + 78);
        if (best_cost < 0 || cost < best_cost) {
            best_cost = cost; plan->gateup_w = shapes[i].w; plan->gateup_sub = shapes[i].sub; plan->gateup_pairs = pairs;
        }
    }
    const int tiles256 = d_model % 256 == 0 ? (d_model / 256) * tok_pairs : 0;
    const bool fills = tiles256 > 0 && tiles256 * 2 >= num_sms * 3 / 4;
    const bool split = tiles256 > 0 && !fills && tiles256 * 4 <= num_sms && nu_pad / kChunkK >= 32;
    plan->down_n = fills || split ? 256 : 128;
    plan->down_ksplit = split ? 2 : 1;
    plan->down_ctas = split ? 4 * tiles256 : (plan->down_n == 256 ? 2 * tiles256 : 2 * (d_model / 128) * tok_pairs);
}

bool si_pair_path_applies(const si_store *s, int T) {
    return T > 128 && s->d_model % 128 == 0;
}

// Both contractions of a call with more than 128 tokens, after the union stage (P holds the call's parameters;
// h_buf has room for t_pad_alloc x nu_pad 16-bit values).
int si_pair_contractions_launch(const si_store *s, GemmParams P, int n_loaded, void *h_buf, size_t h_bytes, cudaStream_t stream) {
    const int d = P.d_model;
    // H holds the tokens padded to 16 rows; a tile's rows past them are not written, and read as zero through the tensor map
    const int t_pad_alloc = (int)si_align_up((size_t)P.T, 16);
    if ((size_t)t_pad_alloc * P.nu_pad * 2 > h_bytes) return SI_ERR_NOMEM;
    P.t_pad_total = t_pad_alloc; P.n_tok = kPairTokens; P.n_split = 1;
    P.h = (const uint16_t *)h_buf; P.h_out = (uint16_t *)h_buf;
    si_pair_plan_t plan;
    si_pair_plan(d, P.nu_pad, P.T, s->num_sms, &plan);
    {
        const int w = plan.gateup_w, sub = plan.gateup_sub, best_pairs = plan.gateup_pairs;
        const size_t stage = 128 * 128 + (size_t)w * sub * 128;
        P.nstage = stages_for(stage);
        const size_t smem = (size_t)P.nstage * stage + sizeof(PairBars);
        CUtensorMap x_map, rec_map;
        int rc = make_tile_map(&x_map, P.x, (size_t)d, (size_t)P.T, (size_t)d * 2, 128);
        if (rc) return rc;
        rc = make_tile_map(&rec_map, P.rec_base, (size_t)3 * d, (size_t)n_loaded, (size_t)P.rec_bytes, w * sub);
        if (rc) return rc;
#define SI_LAUNCH_GATEUP(WW, SS)                                                                                                    \
        do {                                                                                                                        \
            SI_CUDA_TRY(cudaFuncSetAttribute(si_pair_gateup_kernel<WW, SS>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem)); \
            SI_CUDA_TRY(launch_pair(si_pair_gateup_kernel<WW, SS>, 2 * best_pairs, smem, stream, P, x_map, rec_map));               \
        } while (0)
        if (w == 128 && sub == 1) SI_LAUNCH_GATEUP(128, 1);
        else if (w == 96) SI_LAUNCH_GATEUP(96, 1);
        else if (w == 128) SI_LAUNCH_GATEUP(128, 2);
        else SI_LAUNCH_GATEUP(112, 2);
#undef SI_LAUNCH_GATEUP
    }
    {
        const int n = plan.down_n;
        const bool split = plan.down_ksplit == 2;
        P.pair_n = n;
        const size_t stage = 128 * 128 + (size_t)64 * n;
        P.nstage = stages_for(stage);
        const size_t smem = (size_t)P.nstage * stage + sizeof(PairBars);
        CUtensorMap h_map, rec_map;
        int rc = make_tile_map(&h_map, h_buf, (size_t)P.nu_pad, (size_t)t_pad_alloc, (size_t)P.nu_pad * 2, 128);
        if (rc) return rc;
        rc = make_tile_map(&rec_map, P.rec_base, (size_t)3 * d, (size_t)n_loaded, (size_t)P.rec_bytes, 64);
        if (rc) return rc;
        if (split) {
            SI_CUDA_TRY(cudaFuncSetAttribute(si_pair_down_kernel<256, 2>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
            SI_CUDA_TRY(launch_pair(si_pair_down_kernel<256, 2>, plan.down_ctas, smem, stream, P, h_map, rec_map));
        } else if (n == 256) {
            SI_CUDA_TRY(cudaFuncSetAttribute(si_pair_down_kernel<256, 1>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
            SI_CUDA_TRY(launch_pair(si_pair_down_kernel<256, 1>, plan.down_ctas, smem, stream, P, h_map, rec_map));
        } else {
            SI_CUDA_TRY(cudaFuncSetAttribute(si_pair_down_kernel<128, 1>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
            SI_CUDA_TRY(launch_pair(si_pair_down_kernel<128, 1>, plan.down_ctas, smem, stream, P, h_map, rec_map));
        }
    }
    SI_CUDA_TRY(cudaGetLastError());
    return SI_OK;
}
