// Multi-token path (T > 1: batched decode and prefill): the union of the tokens' active lists
// is formed once, and the selective FFN over the union runs as two gathered dense contractions
// on the 5th-generation tensor cores (tcgen05.mma, accumulators in tensor memory):
//
//   union      U = sorted union of the T lists, mask[t] = which entries of U token t selected
//   gate/up    G^T, Up^T [|U| x T] = W_gate[U, :] . X^T, W_up[U, :] . X^T     (K = d_model)
//   combine    H[t, i] = mask[t, i] ? SiLU(G[i, t]) * Up[i, t] : 0, rounded to the store dtype (fused)
//   down       Y^T [d_model x T] = W_down[:, U] . H^T                          (K = |U|)
//
// Token t therefore uses exactly its own list (Section 5 applied per token), whatever the
// other tokens selected; with SI_FLAG_UNION_UNMASKED every token uses the whole union.
//
// Tiling (this file: up to 128 tokens -- batched decode; calls with more tokens run on CTA pairs, si_gemm_pair.cu).
// Both contractions put the weight side on the MMA M dimension (128 rows of the store per tile) and the tokens
// on N (T padded to 16), so the weights -- the dominant bytes -- are read exactly once.  Weight rows are gathered
// straight out of the neuron records with 16-byte cp.async copies into the 128-byte-swizzled shared memory
// layouts the MMA descriptors expect (gate/up rows are K-major, down rows MN-major).  K is split among the CTAs
// of a thread-block cluster (1, 2, 4 or 8 per tile) so that small unions still fill the machine; the CTAs of a
// cluster sum their partial accumulators through distributed shared memory, in rank order -- so results do not
// depend on timing --, and the finishing passes (combine, residual, rounding) run on the summed tile: there are
// no partial tiles in global memory, no counters and no kernels for the finishing passes.
#include "si_tc.cuh"

using namespace si_tc;

namespace {

// ------------------------------------------------------------------------------- union
// sh[0 .. words) holds the bitmap; sh[words .. 2*words + 2) is scratch.  Writes the ascending union, its
// size, and pads the list up to union_cap with valid slots.
__device__ __forceinline__ void union_scan_emit(uint32_t *sh, uint32_t *warp_tot, int words, int n_loaded, int32_t *__restrict__ union_out,
                                                int32_t *__restrict__ n_union_out, int union_cap) {
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    uint32_t *bitmap = sh;                         // [words]
    uint32_t *wprefix = sh + words;                // [words] exclusive popcount prefix
    uint32_t carry = 0;
    for (int base = 0; base < words; base += 1024) {
        int w = base + tid;
        uint32_t c = w < words ? __popc(bitmap[w]) : 0u;
        uint32_t inc = c;
        for (int o = 1; o < 32; o <<= 1) { uint32_t t = __shfl_up_sync(0xFFFFFFFFu, inc, o); if (lane >= o) inc += t; }
        if (lane == 31) warp_tot[warp] = inc;
        __syncthreads();
        if (warp == 0) {
            uint32_t v = warp_tot[lane], vi = v;
            for (int o = 1; o < 32; o <<= 1) { uint32_t t = __shfl_up_sync(0xFFFFFFFFu, vi, o); if (lane >= o) vi += t; }
            warp_tot[lane] = vi - v;
            if (lane == 31) sh[2 * words] = vi;    // total of this block of words
        }
        __syncthreads();
        if (w < words) wprefix[w] = carry + warp_tot[warp] + inc - c;
        carry += sh[2 * words];
        __syncthreads();
    }
    const int n_u = (int)carry;
    if (tid == 0) *n_union_out = n_u;
    // one slot per thread and round: a set bit's position in the union is its word's prefix plus the set
    // bits below it in the word -- no chain from one entry to the next
    for (int i = tid; i < words * 32; i += 1024) {
        const uint32_t bits = bitmap[i >> 5], below = (1u << (i & 31)) - 1u;
        if ((bits >> (i & 31)) & 1u) {
            const int p = (int)wprefix[i >> 5] + __popc(bits & below);
            if (p < union_cap) union_out[p] = i;
        }
    }
    {
        // Padding.  The slots that follow the last entry, as long as they exist: a union that is a run of consecutive
        // slots (a static prefix, a whole layer) stays one over its padding, and tiles of consecutive slots are fetched
        // by tensor copies.  Past the last loaded slot: the first entry.  (Padded positions contribute nothing.)
        int first = 0, last = 0;
        for (int w = 0; w < words; ++w) if (bitmap[w]) { first = w * 32 + __ffs(bitmap[w]) - 1; break; }
        for (int w = words - 1; w >= 0; --w) if (bitmap[w]) { last = w * 32 + 31 - __clz(bitmap[w]); break; }
        for (int p = n_u + tid; p < union_cap; p += 1024) {
            const int v = last + 1 + (p - n_u);
            union_out[p] = v < n_loaded ? v : first;
        }
    }
}

// Sorted union of the lists in one launch.  Every block ORs its share of the list entries into a
// bitmap over the loaded slots and -- when each token has its own list -- into that token's own
// slot bitmap (membership test of the combine step).  The block that finishes last turns the
// bitmap into the ascending union by a popcount prefix scan.  bitmap, tokbits and ticket are zero
// on entry.  blockDim.x = 1024; dynamic shared memory = (2 * words + 2) * 4 bytes.
__global__ void __launch_bounds__(1024)
si_union_build_kernel(const int32_t *__restrict__ idx, const int32_t *__restrict__ offsets, int k_fixed, int n_lists,
                      int n_loaded, uint32_t *bitmap_g, uint32_t *tokbits, int mask_words, unsigned *ticket,
                      int32_t *__restrict__ union_out, int32_t *__restrict__ n_union_out, int union_cap, int32_t *status) {
    extern __shared__ uint32_t sh[];
    __shared__ uint32_t warp_tot[32];
    __shared__ int is_last;
    const int tid = threadIdx.x;
    pdl_launch();
    const long long total = offsets ? offsets[n_lists] : (long long)n_lists * k_fixed;
    for (long long e = (long long)blockIdx.x * blockDim.x + tid; e < total; e += (long long)gridDim.x * blockDim.x) {
        const int s = idx[e];
        if (s < 0 || s >= n_loaded) { if (status) atomicCAS(status, 0, SI_ERR_OUT_OF_RANGE); continue; }
        const uint32_t bit = 1u << (s & 31);
        if (!(bitmap_g[s >> 5] & bit)) atomicOr(&bitmap_g[s >> 5], bit);     // hot slots are set by the first token
        if (tokbits) {
            int t;
            if (offsets) {            // largest t with offsets[t] <= e
                int lo = 0, hi = n_lists;
                while (hi - lo > 1) { int mid = (lo + hi) >> 1; if (offsets[mid] <= e) lo = mid; else hi = mid; }
                t = lo;
            } else {
                t = (int)(e / k_fixed);
            }
            atomicOr(&tokbits[(size_t)t * mask_words + (s >> 5)], bit);
        }
    }
    __threadfence();
    __syncthreads();
    if (tid == 0) is_last = atomicAdd(ticket, 1u) == gridDim.x - 1;
    __syncthreads();
    if (!is_last) return;
    __threadfence();

    // ---- last block: popcount prefix scan over the bitmap -> ascending union
    const int words = (n_loaded + 31) / 32;
    for (int w = tid; w < words; w += 1024) sh[w] = __ldcg(bitmap_g + w);
    __syncthreads();
    union_scan_emit(sh, warp_tot, words, n_loaded, union_out, n_union_out, union_cap);
}

// The same result from one block, for calls with few list entries and few lists: the union's bitmap and
// the tokens' bitmaps are built in shared memory (no global atomics, nothing to clear beforehand: every
// word of the token bitmaps is written once, with plain stores), all list entries of a thread are loaded
// before the first is used and merged per bitmap word in registers, the block clears the arrival counters the later kernels expect to be zero
// (no memset node), and nothing has to cross blocks.  Dynamic shared memory: (2 * words + 2 + n_lists *
// mask_words) * 4 bytes (the last term only with tokbits).
constexpr int kUnionSmallBatch = 16;           // list entries per thread in flight
__global__ void __launch_bounds__(1024)
si_union_small_kernel(const int32_t *__restrict__ idx, const int32_t *__restrict__ offsets, int k_fixed, int n_lists,
                      int n_loaded, uint32_t *zero_g, int zero_words, uint32_t *tokbits, int mask_words,
                      int32_t *__restrict__ union_out, int32_t *__restrict__ n_union_out, int union_cap, int32_t *status) {
    extern __shared__ uint32_t sh[];
    __shared__ uint32_t warp_tot[32];
    const int tid = threadIdx.x;
    pdl_launch();
    const int words = (n_loaded + 31) / 32;
    uint32_t *tok_s = sh + 2 * words + 2;                          // [n_lists][mask_words]
    const int tok_words = tokbits ? n_lists * mask_words : 0;
    const int total = offsets ? offsets[n_lists] : n_lists * k_fixed;
    // thread t takes the consecutive entries [t * per, (t + 1) * per): a list is ascending, so its entries
    // fall into the same bitmap word several in a row, and the thread collects their bits in a register
    // and updates shared memory once per (list, word) run
    // (longer inputs take several rounds of kUnionSmallBatch entries per thread)
    const int rounds = (total + 1024 * kUnionSmallBatch - 1) / (1024 * kUnionSmallBatch);
    const int per = rounds > 1 ? kUnionSmallBatch : (total + 1023) / 1024;
    for (int w = tid; w < zero_words; w += 1024) zero_g[w] = 0u;
    for (int w = tid; w < words; w += 1024) sh[w] = 0u;
    for (int w = tid; w < tok_words; w += 1024) tok_s[w] = 0u;
    __syncthreads();
    for (int round = 0; round < (rounds > 0 ? rounds : 1); ++round) {
        const int e_lo = round * 1024 * kUnionSmallBatch + tid * per;
        int sl[kUnionSmallBatch];
#pragma unroll
        for (int j = 0; j < kUnionSmallBatch; ++j) { const int e = e_lo + j; sl[j] = (j < per && e < total) ? idx[e] : -1; }
        int t = 0, t_end = 0;                                      // list of the current entry, first entry past it
        if (e_lo < total) {
            if (offsets) {            // largest t with offsets[t] <= e_lo
                int lo = 0, hi = n_lists;
                while (hi - lo > 1) { int mid = (lo + hi) >> 1; if (offsets[mid] <= e_lo) lo = mid; else hi = mid; }
                t = lo; t_end = offsets[t + 1];
            } else {
                t = e_lo / k_fixed; t_end = (t + 1) * k_fixed;
            }
        }
        int cur_w = -1, cur_t = 0;
        uint32_t cur_bits = 0;
        auto flush = [&]() {
            if (cur_w >= 0) {
                if ((sh[cur_w] & cur_bits) != cur_bits) atomicOr(&sh[cur_w], cur_bits);     // hot slots are set by the first token
                if (tokbits) atomicOr(&tok_s[cur_t * mask_words + cur_w], cur_bits);
            }
        };
#pragma unroll
        for (int j = 0; j < kUnionSmallBatch; ++j) {
            const int e = e_lo + j, sv = sl[j];
            if (j >= per || e >= total) continue;
            while (e >= t_end) { ++t; t_end = offsets ? offsets[t + 1] : t_end + k_fixed; }   // next list (empty ones skipped)
            if (sv < 0 || sv >= n_loaded) { if (status) atomicCAS(status, 0, SI_ERR_OUT_OF_RANGE); continue; }
            const int w = sv >> 5;
            if (w != cur_w || t != cur_t) { flush(); cur_w = w; cur_t = t; cur_bits = 0; }
            cur_bits |= 1u << (sv & 31);
        }
        flush();
    }
    __syncthreads();
    for (int w = tid; w < tok_words; w += 1024) tokbits[w] = tok_s[w];
    union_scan_emit(sh, warp_tot, words, n_loaded, union_out, n_union_out, union_cap);
    // This kernel reads the caller's lists and writes a copy of the union stage's outputs that nothing else is
    // using, so it may run while the kernel before it in the stream (the down contraction of the call before)
    // still works.  It ends only after that kernel has: whoever waits for this kernel's results then also sees
    // everything that kernel wrote (the next gate/up contraction may read, as its x, the y of the call before).
    pdl_wait();
}

// ------------------------------------------------------------------------------- contractions
// Gate/up contraction.  One CTA per (union tile of 128, K split of d_model, token tile), flat grid.
// D_gate[128 neurons x N tokens] (+)= Wg[U tile, k] . X[tokens, k]^T, same for up, accumulated in
// tensor memory (columns [0,N) gate, [N,2N) up).
__global__ void __launch_bounds__(320, 2)   // kGemmThreads = 288 threads are launched; 320 caps the registers at 96

si_gemm_gateup_kernel(const __grid_constant__ GemmParams P, const __grid_constant__ CUtensorMap x_map,
                      const __grid_constant__ CUtensorMap rec_map) {
    extern __shared__ __align__(1024) uint8_t smem[];
    const int N = P.n_tok;
    const int stage_bytes = 2 * 128 * 128 + N * 128;              // gate tile, up tile, x tile
    uint8_t *tiles = smem;
    uint64_t *full = reinterpret_cast<uint64_t *>(smem + (size_t)P.nstage * stage_bytes);
    uint64_t *empty = full + kMaxStages;
    uint64_t *accbar = empty + kMaxStages;
    uint32_t *tmem_slot = reinterpret_cast<uint32_t *>(accbar + 1);
    volatile int *failed = reinterpret_cast<volatile int *>(tmem_slot + 1);

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    // ---- set-up that needs nothing from the union kernel (runs while that kernel finishes)
    uint32_t ncols = 32; while (ncols < (uint32_t)(2 * N)) ncols <<= 1;
    if (tid == 0) {
        for (int s = 0; s < P.nstage; ++s) { mbar_init(&full[s], kLoaderThreads + 1); mbar_init(&empty[s], 1); }
        mbar_init(accbar, 1);
        *failed = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == kLoaderWarps) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_slot)), "r"(ncols) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = *tmem_slot;

    // Flat grid sized on the host for the largest possible union: one thread-block cluster per union tile of 128,
    // whose CTAs split K = d_model among themselves (cluster size = P.n_split, chosen on the host).  The real union
    // is known here; the clusters of tiles past it leave at once.
    pdl_wait();                                 // the union kernel's results
    pdl_launch();
    const int n_u = *P.n_union;
    const int n_real = n_u > 128 ? (n_u + 127) / 128 : 1;
    const int ns = P.n_split;
    const int ks = ns > 1 ? (int)cluster_ctarank() : 0, mt = blockIdx.x / ns, tt = 0;
    if (mt >= n_real) {
        if (warp == kLoaderWarps)
            asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(ncols) : "memory");
        return;
    }
    bool ok = true;                             // (loader / epilogue threads) no wait of this thread ran out
    const int total_k = P.d_model / kChunkK;                       // chunks; split ks takes an even share of them
    const int c0 = (int)((long long)ks * total_k / ns), c1 = (int)((long long)(ks + 1) * total_k / ns);
    const int n_chunks = c1 > c0 ? c1 - c0 : 0;
    const int tok0 = tt * N;

    if (warp < kLoaderWarps) {
        // ---------------------------------------------------------------- gather loads
        // Copy j of a thread covers 16-byte piece (tid & 7) of tile row 32*j + (tid >> 3): the 32 lanes
        // of a warp instruction read four whole 128-byte row segments, so the gather is coalesced.
        // All addresses advance by constants, so a chunk costs a handful of instructions per copy.
        const int q8 = tid & 7, r32 = tid >> 3;
        const char *grow[4];                                         // gate rows; the up row follows at d_model*2
#pragma unroll
        for (int j = 0; j < 4; ++j)
            grow[j] = P.rec_base + (size_t)P.union_slots[mt * 128 + 32 * j + r32] * P.rec_bytes + q8 * 16 + (size_t)c0 * 128;
        const int off0 = r32 * 128 + ((q8 ^ (r32 & 7)) << 4);      // rows 32*j + r32 share (row & 7)
        const size_t up_off = (size_t)P.d_model * 2;
        // A tile whose 128 union entries are consecutive slots (a static prefix, a whole layer) needs no
        // gather: its gate and up tiles are two TMA copies out of the record matrix
        const int slot_first = P.union_slots[mt * 128];
        const bool run = P.union_slots[mt * 128 + 127] - slot_first == 127;
        int armed = 0;                       // (thread 0) chunks whose tensor copies it has started
        for (int c = 0; c < n_chunks; ++c) {
            const int st = c % P.nstage; const uint32_t ph = (c / P.nstage) & 1;
            if (!mbar_wait(&empty[st], ph ^ 1, P.spin_limit)) { *failed = 1; break; }
            uint8_t *sg = tiles + (size_t)st * stage_bytes + off0, *su = sg + 128 * 128;
            if (!run) {
#pragma unroll
                for (int j = 0; j < 4; ++j) {
                    cp_async16(sg + j * 4096, grow[j]);
                    cp_async16(su + j * 4096, grow[j] + up_off);
                    grow[j] += 128;
                }
            }
            if (tid == 0) armed = c + 1;
            if (tid == 0 && !(P.withhold && blockIdx.x == 0 && c == 0)) {      // the dense X tile comes as one TMA copy (token rows past T read as zero)
                uint8_t *stage = tiles + (size_t)st * stage_bytes;
                mbar_arrive_expect_tx(&full[st], (uint32_t)N * 128u + (run ? 2u * 128u * 128u : 0u));
                if (run) {
                    tma_load_tile(stage, &rec_map, (c0 + c) * kChunkK, slot_first, &full[st]);
                    tma_load_tile(stage + 128 * 128, &rec_map, P.d_model + (c0 + c) * kChunkK, slot_first, &full[st]);
                }
                tma_load_tile(stage + 2 * 128 * 128, &x_map, (c0 + c) * kChunkK, tok0, &full[st]);
            }
            cp_async_arrive_when_landed(&full[st]);
        }
        cp_async_wait_all();                 // nothing of this thread may still be in flight when the CTA ends
        // ---------------------------------------------------------------- epilogue
        ok = mbar_wait(accbar, 0, P.spin_limit) && !*failed;
        if (!ok && tid == 0)                 // a wait ran out: the tensor copies already started must still land before the CTA goes
            for (int c = armed > P.nstage ? armed - P.nstage : 0; c < armed; ++c)
                if (!(P.withhold && blockIdx.x == 0 && c == 0)) mbar_wait(&full[c % P.nstage], (c / P.nstage) & 1, P.spin_limit);
        tc_fence_after();
        // a warp reads tensor-memory lanes 32*(warp % 4) ..: warps w and w + 4 share the rows and take
        // alternate 16-column blocks.  Thread row r = union row mt*128 + r: N gate values, N up values
        const int r = (warp & 3) * 32 + lane, cb = warp >> 2;
        if (ok && ns == 1) {
            // whole K in this CTA: form H straight from the accumulators (no partial tiles); the tile is
            // staged in shared memory -- every MMA has finished reading the stages -- and written out below
            constexpr int kRowPitch = 128 + 8;
            uint16_t *hs = reinterpret_cast<uint16_t *>(smem);
            const int i = mt * 128 + r;
            const int slot = P.union_slots[i];
            for (int n0 = 16 * cb; n0 < N; n0 += 32) {
                uint32_t g[16], u[16];
                tmem_ld16(tmem + ((uint32_t)((warp & 3) * 32) << 16) + (uint32_t)n0, g);
                tmem_ld16(tmem + ((uint32_t)((warp & 3) * 32) << 16) + (uint32_t)(N + n0), u);
                // (no branch per element: SiLU(g) * u is formed for every element and kept or zeroed by a select)
                uint32_t member = 0;                               // bit q: token n0 + q uses this row's neuron
                if (n_chunks > 0 && i < n_u) {
#pragma unroll
                    for (int q = 0; q < 16; ++q) {
                        const int t = tok0 + n0 + q;
                        const uint32_t bit = P.tokbits ? (P.tokbits[(size_t)(t < P.T ? t : 0) * P.mask_words + (slot >> 5)] >> (slot & 31)) & 1u : 1u;
                        member |= (t < P.T ? bit : 0u) << q;
                    }
                }
#pragma unroll
                for (int q = 0; q < 16; ++q) {
                    const float v = si_silu_mul(__uint_as_float(g[q]), __uint_as_float(u[q]));
                    const uint16_t hb = P.fmt ? si_cvt<SI_BF16>::from_float(v) : si_cvt<SI_F16>::from_float(v);
                    hs[(n0 + q) * kRowPitch + r] = (member >> q) & 1u ? hb : (uint16_t)0;
                }
            }
        }
        if (!ok && tid == 0 && P.status) atomicCAS(P.status, 0, SI_ERR_TIMEOUT);
    } else {
        // ---------------------------------------------------------------- MMA issue (one thread)
        if (lane == 0) {
            const uint32_t idesc = make_idesc(P.fmt, 0, 0, 128, N);
            bool ok = true;
            for (int c = 0; c < n_chunks && ok; ++c) {
                const int st = c % P.nstage; const uint32_t ph = (c / P.nstage) & 1;
                ok = mbar_wait(&full[st], ph, P.spin_limit) && !*failed;
                if (!ok) break;
                fence_async_proxy();               // the gathered rows were written by cp.async (generic proxy)
                tc_fence_after();
                const uint32_t sg = smem_u32(tiles + (size_t)st * stage_bytes), su = sg + 128 * 128, sx = su + 128 * 128;
#pragma unroll
                for (int k4 = 0; k4 < 4; ++k4) {
                    const uint64_t bd = make_desc(sx + k4 * 32, 16, 1024);
                    umma(tmem, make_desc(sg + k4 * 32, 16, 1024), bd, idesc, (c | k4) ? 1u : 0u);
                    umma(tmem + (uint32_t)N, make_desc(su + k4 * 32, 16, 1024), bd, idesc, (c | k4) ? 1u : 0u);
                }
                umma_commit(&empty[st]);          // the stage may be refilled once these MMAs have read it
            }
            if (!ok) *failed = 1;
            umma_commit(accbar);                  // accumulators complete (or nothing was issued)
        }
    }
    tc_fence_before();
    __syncthreads();
    if (ns > 1) {
        // ---- K split across the cluster: the partial accumulators are summed through distributed shared memory.
        // CTA j of the cluster owns the tile's rows [j * 128 / ns, (j + 1) * 128 / ns): every CTA writes its partial
        // values of those rows into slot (its rank) of CTA j's staging area (the pipeline stages, free once every
        // CTA's MMAs are complete: first cluster barrier), and after the second barrier CTA j sums the slots in rank
        // order -- so H does not depend on timing -- and forms H for its rows.
        const int rows_per = 128 / ns, pitch = 2 * N + 4;            // floats per staged row: N gate, N up, padding
        float *stg = reinterpret_cast<float *>(smem);                // [ns][rows_per][pitch]
        cluster_sync_all();
        if (warp < kLoaderWarps && ok) {
            tc_fence_after();
            const int r = (warp & 3) * 32 + lane, cb = warp >> 2;
            const uint32_t dst = map_to_cta(smem_u32(stg + ((size_t)ks * rows_per + (r % rows_per)) * pitch), (uint32_t)(r / rows_per));
            for (int n0 = 16 * cb; n0 < 2 * N; n0 += 32) {           // columns [0, N) gate, [N, 2N) up
                uint32_t v[16];
                if (n_chunks > 0) tmem_ld16(tmem + ((uint32_t)((warp & 3) * 32) << 16) + (uint32_t)n0, v);
#pragma unroll
                for (int q = 0; q < 4; ++q)
                    st_cluster_v4(dst + (uint32_t)(n0 + 4 * q) * 4u, n_chunks > 0 ? v[4 * q] : 0u, n_chunks > 0 ? v[4 * q + 1] : 0u,
                                  n_chunks > 0 ? v[4 * q + 2] : 0u, n_chunks > 0 ? v[4 * q + 3] : 0u);
            }
        }
        tc_fence_before();
        cluster_sync_all();
        if (!*failed) {
            // one item = (token n, row rr of this CTA's rows): consecutive threads take consecutive rows, so a
            // token's H values are written side by side
            for (int it = tid; it < rows_per * N; it += kGemmThreads) {
                const int n = it / rows_per, rr = it - n * rows_per;
                const int i = mt * 128 + ks * rows_per + rr, t = tok0 + n;
                float g = 0.f, u = 0.f;
                for (int sp = 0; sp < ns; ++sp) {
                    const float *row = stg + ((size_t)sp * rows_per + rr) * pitch;
                    g += row[n]; u += row[N + n];
                }
                bool member = i < n_u && t < P.T;
                if (member && P.tokbits) {
                    const int slot = P.union_slots[i];
                    member = (P.tokbits[(size_t)t * P.mask_words + (slot >> 5)] >> (slot & 31)) & 1u;
                }
                const float v = si_silu_mul(g, u);
                const uint16_t hb = P.fmt ? si_cvt<SI_BF16>::from_float(v) : si_cvt<SI_F16>::from_float(v);
                P.h_out[(size_t)t * P.nu_pad + i] = member ? hb : (uint16_t)0;
            }
        }
    }
    if (warp == kLoaderWarps) {
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(ncols) : "memory");
    }
    if (ns == 1 && !*failed) {
        // the tile staged by the epilogue: H is [token][position]
        constexpr int kRowPitch = 128 + 8;                           // uint16 per token row of the staging tile
        const uint16_t *hs = reinterpret_cast<const uint16_t *>(smem);
        for (int e = tid; e < N * 16; e += kGemmThreads) {
            const int n = e >> 4, piece = e & 15;
            *reinterpret_cast<uint4 *>(P.h_out + (size_t)(tok0 + n) * P.nu_pad + (size_t)mt * 128 + piece * 8) =
                *reinterpret_cast<const uint4 *>(hs + n * kRowPitch + piece * 8);
        }
    }
}

// Down contraction.  grid = (d_model / 128 column tiles, K splits over the union, token tiles).
// D[128 output columns x N tokens] (+)= Wd[U_k, columns]^T . H[tokens, U_k]^T: A is MN-major (a
// down row is contiguous along the output columns), B is K-major.
__global__ void __launch_bounds__(320, 2)   // kGemmThreads = 288 threads are launched; 320 caps the registers at 96

si_gemm_down_kernel(const __grid_constant__ GemmParams P, const __grid_constant__ CUtensorMap h_map) {
    extern __shared__ __align__(1024) uint8_t smem[];
    const int N = P.n_tok;
    const int stage_bytes = 64 * 256 + N * 128;                   // 64 down-row segments of 128 columns, H tile
    uint8_t *tiles = smem;
    uint64_t *full = reinterpret_cast<uint64_t *>(smem + (size_t)P.nstage * stage_bytes);
    uint64_t *empty = full + kMaxStages;
    uint64_t *accbar = empty + kMaxStages;
    uint32_t *tmem_slot = reinterpret_cast<uint32_t *>(accbar + 1);
    volatile int *failed = reinterpret_cast<volatile int *>(tmem_slot + 1);

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    // grid = (column tiles, K splits): the CTAs of a column tile form a thread-block cluster along y
    const int mt = blockIdx.x, ks = blockIdx.y, tt = 0;
    bool ok = true;                             // (loader / epilogue threads) no wait of this thread ran out
    // ---- set-up that needs nothing from the gate/up kernel (runs while that kernel finishes)
    uint32_t ncols = 32; while (ncols < (uint32_t)N) ncols <<= 1;
    if (tid == 0) {
        for (int s = 0; s < P.nstage; ++s) { mbar_init(&full[s], kLoaderThreads + 1); mbar_init(&empty[s], 1); }
        mbar_init(accbar, 1);
        *failed = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == kLoaderWarps) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_slot)), "r"(ncols) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = *tmem_slot;

    // The gate/up kernel lets this kernel start only after the union kernel has completed, so the union
    // and the down rows it names can be read at once; only H has to wait for the gate/up kernel.
    pdl_launch();                               // the union stage of the next call may be scheduled (it writes other buffers)
    const int n_u = *P.n_union;
    const int total_chunks = (n_u + kChunkK - 1) / kChunkK;        // 64 union entries per chunk
    const int k_per = (total_chunks + P.n_split - 1) / P.n_split;
    const int c0 = ks * k_per, c1 = min(total_chunks, c0 + k_per);
    const int n_chunks = c1 > c0 ? c1 - c0 : 0;
    const int tok0 = tt * N;

    if (warp < kLoaderWarps) {
        // Copy j of a thread covers 16-byte piece (tid & 15) of the 256-byte down-row segment of union
        // entry 16*j + (tid >> 4) of the chunk: a warp instruction reads two whole segments (coalesced).
        const int c16 = tid & 15, e16 = tid >> 4;
        int slots_next[4];                                           // union slots of the next chunk (prefetched)
#pragma unroll
        for (int j = 0; j < 4; ++j)
            slots_next[j] = n_chunks > 0 ? P.union_slots[c0 * kChunkK + 16 * j + e16] : 0;
        // entry kk = 16*j + e16 lands at (kk >> 3) * 2048 + half * 1024 + (kk & 7) * 128 + swizzled piece
        const int k8 = e16 & 7;
        const int dst0 = (e16 >> 3) * 2048 + (c16 >> 3) * 1024 + k8 * 128 + (((c16 & 7) ^ k8) << 4);
        const char *dsrc0 = P.rec_base + (size_t)P.d_model * 4 + (size_t)mt * 256 + c16 * 16;
        // the down rows of the first chunks (one per stage: the ring is empty) are fetched while the
        // gate/up kernel finishes
        const int pre = n_chunks < P.nstage ? n_chunks : P.nstage;
        int armed_to = 0; bool h_primed = false;     // (thread 0) H tiles started: the primed ones, then up to chunk armed_to
        for (int c = 0; c < n_chunks; ++c) {
            const int st = c % P.nstage; const uint32_t ph = (c / P.nstage) & 1;
            int slots[4];
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                slots[j] = slots_next[j];
                if (c + 1 < n_chunks) slots_next[j] = P.union_slots[(c0 + c + 1) * kChunkK + 16 * j + e16];
            }
            if (c == pre) {      // (n_chunks > nstage) the ring is primed: now H is needed
                pdl_wait();
                h_primed = true;
                if (tid == 0)
                    for (int q = 0; q < pre; ++q) {
                        mbar_arrive_expect_tx(&full[q], (uint32_t)N * 128u);
                        tma_load_tile(tiles + (size_t)q * stage_bytes + 64 * 256, &h_map, (c0 + q) * kChunkK, tok0, &full[q]);
                    }
            }
            if (c >= pre && !mbar_wait(&empty[st], ph ^ 1, P.spin_limit)) { *failed = 1; break; }
            uint8_t *sa = tiles + (size_t)st * stage_bytes;
#pragma unroll
            for (int j = 0; j < 4; ++j)                                      // padded entries carry a valid slot
                cp_async16(sa + j * 4096 + dst0, dsrc0 + (size_t)slots[j] * P.rec_bytes);
            if (c >= pre && tid == 0) {      // the dense H tile comes as one TMA copy
                armed_to = c + 1;
                mbar_arrive_expect_tx(&full[st], (uint32_t)N * 128u);
                tma_load_tile(sa + 64 * 256, &h_map, (c0 + c) * kChunkK, tok0, &full[st]);
            }
            cp_async_arrive_when_landed(&full[st]);
        }
        if (n_chunks <= pre) {   // short K range: everything was primed above
            pdl_wait();
            h_primed = true;
            if (tid == 0)
                for (int q = 0; q < pre; ++q) {
                    mbar_arrive_expect_tx(&full[q], (uint32_t)N * 128u);
                    tma_load_tile(tiles + (size_t)q * stage_bytes + 64 * 256, &h_map, (c0 + q) * kChunkK, tok0, &full[q]);
                }
        }
        cp_async_wait_all();                 // nothing of this thread may still be in flight when the CTA ends
        ok = mbar_wait(accbar, 0, P.spin_limit) && !*failed;
        if (!ok && tid == 0) {               // a wait ran out: the tensor copies already started must still land before the CTA goes
            const int armed = armed_to > pre ? armed_to : (h_primed ? pre : 0);
            for (int c = armed > P.nstage ? armed - P.nstage : 0; c < armed; ++c)
                mbar_wait(&full[c % P.nstage], (c / P.nstage) & 1, P.spin_limit);
        }
        tc_fence_after();
        // thread holds output column mt*128 + r for the tokens; warps w and w + 4 share the rows and
        // take alternate 16-token blocks
        const int r = (warp & 3) * 32 + lane, cb = warp >> 2;
        if (ok && P.n_split == 1) {
            // whole K in this CTA: write y straight from the accumulators (a warp writes 32 consecutive
            // columns of one token at a time)
            const int col = mt * 128 + r;
            for (int n0 = 16 * cb; n0 < N; n0 += 32) {
                uint32_t v[16];
                if (n_chunks > 0) tmem_ld16(tmem + ((uint32_t)((warp & 3) * 32) << 16) + (uint32_t)n0, v);
#pragma unroll
                for (int q = 0; q < 16; ++q) {
                    const int t = tok0 + n0 + q;
                    if (t >= P.T) continue;
                    const size_t o = (size_t)t * P.d_model + col;
                    float a = n_chunks > 0 ? __uint_as_float(v[q]) : 0.f;
                    if (P.residual) a += P.fmt ? si_cvt<SI_BF16>::lo((uint32_t)P.x[o]) : si_cvt<SI_F16>::lo((uint32_t)P.x[o]);
                    if (P.y_f32) reinterpret_cast<float *>(P.y)[o] = a;
                    else reinterpret_cast<uint16_t *>(P.y)[o] = P.fmt ? si_cvt<SI_BF16>::from_float(a) : si_cvt<SI_F16>::from_float(a);
                }
            }
        }
        if (!ok && tid == 0 && P.status) atomicCAS(P.status, 0, SI_ERR_TIMEOUT);
    } else {
        pdl_wait();
        if (lane == 0) {
            const uint32_t idesc = make_idesc(P.fmt, 1, 0, 128, N);
            bool ok = true;
            for (int c = 0; c < n_chunks && ok; ++c) {
                const int st = c % P.nstage; const uint32_t ph = (c / P.nstage) & 1;
                ok = mbar_wait(&full[st], ph, P.spin_limit) && !*failed;
                if (!ok) break;
                fence_async_proxy();               // the gathered rows were written by cp.async (generic proxy)
                tc_fence_after();
                const uint32_t sa = smem_u32(tiles + (size_t)st * stage_bytes), sh = sa + 64 * 256;
#pragma unroll
                for (int k4 = 0; k4 < 4; ++k4)     // 16 union entries per MMA = two 8-row groups of 2048 bytes
                    umma(tmem, make_desc(sa + k4 * 4096, 1024, 2048), make_desc(sh + k4 * 32, 16, 1024), idesc,
                         (c | k4) ? 1u : 0u);
                umma_commit(&empty[st]);
            }
            if (!ok) *failed = 1;
            umma_commit(accbar);
        }
    }
    tc_fence_before();
    __syncthreads();
    const int ns = P.n_split;
    if (ns > 1) {
        // ---- K split across the cluster, summed through distributed shared memory (as in the gate/up kernel): CTA j
        // owns output columns [j * 128 / ns, (j + 1) * 128 / ns) of the tile, receives every CTA's partial values
        // of those columns in slot (rank), sums the slots in rank order, adds the residual and writes y.
        const int cols_per = 128 / ns, pitch = N + 4;               // floats per staged column: N tokens, padding
        float *stg = reinterpret_cast<float *>(smem);                // [ns][cols_per][pitch]
        cluster_sync_all();                                          // every CTA's MMAs are complete: the stages are free
        if (warp < kLoaderWarps && ok) {
            tc_fence_after();
            const int r = (warp & 3) * 32 + lane, cb = warp >> 2;
            const uint32_t dst = map_to_cta(smem_u32(stg + ((size_t)ks * cols_per + (r % cols_per)) * pitch), (uint32_t)(r / cols_per));
            for (int n0 = 16 * cb; n0 < N; n0 += 32) {
                uint32_t v[16];
                if (n_chunks > 0) tmem_ld16(tmem + ((uint32_t)((warp & 3) * 32) << 16) + (uint32_t)n0, v);
#pragma unroll
                for (int q = 0; q < 4; ++q)
                    st_cluster_v4(dst + (uint32_t)(n0 + 4 * q) * 4u, n_chunks > 0 ? v[4 * q] : 0u, n_chunks > 0 ? v[4 * q + 1] : 0u,
                                  n_chunks > 0 ? v[4 * q + 2] : 0u, n_chunks > 0 ? v[4 * q + 3] : 0u);
            }
        }
        tc_fence_before();
        cluster_sync_all();
        if (!*failed) {
            // one item = (token n, column cc of this CTA's columns): consecutive threads write consecutive columns
            for (int it = tid; it < cols_per * N; it += kGemmThreads) {
                const int n = it / cols_per, cc = it - n * cols_per, t = tok0 + n;
                if (t >= P.T) continue;
                float a = 0.f;
                for (int sp = 0; sp < ns; ++sp) a += stg[((size_t)sp * cols_per + cc) * pitch + n];
                const size_t o = (size_t)t * P.d_model + (size_t)mt * 128 + ks * cols_per + cc;
                if (P.residual) a += P.fmt ? si_cvt<SI_BF16>::lo((uint32_t)P.x[o]) : si_cvt<SI_F16>::lo((uint32_t)P.x[o]);
                if (P.y_f32) reinterpret_cast<float *>(P.y)[o] = a;
                else reinterpret_cast<uint16_t *>(P.y)[o] = P.fmt ? si_cvt<SI_BF16>::from_float(a) : si_cvt<SI_F16>::from_float(a);
            }
        }
    }
    if (warp == kLoaderWarps) {
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(ncols) : "memory");
    }
}

// y[t][j] = (x[t][j] +) sum over K splits, in split order (here only for calls that select nothing).
template <int DT>
__global__ void si_gemm_reduce_kernel(const float *__restrict__ partial, int n_split, int t_pad_total, int d, int T,
                                      const uint16_t *__restrict__ x, void *__restrict__ y, int y_f32, int residual) {
    const int j = blockIdx.x * blockDim.x + threadIdx.x, t = blockIdx.y;
    if (j >= d || t >= T) return;
    float a = 0.f;
    for (int s = 0; s < n_split; ++s) a += partial[((size_t)s * t_pad_total + t) * d + j];
    if (residual) a += si_cvt<DT>::lo((uint32_t)x[(size_t)t * d + j]);
    if (y_f32) reinterpret_cast<float *>(y)[(size_t)t * d + j] = a;
    else reinterpret_cast<uint16_t *>(y)[(size_t)t * d + j] = si_cvt<DT>::from_float(a);
}

// Any kernel as a programmatic dependent of its predecessor in the stream.
template <typename... KArgs, typename... Args>
cudaError_t launch_pdl(void (*kern)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t stream, Args... args) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid; cfg.blockDim = block; cfg.dynamicSmemBytes = smem; cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr; cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, kern, KArgs(args)...);
}

// Launch a contraction kernel as thread-block clusters of `cluster` CTAs, so that it may be scheduled while the
// previous kernel of the stream is still finishing (the kernel itself waits for that kernel's results with pdl_wait()).
template <typename... KArgs, typename... Args>
cudaError_t launch_after_predecessor(void (*kern)(KArgs...), dim3 grid, dim3 cluster, size_t smem, cudaStream_t stream, Args... args) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid; cfg.blockDim = dim3(kGemmThreads); cfg.dynamicSmemBytes = smem; cfg.stream = stream;
    cudaLaunchAttribute attr[2];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    attr[1].id = cudaLaunchAttributeClusterDimension;
    attr[1].val.clusterDim.x = cluster.x; attr[1].val.clusterDim.y = cluster.y; attr[1].val.clusterDim.z = cluster.z;
    cfg.attrs = attr; cfg.numAttrs = 2;
    return cudaLaunchKernelEx(&cfg, kern, KArgs(args)...);
}

int pick_stages_gemm(size_t stage_bytes, int n_tok) {
    // few tokens: the kernels are latency-bound gathers, two CTAs per SM hide more of it
    size_t budget = n_tok <= 16 ? 112 * 1024 : 200 * 1024;
    int n = (int)(budget / stage_bytes);
    return n > kMaxStages ? kMaxStages : n;
}

// Zero-on-entry scratch of a multi-token call, carved from the workspace's mask region:
// [T][mask_words] token slot bitmaps | [mask_words] union bitmap | counters (ticket, tile counters)
struct UnionScratch { uint32_t *tokbits, *bitmap; unsigned *ticket, *ctr; size_t zero_bytes; int mask_words; };
UnionScratch union_scratch(const si_store *s, char *wsb, const si_ws_layout &ws, int T, int n_loaded, int n_ctr, int half = 0) {
    (void)s;
    UnionScratch u;
    u.mask_words = (int)(si_align_up((size_t)n_loaded, 128) / 32);
    u.tokbits = (uint32_t *)(wsb + ws.mask_off + (size_t)half * ws.mask_half);
    u.bitmap = u.tokbits + (size_t)T * u.mask_words;
    u.ticket = (unsigned *)(u.bitmap + u.mask_words);
    u.ctr = u.ticket + 64;
    u.zero_bytes = ((size_t)(T + 1) * u.mask_words + 64 + (size_t)n_ctr) * 4;
    return u;
}
constexpr long long kUnionSmallEntries = 16 * 1024;     // up to here one block builds the union faster than several
constexpr long long kUnionOverlapEntries = 64 * 1024;   // up to here one block builds it while the call before still runs: its
                                                        // time is hidden, and the several-block kernel (whose bitmaps a memset
                                                        // must clear first, in stream order) cannot run early
constexpr size_t kUnionSmallSmem = 160 * 1024;          // shared memory the one-block union may use
int union_blocks(const si_store *s, long long entries) {
    // one entry per thread while the blocks fit the machine at once: an entry is a chain of dependent
    // global accesses (index, bitmap word, atomic), so the chains should all run side by side
    long long b = (entries + 1023) / 1024;
    if (b < 1) b = 1;
    return (int)(b > 2 * s->num_sms ? 2 * s->num_sms : b);
}

}  // namespace

size_t si_gemm_partial_bytes(const si_store *s, int T_max) {
    (void)s;
    return T_max > 1 ? kPartialCap : 0;
}

// Zero-on-entry words a call needs beyond the bitmaps.
size_t si_gemm_counter_bytes(const si_store *s, size_t nl_pad, size_t t_pad) {
    (void)s; (void)nl_pad; (void)t_pad;
    return 64 * 4;                              // the union kernel's ticket words
}

int si_union_launch(const si_store *s, int layer, int T, const int32_t *idx, const int32_t *idx_offsets,
                    int k_fixed, int32_t *union_out, int32_t *n_union_out, void *workspace, size_t ws_bytes,
                    cudaStream_t stream) {
    si_ws_layout ws = si_ws_carve(s, T, k_fixed, 1);
    if (ws_bytes < ws.total) return SI_ERR_NOMEM;
    const int n_loaded = s->n_loaded[layer];
    const int words = (n_loaded + 31) / 32;
    UnionScratch u = union_scratch(s, (char *)workspace, ws, T, n_loaded, 0);
    const long long entries = idx_offsets ? (long long)T * n_loaded : (long long)T * k_fixed;
    if (entries <= kUnionSmallEntries) {
        si_union_small_kernel<<<1, 1024, (size_t)(2 * words + 2) * 4, stream>>>(
            idx, idx_offsets, k_fixed, T, n_loaded, nullptr, 0, nullptr, u.mask_words, union_out, n_union_out, n_loaded, nullptr);
    } else {
        SI_CUDA_TRY(cudaMemsetAsync(u.bitmap, 0, ((size_t)u.mask_words + 64) * 4, stream));
        si_union_build_kernel<<<union_blocks(s, entries), 1024, (size_t)(2 * words + 2) * 4, stream>>>(
            idx, idx_offsets, k_fixed, T, n_loaded, u.bitmap, nullptr, u.mask_words, u.ticket, union_out, n_union_out,
            n_loaded, nullptr);
    }
    SI_CUDA_TRY(cudaGetLastError());
    return SI_OK;
}

// The union stage of a multi-token call: the ascending union of the lists (padded to nu_pad entries), its
// size, and -- when the tokens have lists of their own -- one slot bitmap per token; the counters the
// contractions expect to be zero are cleared on the way.  One block when the lists are short and few,
// several blocks with global atomics otherwise.
static int union_stage_launch(const si_store *s, int n_loaded, int n_lists, bool own_lists, const int32_t *idx,
                              const int32_t *idx_offsets, int k_fixed, const UnionScratch &us, int32_t *uni,
                              int32_t *n_union, int nu_pad, int32_t *status_dev, cudaStream_t stream, bool may_overlap = false) {
    const int words = (n_loaded + 31) / 32;
    // token bitmaps are only read (and so only cleared) when the tokens have lists of their own
    char *z0 = own_lists ? (char *)us.tokbits : (char *)us.bitmap;
    const size_t zero_bytes = us.zero_bytes - (size_t)(z0 - (char *)us.tokbits);
    const long long entries = idx_offsets ? (long long)n_lists * n_loaded : (long long)n_lists * k_fixed;
    const size_t small_smem = ((size_t)2 * words + 2 + (own_lists ? (size_t)n_lists * us.mask_words : 0)) * 4;
    if (entries <= (may_overlap ? kUnionOverlapEntries : kUnionSmallEntries) && small_smem <= kUnionSmallSmem) {
        // few entries, few lists: one block does everything in shared memory, the clearing of the
        // counters included
        SI_CUDA_TRY(cudaFuncSetAttribute(si_union_small_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kUnionSmallSmem));
        uint32_t *zc = (uint32_t *)us.ticket;                          // ticket words and the arrival counters
        const size_t zc_bytes = us.zero_bytes - (size_t)((char *)us.ticket - (char *)us.tokbits);
        if (may_overlap)      // as a programmatic dependent: it may start while the contraction before it still runs
            SI_CUDA_TRY(launch_pdl(si_union_small_kernel, dim3(1), dim3(1024), small_smem, stream, idx, idx_offsets, k_fixed, n_lists,
                                   n_loaded, zc, (int)(zc_bytes / 4), own_lists ? us.tokbits : (uint32_t *)nullptr, us.mask_words, uni,
                                   n_union, nu_pad, status_dev));
        else
            si_union_small_kernel<<<1, 1024, small_smem, stream>>>(
                idx, idx_offsets, k_fixed, n_lists, n_loaded, zc, (int)(zc_bytes / 4),
                own_lists ? us.tokbits : nullptr, us.mask_words, uni, n_union, nu_pad, status_dev);
    } else {
        SI_CUDA_TRY(cudaMemsetAsync(z0, 0, zero_bytes, stream));
        si_union_build_kernel<<<union_blocks(s, entries), 1024, (size_t)(2 * words + 2) * 4, stream>>>(
            idx, idx_offsets, k_fixed, n_lists, n_loaded, us.bitmap, own_lists ? us.tokbits : nullptr, us.mask_words,
            us.ticket, uni, n_union, nu_pad, status_dev);
    }
    SI_CUDA_TRY(cudaGetLastError());
    return SI_OK;
}

int si_union_masks_launch(const si_store *s, int layer, int T, const int32_t *idx, const int32_t *idx_offsets,
                          int k_fixed, int32_t *union_out, int32_t *n_union_out, uint32_t *masks_out,
                          void *workspace, size_t ws_bytes, cudaStream_t stream) {
    si_ws_layout ws = si_ws_carve(s, T < 2 ? 2 : T, k_fixed, 1);
    if (ws_bytes < ws.total) return SI_ERR_NOMEM;
    char *wsb = (char *)workspace;
    const int n_loaded = s->n_loaded[layer];
    const size_t nl_pad = si_align_up((size_t)n_loaded, 128);
    int32_t *uni = (int32_t *)(wsb + ws.union_off);
    int32_t *n_union = uni + nl_pad;
    long long cap = idx_offsets ? (long long)n_loaded : (long long)T * k_fixed;
    if (cap > n_loaded) cap = n_loaded;
    const int nu_pad = (int)si_align_up((size_t)cap, 128);
    UnionScratch us = union_scratch(s, wsb, ws, T, n_loaded, 0);
    if (us.zero_bytes > ws.mask_half) return SI_ERR_NOMEM;
    int rc = union_stage_launch(s, n_loaded, T, true, idx, idx_offsets, k_fixed, us, uni, n_union, nu_pad, nullptr, stream);
    if (rc) return rc;
    SI_CUDA_TRY(cudaMemcpyAsync(union_out, uni, (size_t)n_loaded * 4, cudaMemcpyDeviceToDevice, stream));
    SI_CUDA_TRY(cudaMemcpyAsync(n_union_out, n_union, 4, cudaMemcpyDeviceToDevice, stream));
    SI_CUDA_TRY(cudaMemcpyAsync(masks_out, us.tokbits, (size_t)T * us.mask_words * 4, cudaMemcpyDeviceToDevice, stream));
    return SI_OK;
}

int si_multi_token_launch(const si_store *s, int layer, const void *x, int T, const int32_t *idx,
                          const int32_t *idx_offsets, int k_fixed, void *y, int y_dtype, unsigned flags,
                          void *workspace, size_t ws_bytes, int32_t *status_dev, cudaStream_t stream,
                          long long spin_limit, int withhold) {
    const int d = s->d_model;
    if (d % 128 != 0) return SI_ERR_UNSUPPORTED;
    si_ws_layout ws = si_ws_carve(s, T < 2 ? 2 : T, k_fixed, 1);       // the multi-token regions exist from T_max = 2 on
    if (ws_bytes < ws.total) return SI_ERR_NOMEM;
    char *wsb = (char *)workspace;
    const int n_loaded = s->n_loaded[layer];
    const bool shared = (flags & SI_FLAG_SHARED_LIST) != 0;
    if (n_loaded == 0 || k_fixed == 0) {
        // nothing selected: y = 0 (or x)
        const int threads = 256;
        dim3 grid((d + threads - 1) / threads, T);
        if (s->dtype == SI_BF16)
            si_gemm_reduce_kernel<SI_BF16><<<grid, threads, 0, stream>>>(nullptr, 0, 0, d, T, (const uint16_t *)x, y, y_dtype == SI_F32, (flags & SI_FLAG_RESIDUAL) != 0);
        else
            si_gemm_reduce_kernel<SI_F16><<<grid, threads, 0, stream>>>(nullptr, 0, 0, d, T, (const uint16_t *)x, y, y_dtype == SI_F32, (flags & SI_FLAG_RESIDUAL) != 0);
        SI_CUDA_TRY(cudaGetLastError());
        return SI_OK;
    }
    // ---- union (this call's copy of the union stage's outputs: the other copy may still be read by the call before)
    const int half = (int)(s->mt_calls.fetch_add(1u, std::memory_order_relaxed) & 1u);
    const size_t nl_pad = si_align_up((size_t)n_loaded, 128);
    int32_t *uni = (int32_t *)(wsb + ws.union_off + (size_t)half * ws.union_half);
    int32_t *n_union = uni + nl_pad;                       // one int32 (64 reserved)
    // host-known upper bound of the union size sizes the grids
    long long cap = shared ? (long long)k_fixed : (idx_offsets ? (long long)n_loaded : (long long)T * k_fixed);
    if (cap > n_loaded) cap = n_loaded;
    const int nu_pad = (int)si_align_up((size_t)cap, 128);
    const int t_pad_total = (int)si_align_up((size_t)T, 16);
    const int m_tiles = nu_pad / 128;
    const bool own_lists = !shared && !(flags & SI_FLAG_UNION_UNMASKED);   // membership differs per token
    UnionScratch us = union_scratch(s, wsb, ws, T, n_loaded, 0, half);
    if (us.zero_bytes > ws.mask_half) return SI_ERR_NOMEM;
    {
        int rc = union_stage_launch(s, n_loaded, shared ? 1 : T, own_lists, idx, idx_offsets, k_fixed, us, uni, n_union,
                                    nu_pad, status_dev, stream, true);
        if (rc) return rc;
    }
    // ---- tiling (calls with more than 128 tokens leave for the CTA-pair kernels below: one token tile here)
    const int n_tok = t_pad_total, t_pad_alloc = t_pad_total;
    GemmParams P;
    P.rec_base = (const char *)s->records(layer); P.rec_bytes = (int)s->record_bytes(); P.d_model = d; P.chunks = d / 8;
    P.union_slots = uni; P.n_union = n_union; P.nu_pad = nu_pad;
    P.x = (const uint16_t *)x; P.T = T; P.n_tok = n_tok;
    P.h = (const uint16_t *)(wsb + ws.h_off); P.t_pad_total = t_pad_alloc;
    P.fmt = s->dtype == SI_BF16 ? 1 : 0;
    P.status = status_dev;
    P.tokbits = own_lists ? us.tokbits : nullptr; P.mask_words = us.mask_words;
    P.h_out = (uint16_t *)(wsb + ws.h_off);
    P.y = y; P.y_f32 = y_dtype == SI_F32; P.residual = (flags & SI_FLAG_RESIDUAL) != 0;
    P.spin_limit = spin_limit > 0 ? spin_limit : kSpinLimit; P.withhold = withhold;
    P.pair_n = 0;
    if (si_pair_path_applies(s, T))
        return si_pair_contractions_launch(s, P, n_loaded, wsb + ws.h_off, ws.h_bytes, stream);
    // (here T <= 128: one token tile.)  Both contractions split K among the CTAs of a thread-block cluster (1, 2, 4 or
    // 8 CTAs per tile), which sum their partial accumulators through distributed shared memory.  The cluster sizes
    // aim at one wave of CTAs over the SM slots (two CTAs per SM with few tokens: the gathers are latency-bound).
    const int target = (t_pad_alloc <= 16 ? 2 : 1) * s->num_sms;
    const int k_chunks = d / kChunkK;
    if ((size_t)t_pad_alloc * nu_pad * 2 > ws.h_bytes) return SI_ERR_NOMEM;
    {
        // gate/up: the grid is sized for the largest possible union, whose tiles past the real union leave at once
        int s1 = 1;
        while (s1 < 8 && s1 * 2 <= k_chunks && m_tiles * s1 * 2 <= target) s1 *= 2;
        const size_t stage = 2 * 128 * 128 + (size_t)n_tok * 128;
        P.nstage = pick_stages_gemm(stage, n_tok); P.n_split = s1;
        if (P.nstage < 2) return SI_ERR_UNSUPPORTED;
        if (s1 > 1 && (size_t)128 * (2 * n_tok + 4) * 4 > (size_t)P.nstage * stage) return SI_ERR_UNSUPPORTED;   // staging area of the cluster sum
        size_t smem = (size_t)P.nstage * stage + 256;
        SI_CUDA_TRY(cudaFuncSetAttribute(si_gemm_gateup_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
        CUtensorMap x_map, rec_map;
        int rc = make_tile_map(&x_map, x, (size_t)d, (size_t)T, (size_t)d * 2, n_tok);
        if (rc) return rc;
        // the layer's records as a matrix [n_loaded][3 * d_model]: 128 consecutive slots x 64 columns per tile
        rc = make_tile_map(&rec_map, P.rec_base, (size_t)3 * d, (size_t)n_loaded, (size_t)P.rec_bytes, 128);
        if (rc) return rc;
        SI_CUDA_TRY(launch_after_predecessor(si_gemm_gateup_kernel, dim3(m_tiles * s1), dim3(s1), smem, stream, P, x_map, rec_map));
    }
    {
        // down: K = the union
        int s2 = 1;
        while (s2 < 8 && s2 * 2 <= nu_pad / kChunkK && (d / 128) * s2 * 2 <= target) s2 *= 2;
        const size_t stage = 64 * 256 + (size_t)n_tok * 128;
        P.nstage = pick_stages_gemm(stage, n_tok); P.n_split = s2;
        if (P.nstage < 2) return SI_ERR_UNSUPPORTED;
        if (s2 > 1 && (size_t)128 * (n_tok + 4) * 4 > (size_t)P.nstage * stage) return SI_ERR_UNSUPPORTED;
        size_t smem = (size_t)P.nstage * stage + 256;
        SI_CUDA_TRY(cudaFuncSetAttribute(si_gemm_down_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
        CUtensorMap h_map;
        int rc = make_tile_map(&h_map, wsb + ws.h_off, (size_t)nu_pad, (size_t)t_pad_alloc, (size_t)nu_pad * 2, n_tok);
        if (rc) return rc;
        SI_CUDA_TRY(launch_after_predecessor(si_gemm_down_kernel, dim3(d / 128, s2, 1), dim3(1, s2, 1), smem, stream, P, h_map));
    }
    SI_CUDA_TRY(cudaGetLastError());
    return SI_OK;
}
