// Multi-token path (T > 1: batched decode and prefill): the union of the tokens' active lists
// is formed once, and the selective FFN over the union runs as two gathered dense contractions
// on the 5th-generation tensor cores (tcgen05.mma, accumulators in tensor memory):
//
//   union      U = sorted union of the T lists, mask[t] = which entries of U token t selected
//   gate/up    G^T, Up^T [|U| x T] = W_gate[U, :] . X^T, W_up[U, :] . X^T     (K = d_model)
//   combine    H[t, i] = mask[t, i] ? SiLU(G[i, t]) * Up[i, t] : 0, rounded to the store dtype
//   down       Y^T [d_model x T] = W_down[:, U] . H^T                          (K = |U|)
//
// Token t therefore uses exactly its own list (Section 5 applied per token), whatever the
// other tokens selected; with SI_FLAG_UNION_UNMASKED every token uses the whole union.
//
// Tiling.  Both contractions put the weight side on the MMA M dimension (128 rows of the
// store per CTA tile) and the tokens on N (T padded to 16, at most 256 per tile), so the
// weights -- the dominant bytes -- are read exactly once.  Weight rows are gathered straight
// out of the neuron records with 16-byte cp.async copies into the 128-byte-swizzled shared
// memory layouts the MMA descriptors expect (gate/up rows are K-major, down rows MN-major).
// K is split across CTAs so that small unions still fill the machine; the fp32 partial tiles
// are summed in split order by the combine / reduce kernels, so results are deterministic.
#include "si_common.cuh"

namespace {

constexpr int kLoaderThreads = 128;              // warps 0..3: gather loads, later the epilogue
constexpr int kGemmThreads = kLoaderThreads + 32; // warp 4: MMA issue + tensor-memory allocation
constexpr int kMaxStages = 6;
constexpr int kChunkK = 64;                      // K elements per pipeline stage (128 bytes per row)
constexpr long long kSpinLimit = 1ll << 24;      // bounded waits (mbarrier probes)
constexpr size_t kPartialCap = (size_t)64 << 20; // bytes of fp32 partial tiles per contraction

__device__ __forceinline__ uint32_t smem_u32(const void *p) { return (uint32_t)__cvta_generic_to_shared(p); }
__device__ __forceinline__ void mbar_init(uint64_t *bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint64_t *bar) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(bar)) : "memory");
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
// Bounded wait: false after kSpinLimit unsuccessful probes.
__device__ __forceinline__ bool mbar_wait(uint64_t *bar, uint32_t parity) {
    for (long long i = 0; i < kSpinLimit; ++i)
        if (mbar_try_wait(bar, parity)) return true;
    return false;
}
__device__ __forceinline__ void cp_async16(void *dst_smem, const void *src) {
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(smem_u32(dst_smem)), "l"(src) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N>
__device__ __forceinline__ void cp_async_wait() { asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory"); }
// wait until at most n of this thread's committed copy groups are still in flight (n <= 5)
__device__ __forceinline__ void cp_async_wait_dyn(int n) {
    switch (n) {
        case 0: cp_async_wait<0>(); break;
        case 1: cp_async_wait<1>(); break;
        case 2: cp_async_wait<2>(); break;
        case 3: cp_async_wait<3>(); break;
        case 4: cp_async_wait<4>(); break;
        default: cp_async_wait<5>(); break;
    }
}
__device__ __forceinline__ void fence_async_proxy() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }

// Shared-memory matrix descriptor (sm_100 format): start address, leading / stride byte
// offsets in 16-byte units, descriptor version 1, 128-byte swizzle.
__device__ __forceinline__ uint64_t make_desc(uint32_t smem_addr, uint32_t lbo_bytes, uint32_t sbo_bytes) {
    uint32_t lo = ((smem_addr >> 4) & 0x3FFFu) | (((lbo_bytes >> 4) & 0x3FFFu) << 16);
    uint32_t hi = ((sbo_bytes >> 4) & 0x3FFFu) | (1u << 14) | (2u << 29);
    return ((uint64_t)hi << 32) | lo;
}
// Instruction descriptor for kind::f16: fp32 accumulate, A/B format (0 f16, 1 bf16), majors.
__device__ __forceinline__ uint32_t make_idesc(int fmt, int a_mn_major, int b_mn_major, int M, int N) {
    return (1u << 4) | ((uint32_t)fmt << 7) | ((uint32_t)fmt << 10) | ((uint32_t)a_mn_major << 15) |
           ((uint32_t)b_mn_major << 16) | ((uint32_t)(N >> 3) << 17) | ((uint32_t)(M >> 4) << 24);
}
__device__ __forceinline__ void umma(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc, uint32_t accumulate) {
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, {%5, %5, %5, %5}, p;\n\t}"
        ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate), "r"(0u) : "memory");
}
__device__ __forceinline__ void umma_commit(uint64_t *bar) {
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(smem_u32(bar)) : "memory");
}
__device__ __forceinline__ void tmem_ld16(uint32_t taddr, uint32_t (&r)[16]) {
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15}, [%16];"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
          "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15])
        : "r"(taddr));
    asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
}

// ------------------------------------------------------------------------------- union
// Step 1 (many CTAs): OR every list entry into a bitmap over the loaded slots (zero on entry).
__global__ void si_union_bitmap_kernel(const int32_t *__restrict__ idx, const int32_t *__restrict__ offsets, int k_fixed,
                                       int n_lists, int n_loaded, uint32_t *__restrict__ bitmap, int32_t *status) {
    const long long total = offsets ? offsets[n_lists] : (long long)n_lists * k_fixed;
    for (long long e = (long long)blockIdx.x * blockDim.x + threadIdx.x; e < total; e += (long long)gridDim.x * blockDim.x) {
        const int s = idx[e];
        if (s < 0 || s >= n_loaded) { if (status) atomicCAS(status, 0, SI_ERR_OUT_OF_RANGE); continue; }
        const uint32_t bit = 1u << (s & 31);
        if (!(bitmap[s >> 5] & bit)) atomicOr(&bitmap[s >> 5], bit);     // hot slots are set by the first token
    }
}

// Step 2 (one CTA): popcount prefix scan over the bitmap -> sorted union, slot -> position map.
__global__ void __launch_bounds__(1024)
si_union_kernel(const uint32_t *__restrict__ bitmap_g, int n_loaded, int32_t *__restrict__ union_out,
                int32_t *__restrict__ n_union_out, int32_t *__restrict__ pos_of_slot, int union_cap) {
    extern __shared__ uint32_t sh[];
    uint32_t *bitmap = sh;                         // [words]
    uint32_t *wprefix = sh + (n_loaded + 31) / 32; // [words] exclusive popcount prefix
    __shared__ uint32_t warp_tot[32];
    const int words = (n_loaded + 31) / 32;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    for (int w = tid; w < words; w += 1024) bitmap[w] = bitmap_g[w];
    __syncthreads();
    // exclusive prefix of popcounts over the bitmap words (words <= 2048 for d_ff <= 65536)
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
            if (lane == 31) warp_tot[31] = vi - v, sh[2 * words] = vi;   // total of this block of words
        }
        __syncthreads();
        if (w < words) wprefix[w] = carry + warp_tot[warp] + inc - c;
        carry += sh[2 * words];
        __syncthreads();
    }
    const int n_u = (int)carry;
    if (tid == 0) *n_union_out = n_u;
    // emit the union (ascending) and the slot -> position map
    for (int w = tid; w < words; w += 1024) {
        uint32_t bits = bitmap[w]; int p = (int)wprefix[w];
        while (bits) {
            int bpos = __ffs(bits) - 1; bits &= bits - 1;
            int s = w * 32 + bpos;
            if (p < union_cap) union_out[p] = s;
            pos_of_slot[s] = p;
            ++p;
        }
    }
    // pad the union up to the capacity with its first entry (masked out everywhere)
    __syncthreads();
    {
        int first = 0;
        for (int w = 0; w < words; ++w) if (bitmap[w]) { first = w * 32 + __ffs(bitmap[w]) - 1; break; }
        for (int p = n_u + tid; p < union_cap; p += 1024) union_out[p] = first;
    }
}

// Membership masks over union positions, many CTAs: mask[t] bit p set iff U[p] is in list t.
// The masks are zero on entry (memset by the host side of the call).
__global__ void si_union_masks_kernel(const int32_t *__restrict__ idx, const int32_t *__restrict__ offsets, int k_fixed,
                                      int T, int shared_list, int n_loaded, const int32_t *__restrict__ n_union,
                                      const int32_t *__restrict__ pos_of_slot, uint32_t *__restrict__ masks,
                                      int mask_words, int unmasked) {
    const long long gid = (long long)blockIdx.x * blockDim.x + threadIdx.x, gstride = (long long)gridDim.x * blockDim.x;
    if (unmasked || shared_list) {
        // every token uses the whole union (with one shared list the union is that list)
        const int n_u = *n_union;
        for (long long i = gid; i < (long long)T * mask_words; i += gstride) {
            const int lo = (int)(i % mask_words) * 32;
            masks[i] = lo + 32 <= n_u ? 0xFFFFFFFFu : (lo < n_u ? ((1u << (n_u - lo)) - 1u) : 0u);
        }
        return;
    }
    const long long total = offsets ? offsets[T] : (long long)T * k_fixed;
    for (long long e = gid; e < total; e += gstride) {
        int t;
        if (offsets) {            // largest t with offsets[t] <= e
            int lo = 0, hi = T;
            while (hi - lo > 1) { int mid = (lo + hi) >> 1; if (offsets[mid] <= e) lo = mid; else hi = mid; }
            t = lo;
        } else {
            t = (int)(e / k_fixed);
        }
        const int s = idx[e];
        if (s < 0 || s >= n_loaded) continue;
        const int p = pos_of_slot[s];
        atomicOr(&masks[(size_t)t * mask_words + (p >> 5)], 1u << (p & 31));
    }
}

// ------------------------------------------------------------------------------- contractions
struct GemmParams {
    const char *rec_base;          // records of the layer
    int rec_bytes, d_model, chunks;
    const int32_t *union_slots;    // padded union (device)
    const int32_t *n_union;        // device
    int nu_pad;                    // padded union size the grids were sized for
    const uint16_t *x;             // [T, d_model]
    int T, n_tok;                  // tokens, N of the MMA (multiple of 16, <= 256)
    const uint16_t *h;             // [t_pad_total][nu_pad] (down)
    int t_pad_total;
    float *partial;                // gate/up: [S][2][nu_pad][t_pad_total]; down: [S][t_pad_total][d_model]
    int n_split;                   // K splits
    int fmt;                       // 0 f16, 1 bf16
    int nstage;
    int32_t *status;
};

// Gate/up contraction.  grid = (union tiles of 128, K splits of d_model, token tiles).
// D_gate[128 neurons x N tokens] (+)= Wg[U tile, k] . X[tokens, k]^T, same for up, accumulated in
// tensor memory (columns [0,N) gate, [N,2N) up).
__global__ void __launch_bounds__(kGemmThreads, 2)
si_gemm_gateup_kernel(const __grid_constant__ GemmParams P) {
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
    const int mt = blockIdx.x, ks = blockIdx.y, tt = blockIdx.z;
    const int n_u = *P.n_union;
    if (mt * 128 >= n_u && mt > 0) return;                          // nothing of the union in this tile
    const int k_per = (P.d_model / kChunkK + P.n_split - 1) / P.n_split;   // chunks per split
    const int c0 = ks * k_per, c1 = min(P.d_model / kChunkK, c0 + k_per);
    const int n_chunks = c1 > c0 ? c1 - c0 : 0;
    const int tok0 = tt * 256;

    uint32_t ncols = 32; while (ncols < (uint32_t)(2 * N)) ncols <<= 1;
    if (tid == 0) {
        for (int s = 0; s < P.nstage; ++s) { mbar_init(&full[s], kLoaderThreads); mbar_init(&empty[s], 1); }
        mbar_init(accbar, 1);
        *failed = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 4) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_slot)), "r"(ncols) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = *tmem_slot;

    if (warp < 4) {
        // ---------------------------------------------------------------- gather loads
        // Copy j of a thread covers 16-byte piece (tid & 7) of tile row 16*j + (tid >> 3): the 32 lanes
        // of a warp instruction read four whole 128-byte row segments, so the gather is coalesced.
        const int q8 = tid & 7;
        const char *grow[8];                                         // gate rows; the up row follows at d_model*2
#pragma unroll
        for (int j = 0; j < 8; ++j)
            grow[j] = P.rec_base + (size_t)P.union_slots[mt * 128 + 16 * j + (tid >> 3)] * P.rec_bytes + q8 * 16;
        const int r = tid;                                           // epilogue: this thread's tile row
        int pending = 0;                                             // committed groups not yet signalled
        const int la = P.nstage - 1 < 5 ? P.nstage - 1 : 5;         // chunks of copies kept in flight
        for (int c = 0; c < n_chunks; ++c) {
            const int st = c % P.nstage; const uint32_t ph = (c / P.nstage) & 1;
            if (!mbar_wait(&empty[st], ph ^ 1)) { *failed = 1; break; }
            uint8_t *sg = tiles + (size_t)st * stage_bytes, *su = sg + 128 * 128, *sx = su + 128 * 128;
#pragma unroll
            for (int j = 0; j < 8; ++j) {
                const int row = 16 * j + (tid >> 3);
                const char *gsrc = grow[j] + (size_t)(c0 + c) * 128;
                const int off = row * 128 + ((q8 ^ (row & 7)) << 4);
                cp_async16(sg + off, gsrc);
                cp_async16(su + off, gsrc + (size_t)P.d_model * 2);
            }
            for (int e = tid; e < N * 8; e += kLoaderThreads) {
                const int n = e >> 3, q = e & 7;
                const int tok = tok0 + n;
                if (tok < P.T)
                    cp_async16(sx + n * 128 + ((q ^ (n & 7)) << 4),
                               reinterpret_cast<const char *>(P.x) + ((size_t)tok * P.d_model + (size_t)(c0 + c) * kChunkK) * 2 + q * 16);
                else
                    *reinterpret_cast<uint4 *>(sx + n * 128 + ((q ^ (n & 7)) << 4)) = make_uint4(0, 0, 0, 0);
            }
            cp_async_commit();
            ++pending;
            if (pending == la + 1) {     // keep `la` chunks of copies in flight per thread
                cp_async_wait_dyn(la);
                fence_async_proxy();
                mbar_arrive(&full[(c - la) % P.nstage]);
                --pending;
            }
        }
        // drain
        if (!*failed) {
            const int done = n_chunks;
            for (; pending > 0; --pending) {
                cp_async_wait_dyn(pending - 1);
                fence_async_proxy();
                mbar_arrive(&full[(done - pending) % P.nstage]);
            }
        } else {
            cp_async_wait<0>();
        }
        // ---------------------------------------------------------------- epilogue
        bool ok = !*failed && mbar_wait(accbar, 0);
        tc_fence_after();
        if (ok && n_chunks > 0) {
            // thread r holds union row mt*128 + r: N gate values then N up values
            float *pg = P.partial + (((size_t)ks * 2 + 0) * P.nu_pad + (size_t)mt * 128 + r) * P.t_pad_total + tok0;
            float *pu = P.partial + (((size_t)ks * 2 + 1) * P.nu_pad + (size_t)mt * 128 + r) * P.t_pad_total + tok0;
            for (int n0 = 0; n0 < N; n0 += 16) {
                uint32_t v[16];
                tmem_ld16(tmem + ((uint32_t)(warp * 32) << 16) + (uint32_t)n0, v);
#pragma unroll
                for (int q = 0; q < 4; ++q)
                    *reinterpret_cast<uint4 *>(pg + n0 + 4 * q) = make_uint4(v[4 * q], v[4 * q + 1], v[4 * q + 2], v[4 * q + 3]);
                tmem_ld16(tmem + ((uint32_t)(warp * 32) << 16) + (uint32_t)(N + n0), v);
#pragma unroll
                for (int q = 0; q < 4; ++q)
                    *reinterpret_cast<uint4 *>(pu + n0 + 4 * q) = make_uint4(v[4 * q], v[4 * q + 1], v[4 * q + 2], v[4 * q + 3]);
            }
        } else if (ok) {
            float *pg = P.partial + (((size_t)ks * 2 + 0) * P.nu_pad + (size_t)mt * 128 + r) * P.t_pad_total + tok0;
            float *pu = P.partial + (((size_t)ks * 2 + 1) * P.nu_pad + (size_t)mt * 128 + r) * P.t_pad_total + tok0;
            for (int n = 0; n < N; ++n) { pg[n] = 0.f; pu[n] = 0.f; }
        }
        if (!ok && tid == 0 && P.status) atomicCAS(P.status, 0, SI_ERR_TIMEOUT);
    } else {
        // ---------------------------------------------------------------- MMA issue (one thread)
        if (lane == 0) {
            const uint32_t idesc = make_idesc(P.fmt, 0, 0, 128, N);
            bool ok = true;
            for (int c = 0; c < n_chunks && ok; ++c) {
                const int st = c % P.nstage; const uint32_t ph = (c / P.nstage) & 1;
                ok = mbar_wait(&full[st], ph) && !*failed;
                if (!ok) break;
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
    if (warp == 4) {
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(ncols) : "memory");
    }
}

// H[t][i] = mask ? SiLU(sum_s G) * (sum_s U) : 0, rounded to the store dtype.  grid over (t, i).
template <int DT>
__global__ void si_gemm_combine_kernel(const float *__restrict__ partial, int n_split, int nu_pad, int t_pad_total,
                                       int T, const int32_t *__restrict__ n_union, const uint32_t *__restrict__ masks,
                                       int mask_words, uint16_t *__restrict__ h) {
    // threads run over tokens fastest (the partial tiles are [position][token]); H is [token][position]
    const int t = blockIdx.x * 32 + (threadIdx.x & 31);
    const int i = blockIdx.y * 8 + (threadIdx.x >> 5);
    if (i >= nu_pad || t >= t_pad_total) return;
    float out = 0.f;
    if (t < T && i < *n_union && ((masks[(size_t)t * mask_words + (i >> 5)] >> (i & 31)) & 1u)) {
        float g = 0.f, u = 0.f;
        for (int s = 0; s < n_split; ++s) {
            g += partial[(((size_t)s * 2 + 0) * nu_pad + i) * t_pad_total + t];
            u += partial[(((size_t)s * 2 + 1) * nu_pad + i) * t_pad_total + t];
        }
        out = si_silu_mul(g, u);
    }
    h[(size_t)t * nu_pad + i] = si_cvt<DT>::from_float(out);
}

// Down contraction.  grid = (d_model / 128 column tiles, K splits over the union, token tiles).
// D[128 output columns x N tokens] (+)= Wd[U_k, columns]^T . H[tokens, U_k]^T: A is MN-major (a
// down row is contiguous along the output columns), B is K-major.
__global__ void __launch_bounds__(kGemmThreads, 2)
si_gemm_down_kernel(const __grid_constant__ GemmParams P) {
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
    const int mt = blockIdx.x, ks = blockIdx.y, tt = blockIdx.z;
    const int n_u = *P.n_union;
    const int total_chunks = (n_u + kChunkK - 1) / kChunkK;        // 64 union entries per chunk
    const int k_per = (total_chunks + P.n_split - 1) / P.n_split;
    const int c0 = ks * k_per, c1 = min(total_chunks, c0 + k_per);
    const int n_chunks = c1 > c0 ? c1 - c0 : 0;
    const int tok0 = tt * 256;

    uint32_t ncols = 32; while (ncols < (uint32_t)N) ncols <<= 1;
    if (tid == 0) {
        for (int s = 0; s < P.nstage; ++s) { mbar_init(&full[s], kLoaderThreads); mbar_init(&empty[s], 1); }
        mbar_init(accbar, 1);
        *failed = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 4) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_slot)), "r"(ncols) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = *tmem_slot;

    if (warp < 4) {
        // Copy j of a thread covers 16-byte piece (tid & 15) of the 256-byte down-row segment of union
        // entry 8*j + (tid >> 4) of the chunk: a warp instruction reads two whole segments (coalesced).
        const int c16 = tid & 15;
        int pending = 0;
        const int la = P.nstage - 1 < 5 ? P.nstage - 1 : 5;
        int slots_next[8];                                           // union slots of the next chunk (prefetched)
#pragma unroll
        for (int j = 0; j < 8; ++j)
            slots_next[j] = n_chunks > 0 ? P.union_slots[c0 * kChunkK + 8 * j + (tid >> 4)] : 0;
        for (int c = 0; c < n_chunks; ++c) {
            const int st = c % P.nstage; const uint32_t ph = (c / P.nstage) & 1;
            int slots[8];
#pragma unroll
            for (int j = 0; j < 8; ++j) {
                slots[j] = slots_next[j];
                if (c + 1 < n_chunks) slots_next[j] = P.union_slots[(c0 + c + 1) * kChunkK + 8 * j + (tid >> 4)];
            }
            if (!mbar_wait(&empty[st], ph ^ 1)) { *failed = 1; break; }
            uint8_t *sa = tiles + (size_t)st * stage_bytes, *sh = sa + 64 * 256;
#pragma unroll
            for (int j = 0; j < 8; ++j) {
                const int kk = 8 * j + (tid >> 4);                              // union entry of the chunk
                const int slot = slots[j];                                      // padded entries carry a valid slot
                const char *src = P.rec_base + (size_t)slot * P.rec_bytes + (size_t)P.d_model * 4 +
                                  (size_t)mt * 256 + c16 * 16;
                const int half = c16 >> 3, q = c16 & 7, k8 = kk & 7;
                cp_async16(sa + (kk >> 3) * 2048 + half * 1024 + k8 * 128 + ((q ^ k8) << 4), src);
            }
            for (int e = tid; e < N * 8; e += kLoaderThreads) {
                const int n = e >> 3, q = e & 7;
                cp_async16(sh + n * 128 + ((q ^ (n & 7)) << 4),
                           reinterpret_cast<const char *>(P.h) + ((size_t)(tok0 + n) * P.nu_pad + (size_t)(c0 + c) * kChunkK) * 2 + q * 16);
            }
            cp_async_commit();
            ++pending;
            if (pending == la + 1) {
                cp_async_wait_dyn(la);
                fence_async_proxy();
                mbar_arrive(&full[(c - la) % P.nstage]);
                --pending;
            }
        }
        if (!*failed) {
            const int done = n_chunks;
            for (; pending > 0; --pending) {
                cp_async_wait_dyn(pending - 1);
                fence_async_proxy();
                mbar_arrive(&full[(done - pending) % P.nstage]);
            }
        } else {
            cp_async_wait<0>();
        }
        bool ok = !*failed && mbar_wait(accbar, 0);
        tc_fence_after();
        // thread holds output column mt*128 + tid for N tokens
        float *py = P.partial + ((size_t)ks * P.t_pad_total + tok0) * P.d_model + (size_t)mt * 128 + tid;
        if (ok && n_chunks > 0) {
            for (int n0 = 0; n0 < N; n0 += 16) {
                uint32_t v[16];
                tmem_ld16(tmem + ((uint32_t)(warp * 32) << 16) + (uint32_t)n0, v);
#pragma unroll
                for (int q = 0; q < 16; ++q) py[(size_t)(n0 + q) * P.d_model] = __uint_as_float(v[q]);
            }
        } else if (ok) {
            for (int n = 0; n < N; ++n) py[(size_t)n * P.d_model] = 0.f;
        }
        if (!ok && tid == 0 && P.status) atomicCAS(P.status, 0, SI_ERR_TIMEOUT);
    } else {
        if (lane == 0) {
            const uint32_t idesc = make_idesc(P.fmt, 1, 0, 128, N);
            bool ok = true;
            for (int c = 0; c < n_chunks && ok; ++c) {
                const int st = c % P.nstage; const uint32_t ph = (c / P.nstage) & 1;
                ok = mbar_wait(&full[st], ph) && !*failed;
                if (!ok) break;
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
    if (warp == 4) {
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(ncols) : "memory");
    }
}

// y[t][j] = (x[t][j] +) sum over K splits, in split order.
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

int pick_stages_gemm(size_t stage_bytes, int n_tok) {
    // few tokens: the kernels are latency-bound gathers, two CTAs per SM hide more of it
    size_t budget = n_tok <= 64 ? 112 * 1024 : 200 * 1024;
    int n = (int)(budget / stage_bytes);
    return n > kMaxStages ? kMaxStages : n;
}

}  // namespace

size_t si_gemm_partial_bytes(const si_store *s, int T_max) {
    (void)s;
    return T_max > 1 ? kPartialCap : 0;
}

int si_union_launch(const si_store *s, int layer, int T, const int32_t *idx, const int32_t *idx_offsets,
                    int k_fixed, int32_t *union_out, int32_t *n_union_out, void *workspace, size_t ws_bytes,
                    cudaStream_t stream) {
    si_ws_layout ws = si_ws_carve(s, T, k_fixed, 1);
    if (ws_bytes < ws.total) return SI_ERR_NOMEM;
    char *wsb = (char *)workspace;
    const int n_loaded = s->n_loaded[layer];
    const int words = (n_loaded + 31) / 32;
    int32_t *pos = (int32_t *)(wsb + ws.union_off) + si_align_up((size_t)n_loaded, 128) + 64;
    uint32_t *masks = (uint32_t *)(wsb + ws.mask_off);
    const int mask_words = (int)(si_align_up((size_t)n_loaded, 128) / 32);
    size_t smem = (size_t)(2 * words + 2) * 4;
    uint32_t *bitmap = masks + (size_t)T * mask_words;
    SI_CUDA_TRY(cudaMemsetAsync(masks, 0, ((size_t)T * mask_words + words) * 4, stream));
    si_union_bitmap_kernel<<<64, 256, 0, stream>>>(idx, idx_offsets, k_fixed, T, n_loaded, bitmap, nullptr);
    si_union_kernel<<<1, 1024, smem, stream>>>(bitmap, n_loaded, union_out, n_union_out, pos, n_loaded);
    si_union_masks_kernel<<<64, 256, 0, stream>>>(idx, idx_offsets, k_fixed, T, 0, n_loaded, n_union_out, pos, masks,
                                                  mask_words, 0);
    SI_CUDA_TRY(cudaGetLastError());
    return SI_OK;
}

int si_multi_token_launch(const si_store *s, int layer, const void *x, int T, const int32_t *idx,
                          const int32_t *idx_offsets, int k_fixed, void *y, int y_dtype, unsigned flags,
                          void *workspace, size_t ws_bytes, int32_t *status_dev, cudaStream_t stream) {
    const int d = s->d_model;
    if (d % 128 != 0) return SI_ERR_UNSUPPORTED;
    si_ws_layout ws = si_ws_carve(s, T, k_fixed, 1);
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
    // ---- union
    const size_t nl_pad = si_align_up((size_t)n_loaded, 128);
    int32_t *uni = (int32_t *)(wsb + ws.union_off);
    int32_t *n_union = uni + nl_pad;                       // one int32 (64 reserved)
    int32_t *pos = uni + nl_pad + 64;
    uint32_t *masks = (uint32_t *)(wsb + ws.mask_off);
    const int mask_words = (int)(nl_pad / 32);
    // host-known upper bound of the union size sizes the grids
    long long cap = shared ? (long long)k_fixed : (idx_offsets ? (long long)n_loaded : (long long)T * k_fixed);
    if (cap > n_loaded) cap = n_loaded;
    const int nu_pad = (int)si_align_up((size_t)cap, 128);
    {
        const int words = (n_loaded + 31) / 32;
        size_t smem = (size_t)(2 * words + 2) * 4;
        uint32_t *bitmap = masks + (size_t)T * mask_words;
        SI_CUDA_TRY(cudaMemsetAsync(masks, 0, ((size_t)T * mask_words + words) * 4, stream));
        si_union_bitmap_kernel<<<s->num_sms, 256, 0, stream>>>(idx, idx_offsets, k_fixed, shared ? 1 : T, n_loaded, bitmap,
                                                               status_dev);
        si_union_kernel<<<1, 1024, smem, stream>>>(bitmap, n_loaded, uni, n_union, pos, nu_pad);
        si_union_masks_kernel<<<2 * s->num_sms, 256, 0, stream>>>(idx, idx_offsets, k_fixed, T, shared ? 1 : 0, n_loaded,
                                                                   n_union, pos, masks, mask_words,
                                                                   (flags & SI_FLAG_UNION_UNMASKED) != 0);
    }
    // ---- tiling
    const int t_pad_total = (int)si_align_up((size_t)T, 16);
    const int tok_tiles = (t_pad_total + 255) / 256;
    const int n_tok = tok_tiles > 1 ? 256 : t_pad_total;
    // with several token tiles every tile must be full width: pad the token dimension
    const int t_pad_alloc = tok_tiles * n_tok;
    const int m_tiles = nu_pad / 128;
    GemmParams P;
    P.rec_base = (const char *)s->records(layer); P.rec_bytes = (int)s->record_bytes(); P.d_model = d; P.chunks = d / 8;
    P.union_slots = uni; P.n_union = n_union; P.nu_pad = nu_pad;
    P.x = (const uint16_t *)x; P.T = T; P.n_tok = n_tok;
    P.h = (const uint16_t *)(wsb + ws.h_off); P.t_pad_total = t_pad_alloc;
    P.partial = (float *)(wsb + ws.partial_off);
    P.fmt = s->dtype == SI_BF16 ? 1 : 0;
    P.status = status_dev;
    // gate/up: split K = d_model so that about one wave of CTAs is launched
    // the grid is sized for the largest possible union; with few tokens the real union is much
    // smaller and the surplus CTAs exit at once, so aim at about two CTAs per SM there
    int s1 = (t_pad_alloc <= 64 ? 2 * s->num_sms + m_tiles * tok_tiles - 1 : s->num_sms) / (m_tiles * tok_tiles);
    const int k_chunks = d / kChunkK;
    if (s1 < 1) s1 = 1;
    if (s1 > 8) s1 = 8;
    if (s1 > k_chunks) s1 = k_chunks;
    while (s1 > 1 && (size_t)s1 * 2 * nu_pad * t_pad_alloc * 4 > kPartialCap) --s1;
    if ((size_t)s1 * 2 * nu_pad * t_pad_alloc * 4 > ws.partial_bytes) return SI_ERR_NOMEM;
    if ((size_t)t_pad_alloc * nu_pad * 2 > ws.h_bytes) return SI_ERR_NOMEM;
    {
        const size_t stage = 2 * 128 * 128 + (size_t)n_tok * 128;
        P.nstage = pick_stages_gemm(stage, n_tok); P.n_split = s1;
        if (P.nstage < 2) return SI_ERR_UNSUPPORTED;
        size_t smem = (size_t)P.nstage * stage + 256;
        SI_CUDA_TRY(cudaFuncSetAttribute(si_gemm_gateup_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
        dim3 grid(m_tiles, s1, tok_tiles);
        si_gemm_gateup_kernel<<<grid, kGemmThreads, smem, stream>>>(P);
    }
    {
        dim3 grid((t_pad_alloc + 31) / 32, (nu_pad + 7) / 8);
        if (s->dtype == SI_BF16)
            si_gemm_combine_kernel<SI_BF16><<<grid, 256, 0, stream>>>(P.partial, s1, nu_pad, t_pad_alloc, T, n_union, masks, mask_words, (uint16_t *)(wsb + ws.h_off));
        else
            si_gemm_combine_kernel<SI_F16><<<grid, 256, 0, stream>>>(P.partial, s1, nu_pad, t_pad_alloc, T, n_union, masks, mask_words, (uint16_t *)(wsb + ws.h_off));
    }
    // down: split K = union
    int s2 = (t_pad_alloc <= 64 ? 2 * s->num_sms : s->num_sms) / ((d / 128) * tok_tiles);
    if (s2 < 1) s2 = 1;
    if (s2 > 8) s2 = 8;
    if (s2 > nu_pad / kChunkK) s2 = nu_pad / kChunkK;
    while (s2 > 1 && (size_t)s2 * t_pad_alloc * d * 4 > kPartialCap) --s2;
    if ((size_t)s2 * t_pad_alloc * d * 4 > ws.partial_bytes) return SI_ERR_NOMEM;
    {
        const size_t stage = 64 * 256 + (size_t)n_tok * 128;
        P.nstage = pick_stages_gemm(stage, n_tok); P.n_split = s2;
        size_t smem = (size_t)P.nstage * stage + 256;
        SI_CUDA_TRY(cudaFuncSetAttribute(si_gemm_down_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
        dim3 grid(d / 128, s2, tok_tiles);
        si_gemm_down_kernel<<<grid, kGemmThreads, smem, stream>>>(P);
    }
    {
        dim3 grid((d + 255) / 256, T);
        if (s->dtype == SI_BF16)
            si_gemm_reduce_kernel<SI_BF16><<<grid, 256, 0, stream>>>(P.partial, s2, t_pad_alloc, d, T, (const uint16_t *)x, y, y_dtype == SI_F32, (flags & SI_FLAG_RESIDUAL) != 0);
        else
            si_gemm_reduce_kernel<SI_F16><<<grid, 256, 0, stream>>>(P.partial, s2, t_pad_alloc, d, T, (const uint16_t *)x, y, y_dtype == SI_F32, (flags & SI_FLAG_RESIDUAL) != 0);
    }
    SI_CUDA_TRY(cudaGetLastError());
    return SI_OK;
}
