// Runtime selector (Section 5: rank a token's activations from the largest down and record the
// indices of the top alpha).
//
// No sort is needed to obtain the set: one CTA per score row finds the k-th largest value by
// a 3-pass radix select (digits of 11, 11 and 10 bits) over order-preserving 32-bit keys held in
// shared memory, then one index-ordered prefix scan emits the selected indices ascending.  Ties at the k-th
// value go to the lower indices; +0 == -0; NaN has the lowest key.  All integer decisions:
// the result is exact and unique.
#include "si_common.cuh"

namespace {

constexpr int kSelThreads = 1024;
constexpr int kSmemKeys = 48 * 1024;   // rows up to this many scores keep their keys in shared memory
constexpr int kBins = 2048;            // histogram bins: digits of 11, 11 and 10 bits

__device__ __forceinline__ uint32_t score_key(float s, bool use_abs) {
    if (s != s) return 0u;                     // NaN: below everything
    if (use_abs) s = fabsf(s);
    if (s == 0.f) s = 0.f;                     // -0 -> +0
    uint32_t b = __float_as_uint(s);
    return (b & 0x80000000u) ? ~b : (b | 0x80000000u);
}

// Exclusive block scan of a pair of counters packed as (hi: a, lo: b) in 64 bits.
__device__ __forceinline__ unsigned long long block_exclusive_scan(unsigned long long v,
                                                                   unsigned long long *warp_tot,
                                                                   unsigned long long *total) {
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    unsigned long long inc = v;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        unsigned long long t = __shfl_up_sync(0xFFFFFFFFu, inc, o);
        if (lane >= o) inc += t;
    }
    if (lane == 31) warp_tot[warp] = inc;
    __syncthreads();
    if (warp == 0) {
        unsigned long long w = lane < kSelThreads / 32 ? warp_tot[lane] : 0ull;
        unsigned long long winc = w;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            unsigned long long t = __shfl_up_sync(0xFFFFFFFFu, winc, o);
            if (lane >= o) winc += t;
        }
        warp_tot[lane] = winc - w;                   // exclusive prefix of warp totals
        if (lane == 31) *total = winc;
    }
    __syncthreads();
    return warp_tot[warp] + inc - v;
}

// keys[i] = score_key(s[i]) for the whole row, by all threads of the CTA
__device__ __forceinline__ void load_keys(const float *__restrict__ s, uint32_t *keys, int n, bool use_abs) {
    const int tid = threadIdx.x;
    if (((reinterpret_cast<uintptr_t>(s) | reinterpret_cast<uintptr_t>(keys)) & 15u) == 0) {
        // all of a thread's 16-byte loads are issued before the first key is formed
        const float4 *s4 = reinterpret_cast<const float4 *>(s);
        const int n4 = n >> 2;
        for (int q0 = 0; q0 < n4; q0 += 4 * kSelThreads) {
            float4 v[4];
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                const int q = q0 + j * kSelThreads + tid;
                v[j] = q < n4 ? __ldg(s4 + q) : make_float4(0.f, 0.f, 0.f, 0.f);
            }
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                const int q = q0 + j * kSelThreads + tid;
                if (q < n4) {
                    uint4 kk;
                    kk.x = score_key(v[j].x, use_abs); kk.y = score_key(v[j].y, use_abs);
                    kk.z = score_key(v[j].z, use_abs); kk.w = score_key(v[j].w, use_abs);
                    *reinterpret_cast<uint4 *>(keys + 4 * q) = kk;
                }
            }
        }
        for (int i = 4 * n4 + tid; i < n; i += kSelThreads) keys[i] = score_key(s[i], use_abs);
    } else {
        for (int i = tid; i < n; i += kSelThreads) keys[i] = score_key(s[i], use_abs);
    }
}

// The same for a row of 16-bit scores (DT: SI_F16 / SI_BF16; widening to fp32 is exact, so the keys are
// those of the widened row)
template <int DT>
__device__ __forceinline__ void load_keys16(const uint16_t *__restrict__ s, uint32_t *keys, int n, bool use_abs) {
    const int tid = threadIdx.x;
    if (((reinterpret_cast<uintptr_t>(s) | reinterpret_cast<uintptr_t>(keys)) & 15u) == 0) {
        const uint4 *s8 = reinterpret_cast<const uint4 *>(s);
        const int n8 = n >> 3;
        for (int q0 = 0; q0 < n8; q0 += 2 * kSelThreads) {
            uint4 v[2];
#pragma unroll
            for (int j = 0; j < 2; ++j) {
                const int q = q0 + j * kSelThreads + tid;
                v[j] = q < n8 ? __ldg(s8 + q) : make_uint4(0, 0, 0, 0);
            }
#pragma unroll
            for (int j = 0; j < 2; ++j) {
                const int q = q0 + j * kSelThreads + tid;
                if (q < n8) {
                    uint4 lo, hi;
                    lo.x = score_key(si_cvt<DT>::lo(v[j].x), use_abs); lo.y = score_key(si_cvt<DT>::hi(v[j].x), use_abs);
                    lo.z = score_key(si_cvt<DT>::lo(v[j].y), use_abs); lo.w = score_key(si_cvt<DT>::hi(v[j].y), use_abs);
                    hi.x = score_key(si_cvt<DT>::lo(v[j].z), use_abs); hi.y = score_key(si_cvt<DT>::hi(v[j].z), use_abs);
                    hi.z = score_key(si_cvt<DT>::lo(v[j].w), use_abs); hi.w = score_key(si_cvt<DT>::hi(v[j].w), use_abs);
                    *reinterpret_cast<uint4 *>(keys + 8 * q) = lo;
                    *reinterpret_cast<uint4 *>(keys + 8 * q + 4) = hi;
                }
            }
        }
        for (int i = 8 * n8 + tid; i < n; i += kSelThreads) keys[i] = score_key(si_cvt<DT>::lo((uint32_t)s[i]), use_abs);
    } else {
        for (int i = tid; i < n; i += kSelThreads) keys[i] = score_key(si_cvt<DT>::lo((uint32_t)s[i]), use_abs);
    }
}

// Top-k of rows of at most PER * 1024 scores (0 < k < n): thread t keeps the keys of its index range
// [t*per, (t+1)*per) in registers, so the three radix passes and the emission read no memory but the
// histogram.  Each thread clears the two bins it reads, which readies the histogram for the next pass.
// SRC: type of the scores (SI_F32, or a 16-bit type).  With vote_counts set, every selected index adds one
// to its entry there (the frequency count of the prefill vote) and idx_out may be NULL.
template <int PER, int SRC>
__global__ void __launch_bounds__(kSelThreads)
si_select_topk_reg_kernel(const void *__restrict__ scores, int n, int row_stride, int k, int use_abs,
                          int32_t *__restrict__ idx_out, int out_stride, int cap, int32_t *__restrict__ n_out,
                          int *__restrict__ vote_counts) {
    extern __shared__ __align__(16) uint32_t smem_keys[];
    __shared__ __align__(8) unsigned int hist[kBins];
    __shared__ unsigned int warp_cnt[32];
    __shared__ unsigned long long warp_tot[32];
    __shared__ unsigned long long total;
    __shared__ uint32_t sh_prefix, sh_mask;
    __shared__ int sh_need;

    const int row = blockIdx.x, tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    int32_t *out = idx_out ? idx_out + (size_t)row * out_stride : nullptr;
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");   // a dependent kernel waits for the lists itself
    hist[tid] = 0; hist[tid + kSelThreads] = 0;
    if (SRC == SI_F32) load_keys(reinterpret_cast<const float *>(scores) + (size_t)row * row_stride, smem_keys, n, use_abs != 0);
    else load_keys16<SRC == SI_F32 ? SI_BF16 : SRC>(reinterpret_cast<const uint16_t *>(scores) + (size_t)row * row_stride, smem_keys, n, use_abs != 0);
    if (tid == 0) { sh_prefix = 0; sh_mask = 0; sh_need = k; }
    __syncthreads();
    const int per = (n + kSelThreads - 1) / kSelThreads;
    const int lo = min(n, tid * per), cnt = min(n, lo + per) - lo;
    uint32_t kr[PER];
#pragma unroll
    for (int j = 0; j < PER; ++j) kr[j] = j < cnt ? smem_keys[lo + j] : 0u;

#pragma unroll 1
    for (int pass = 0; pass < 3; ++pass) {
        const int shift = pass == 0 ? 21 : (pass == 1 ? 10 : 0);
        const uint32_t dmask = pass == 2 ? 1023u : 2047u;
        const uint32_t prefix = sh_prefix, mask = sh_mask;
        const int need = sh_need;
#pragma unroll
        for (int j = 0; j < PER; ++j)
            if (j < cnt && (kr[j] & mask) == prefix) atomicAdd(&hist[(kr[j] >> shift) & dmask], 1u);
        __syncthreads();
        // thread t owns bins 2047 - 2t and 2046 - 2t: a prefix sum over threads is a suffix sum over bins
        uint2 *hp = reinterpret_cast<uint2 *>(hist) + (kSelThreads - 1 - tid);
        const uint2 c2 = *hp;
        *hp = make_uint2(0u, 0u);
        const unsigned c_hi = c2.y, c_lo = c2.x, pair = c_hi + c_lo;
        unsigned inc = pair;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            const unsigned t = __shfl_up_sync(0xFFFFFFFFu, inc, o);
            if (lane >= o) inc += t;
        }
        if (lane == 31) warp_cnt[warp] = inc;
        __syncthreads();
        const unsigned wt = warp_cnt[lane];
        const unsigned excl = __reduce_add_sync(0xFFFFFFFFu, lane < warp ? wt : 0u) + inc - pair;   // keys in bins above this pair
        // the keys in play are at least `need`, so exactly one bin satisfies this (bin 0 at the latest)
        if (excl < (unsigned)need && (unsigned)need <= excl + c_hi) {
            sh_need = need - (int)excl;
            sh_prefix = prefix | ((uint32_t)(kBins - 1 - 2 * tid) << shift);
            sh_mask = mask | (dmask << shift);
        } else if (excl + c_hi < (unsigned)need && (unsigned)need <= excl + pair) {
            sh_need = need - (int)(excl + c_hi);
            sh_prefix = prefix | ((uint32_t)(kBins - 2 - 2 * tid) << shift);
            sh_mask = mask | (dmask << shift);
        }
        __syncthreads();
    }
    const uint32_t kstar = sh_prefix;
    const int r = sh_need;                 // r of the keys equal to kstar are taken, the lowest indices first

    uint32_t gm = 0, em = 0;
#pragma unroll
    for (int j = 0; j < PER; ++j) {
        if (j < cnt) { gm |= (uint32_t)(kr[j] > kstar) << j; em |= (uint32_t)(kr[j] == kstar) << j; }
    }
    const unsigned long long mine = ((unsigned long long)__popc(gm) << 32) | (unsigned long long)__popc(em);
    const unsigned long long before = block_exclusive_scan(mine, warp_tot, &total);
    const int gt_before = (int)(before >> 32), eq_before = (int)(before & 0xFFFFFFFFu);
    int eq_take = r - eq_before;
    eq_take = eq_take < 0 ? 0 : eq_take;
    uint32_t e = em, take = gm;
    for (int c = 0; c < eq_take && e; ++c) { take |= e & (0u - e); e &= e - 1; }
    int pos = gt_before + min(eq_before, r);
    while (take) {
        const int b = __ffs(take) - 1;
        take &= take - 1;
        if (out && pos < cap) out[pos] = lo + b;
        if (vote_counts) atomicAdd(&vote_counts[lo + b], 1);
        ++pos;
    }
    if (tid == 0 && n_out) {
        const int tot_gt = (int)(total >> 32), tot_eq = (int)(total & 0xFFFFFFFFu);
        n_out[row] = tot_gt + min(tot_eq, r);
    }
}

__global__ void __launch_bounds__(kSelThreads)
si_select_kernel(const float *__restrict__ scores, int n, int row_stride, int mode, int k, float tau,
                 int use_abs, int32_t *__restrict__ idx_out, int out_stride, int cap,
                 int32_t *__restrict__ n_out, uint32_t *__restrict__ key_spill, int keys_in_smem) {
    extern __shared__ __align__(16) uint32_t smem_keys[];
    __shared__ __align__(8) unsigned int hist[kBins];
    __shared__ unsigned long long warp_tot[32];
    __shared__ unsigned long long total;
    __shared__ uint32_t sh_prefix, sh_mask;
    __shared__ int sh_need;

    const int row = blockIdx.x, tid = threadIdx.x;
    const float *s = scores + (size_t)row * row_stride;
    int32_t *out = idx_out + (size_t)row * out_stride;
    uint32_t *keys = keys_in_smem ? smem_keys : key_spill + (size_t)row * n;

    uint32_t kstar = 0; int r = 0;          // threshold key and how many of its ties to take
    if (mode == SI_SELECT_TOPK) {
        load_keys(s, keys, n, use_abs != 0);
        if (tid == 0) { sh_prefix = 0; sh_mask = 0; sh_need = k; }
        __syncthreads();
        if (k > 0 && k < n) {
#pragma unroll 1
            for (int pass = 0; pass < 3; ++pass) {
                const int shift = pass == 0 ? 21 : (pass == 1 ? 10 : 0);
                const uint32_t dmask = pass == 2 ? 1023u : 2047u;
                hist[tid] = 0; hist[tid + kSelThreads] = 0;
                __syncthreads();
                const uint32_t prefix = sh_prefix, mask = sh_mask;
                const int need = sh_need;
                // histogram of the current digit over the keys that still match the prefix
                for (int i = tid; i < n; i += kSelThreads) {
                    const uint32_t key = keys[i];
                    if ((key & mask) == prefix) atomicAdd(&hist[(key >> shift) & dmask], 1u);
                }
                __syncthreads();
                // find the digit where the count from the largest digit down reaches `need`: thread t owns
                // bins 2047 - 2t and 2046 - 2t, so a prefix sum over threads is a suffix sum over bins
                const uint2 c2 = reinterpret_cast<const uint2 *>(hist)[kSelThreads - 1 - tid];
                const unsigned c_hi = c2.y, c_lo = c2.x, pair = c_hi + c_lo;
                unsigned inc = pair;
#pragma unroll
                for (int o = 1; o < 32; o <<= 1) {
                    const unsigned t = __shfl_up_sync(0xFFFFFFFFu, inc, o);
                    if ((tid & 31) >= o) inc += t;
                }
                if ((tid & 31) == 31) warp_tot[tid >> 5] = inc;
                __syncthreads();
                if (tid < 32) {
                    const unsigned w = (unsigned)warp_tot[tid];
                    unsigned winc = w;
#pragma unroll
                    for (int o = 1; o < 32; o <<= 1) {
                        const unsigned t = __shfl_up_sync(0xFFFFFFFFu, winc, o);
                        if (tid >= o) winc += t;
                    }
                    warp_tot[tid] = winc - w;
                }
                __syncthreads();
                const unsigned excl = (unsigned)warp_tot[tid >> 5] + inc - pair;    // keys in bins above this pair
                // the keys in play are at least `need`, so exactly one bin satisfies this (bin 0 at the latest)
                if (excl < (unsigned)need && (unsigned)need <= excl + c_hi) {
                    sh_need = need - (int)excl;
                    sh_prefix = prefix | ((uint32_t)(kBins - 1 - 2 * tid) << shift);
                    sh_mask = mask | (dmask << shift);
                } else if (excl + c_hi < (unsigned)need && (unsigned)need <= excl + pair) {
                    sh_need = need - (int)(excl + c_hi);
                    sh_prefix = prefix | ((uint32_t)(kBins - 2 - 2 * tid) << shift);
                    sh_mask = mask | (dmask << shift);
                }
                __syncthreads();
            }
            kstar = sh_prefix; r = sh_need;    // r of the keys equal to kstar are taken
        } else if (k >= n) {
            kstar = 0; r = n;                   // everything: all keys >= 0, ties = all
        } else {
            kstar = 0xFFFFFFFFu; r = 0;         // k == 0: nothing is taken (guards below)
        }
    }

    // index-ordered emission: thread t owns the contiguous range [t*per, (t+1)*per)
    const int per = (n + kSelThreads - 1) / kSelThreads;
    const int lo = min(n, tid * per), hi = min(n, lo + per);
    auto classify = [&](int i, bool &gt, bool &eq) {
        if (mode == SI_SELECT_TOPK) {
            const uint32_t key = keys[i];
            gt = (k > 0) && key > kstar; eq = (k > 0) && key == kstar;
            if (k >= n) { gt = false; eq = true; }
        } else {
            float v = s[i];
            if (use_abs) v = fabsf(v);
            gt = v > tau; eq = false;
        }
    };
    if (per <= 32) {
        // the range's answers fit two 32-bit masks: classify once, then walk the set bits
        uint32_t gm = 0, em = 0;
        for (int i = lo; i < hi; ++i) {
            bool gt, eq;
            classify(i, gt, eq);
            gm |= (uint32_t)gt << (i - lo); em |= (uint32_t)eq << (i - lo);
        }
        const unsigned long long mine = ((unsigned long long)__popc(gm) << 32) | (unsigned long long)__popc(em);
        const unsigned long long before = block_exclusive_scan(mine, warp_tot, &total);
        const int gt_before = (int)(before >> 32), eq_before = (int)(before & 0xFFFFFFFFu);
        int eq_take = r - eq_before;                           // ties of this range that are still taken: its first ones
        eq_take = eq_take < 0 ? 0 : eq_take;
        uint32_t e = em, take = gm;
        for (int c = 0; c < eq_take && e; ++c) { take |= e & (0u - e); e &= e - 1; }
        int pos = gt_before + min(eq_before, r);
        while (take) {
            const int b = __ffs(take) - 1;
            take &= take - 1;
            if (pos < cap) out[pos] = lo + b;
            ++pos;
        }
    } else {
        unsigned long long mine = 0;   // (hi 32: # strictly above threshold, lo 32: # ties)
        for (int i = lo; i < hi; ++i) {
            bool gt, eq;
            classify(i, gt, eq);
            mine += ((unsigned long long)gt << 32) | (unsigned long long)eq;
        }
        const unsigned long long before = block_exclusive_scan(mine, warp_tot, &total);
        int gt_before = (int)(before >> 32), eq_before = (int)(before & 0xFFFFFFFFu);
        for (int i = lo; i < hi; ++i) {
            bool gt, eq;
            classify(i, gt, eq);
            if (gt || (eq && eq_before < r)) {
                const int pos = gt_before + min(eq_before, r);
                if (pos < cap) out[pos] = i;
            }
            gt_before += gt; eq_before += eq;
        }
    }
    if (tid == 0 && n_out) {
        int tot_gt = (int)(total >> 32), tot_eq = (int)(total & 0xFFFFFFFFu);
        n_out[row] = tot_gt + min(tot_eq, r);
    }
}

int select_set_attrs() {
    static bool attr_set = false;
    if (!attr_set) {
        SI_CUDA_TRY(cudaFuncSetAttribute(si_select_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemKeys * 4));
#define SI_SEL_ATTR(P, S) SI_CUDA_TRY(cudaFuncSetAttribute(si_select_topk_reg_kernel<P, S>, cudaFuncAttributeMaxDynamicSharedMemorySize, P * kSelThreads * 4))
#define SI_SEL_ATTRS(S) SI_SEL_ATTR(4, S); SI_SEL_ATTR(8, S); SI_SEL_ATTR(16, S); SI_SEL_ATTR(32, S)
        SI_SEL_ATTRS(SI_F32); SI_SEL_ATTRS(SI_F16); SI_SEL_ATTRS(SI_BF16);
#undef SI_SEL_ATTRS
#undef SI_SEL_ATTR
        attr_set = true;
    }
    return SI_OK;
}

// the common case: a proper subset of a row whose keys fit the threads' registers
int select_reg_launch(const void *scores, int src, int n_rows, int n, int row_stride, int k, int use_abs, int32_t *idx_out,
                      int out_stride, int cap, int32_t *n_out, int *vote_counts, cudaStream_t stream) {
    const int per = (n + kSelThreads - 1) / kSelThreads;
#define SI_SELECT_REG2(P, S)                                                                                             \
    si_select_topk_reg_kernel<P, S><<<n_rows, kSelThreads, (size_t)n * 4, stream>>>(scores, n, row_stride, k, use_abs, \
                                                                                    idx_out, out_stride, cap, n_out, vote_counts)
#define SI_SELECT_REG(P)                                                   \
    do {                                                                   \
        if (src == SI_F32) SI_SELECT_REG2(P, SI_F32);                      \
        else if (src == SI_F16) SI_SELECT_REG2(P, SI_F16);                 \
        else SI_SELECT_REG2(P, SI_BF16);                                   \
    } while (0)
    if (per <= 4) SI_SELECT_REG(4);
    else if (per <= 8) SI_SELECT_REG(8);
    else if (per <= 16) SI_SELECT_REG(16);
    else SI_SELECT_REG(32);
#undef SI_SELECT_REG
#undef SI_SELECT_REG2
    SI_CUDA_TRY(cudaGetLastError());
    return SI_OK;
}

}  // namespace

size_t si_select_ws_bytes_impl(int n) {
    return n > kSmemKeys ? si_align_up((size_t)n * 4, 256) : 256;
}

int si_select_launch(const float *scores, int n_rows, int n, int row_stride, int mode, int k,
                     float tau, unsigned flags, int32_t *idx_out, int out_stride, int cap,
                     int32_t *n_out, void *workspace, size_t ws_bytes, cudaStream_t stream) {
    if (n_rows <= 0) return SI_OK;
    const int in_smem = n <= kSmemKeys;
    if (!in_smem && ws_bytes < (size_t)n_rows * n * 4) return SI_ERR_NOMEM;
    size_t smem = in_smem ? (size_t)(n > 0 ? n : 1) * 4 : 0;
    int arc = select_set_attrs();
    if (arc) return arc;
    const int use_abs = (flags & SI_FLAG_SCORE_ABS) != 0;
    if (mode == SI_SELECT_TOPK && k > 0 && k < n && n <= 32 * kSelThreads)
        return select_reg_launch(scores, SI_F32, n_rows, n, row_stride, k, use_abs, idx_out, out_stride, cap, n_out, nullptr, stream);
    si_select_kernel<<<n_rows, kSelThreads, smem, stream>>>(scores, n, row_stride, mode, k, tau, use_abs, idx_out,
                                                            out_stride, cap, n_out, (uint32_t *)workspace, in_smem);
    SI_CUDA_TRY(cudaGetLastError());
    return SI_OK;
}

// Per-token top-k of T rows (fp32 or 16-bit scores) counted straight into counts[n] (zero on entry): the
// first two steps of the prefill vote in one launch.  SI_ERR_UNSUPPORTED when the rows do not fit the
// register kernel (the caller then selects into lists and counts them).
int si_select_vote_launch(const void *scores, int src_dtype, int n_rows, int n, int row_stride, int k, unsigned flags,
                          int *counts, cudaStream_t stream) {
    if (!(k > 0 && k < n && n <= 32 * kSelThreads)) return SI_ERR_UNSUPPORTED;
    if (n_rows <= 0) return SI_OK;
    int rc = select_set_attrs();
    if (rc) return rc;
    return select_reg_launch(scores, src_dtype, n_rows, n, row_stride, k, (flags & SI_FLAG_SCORE_ABS) != 0, nullptr, 0, 0,
                             nullptr, counts, stream);
}

extern "C" int si_select_workspace_bytes(int n, size_t *bytes_out) {
    if (n < 0 || !bytes_out) return SI_ERR_INVALID_ARG;
    *bytes_out = si_select_ws_bytes_impl(n);
    return SI_OK;
}

extern "C" int si_select(const float *scores, int n, int mode, int k, float tau, unsigned flags,
                         int32_t *idx_out, int cap, int32_t *n_out, void *workspace, size_t ws_bytes,
                         void *stream) {
    if (!scores || !idx_out || n < 0 || cap < 0) return SI_ERR_INVALID_ARG;
    if (mode != SI_SELECT_TOPK && mode != SI_SELECT_THRESHOLD) return SI_ERR_INVALID_ARG;
    if (mode == SI_SELECT_TOPK && (k < 0 || k > n)) return SI_ERR_INVALID_ARG;
    if (mode == SI_SELECT_TOPK && cap < k) return SI_ERR_NOMEM;
    if (!si_aligned16(scores) || !si_aligned16(idx_out)) return SI_ERR_ALIGNMENT;
    if (n > kSmemKeys && (!workspace || ws_bytes < (size_t)n * 4)) return SI_ERR_NOMEM;
    if (n == 0) {
        if (n_out) SI_CUDA_TRY(cudaMemsetAsync(n_out, 0, 4, (cudaStream_t)stream));
        return SI_OK;
    }
    return si_select_launch(scores, 1, n, n, mode, k, tau, flags, idx_out, cap, cap, n_out, workspace,
                            ws_bytes, (cudaStream_t)stream);
}
