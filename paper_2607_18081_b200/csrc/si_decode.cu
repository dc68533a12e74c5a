// Batch-1 selective decode (Section 5, "Selective Computation"):
//     y = sum over selected slots i of SiLU(gate_i . x) * (up_i . x) * down_i
// Purely HBM-bound: 6*d_model bytes and 6*d_model flops per selected neuron.
//
// Two implementations share the per-record arithmetic:
//   * "simple": one launch per step, records read with 16-byte global loads, per-CTA fp32
//     partial outputs reduced in CTA order by a second kernel;
//   * "persistent" (si_decode_persistent.cuh): one launch for any number of steps, records
//     streamed through a shared-memory ring by bulk async copies.
// Both accumulate in a fixed order, so results are run-to-run bit-identical.
#include <atomic>

#include "si_common.cuh"
#include "si_decode_persistent.cuh"

namespace {

constexpr int kThreads = 256;
constexpr int kSimpleCtasPerSm = 2;

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

__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xFFFFFFFFu, v, o);
    return v;
}

// One CTA walks list positions blockIdx.x, blockIdx.x + G, ... two at a time.  Thread t
// owns 16-byte chunks t, t + 256, ... of every row, i.e. 8*NCH output columns.
template <int DT, int NCH>
__global__ void __launch_bounds__(kThreads)
si_decode_partial_kernel(const uint4 *__restrict__ rec, int n_loaded, int chunks,
                         const uint4 *__restrict__ x, const int32_t *__restrict__ idx,
                         const int32_t *__restrict__ offsets, int list, int k_fixed,
                         float *__restrict__ partial, int32_t *status) {
    __shared__ float red[2][kThreads / 32][4];
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");   // the reduce kernel may be scheduled already
    asm volatile("griddepcontrol.wait;" ::: "memory");                // x and the list may come from the kernel before
    const int base = offsets ? offsets[list] : list * k_fixed;
    const int k = offsets ? offsets[list + 1] - base : k_fixed;
    idx += base;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    float xr[NCH][8], acc[NCH][8];
#pragma unroll
    for (int i = 0; i < NCH; ++i) {
        int c = tid + kThreads * i;
        uint4 v = c < chunks ? __ldg(x + c) : make_uint4(0, 0, 0, 0);
        unpack8<DT>(v, xr[i]);
#pragma unroll
        for (int e = 0; e < 8; ++e) acc[i][e] = 0.f;
    }
    const int G = gridDim.x;
    int it = 0;
    for (int p = blockIdx.x; p < k; p += 2 * G, ++it) {
        int s0 = idx[p];
        int s1 = (p + G < k) ? idx[p + G] : -1;
        bool ok0 = s0 >= 0 && s0 < n_loaded;
        bool ok1 = s1 >= 0 && s1 < n_loaded;
        if (tid == 0 && status && (!ok0 || (!ok1 && p + G < k))) atomicCAS(status, 0, SI_ERR_OUT_OF_RANGE);
        const uint4 *r0 = rec + (size_t)(ok0 ? s0 : 0) * 3 * chunks;
        const uint4 *r1 = rec + (size_t)(ok1 ? s1 : 0) * 3 * chunks;
        float g0 = 0.f, u0 = 0.f, g1 = 0.f, u1 = 0.f;
        uint4 dn0[NCH], dn1[NCH];
#pragma unroll
        for (int i = 0; i < NCH; ++i) {
            int c = tid + kThreads * i;
            dn0[i] = dn1[i] = make_uint4(0, 0, 0, 0);
            if (c < chunks) {
                if (ok0) {
                    uint4 a = __ldg(r0 + c), b = __ldg(r0 + chunks + c);
                    dn0[i] = __ldg(r0 + 2 * chunks + c);
                    g0 += dot8<DT>(a, xr[i]); u0 += dot8<DT>(b, xr[i]);
                }
                if (ok1) {
                    uint4 a = __ldg(r1 + c), b = __ldg(r1 + chunks + c);
                    dn1[i] = __ldg(r1 + 2 * chunks + c);
                    g1 += dot8<DT>(a, xr[i]); u1 += dot8<DT>(b, xr[i]);
                }
            }
        }
        g0 = warp_sum(g0); u0 = warp_sum(u0); g1 = warp_sum(g1); u1 = warp_sum(u1);
        float(*buf)[4] = red[it & 1];
        if (lane == 0) { buf[warp][0] = g0; buf[warp][1] = u0; buf[warp][2] = g1; buf[warp][3] = u1; }
        __syncthreads();
        g0 = u0 = g1 = u1 = 0.f;
#pragma unroll
        for (int w = 0; w < kThreads / 32; ++w) {
            g0 += buf[w][0]; u0 += buf[w][1]; g1 += buf[w][2]; u1 += buf[w][3];
        }
        float h0 = ok0 ? si_silu_mul(g0, u0) : 0.f;
        float h1 = ok1 ? si_silu_mul(g1, u1) : 0.f;
#pragma unroll
        for (int i = 0; i < NCH; ++i) {
            float f0[8], f1[8];
            unpack8<DT>(dn0[i], f0); unpack8<DT>(dn1[i], f1);
#pragma unroll
            for (int e = 0; e < 8; ++e) acc[i][e] = fmaf(h1, f1[e], fmaf(h0, f0[e], acc[i][e]));
        }
    }
    float4 *out = reinterpret_cast<float4 *>(partial + (size_t)blockIdx.x * chunks * 8);
#pragma unroll
    for (int i = 0; i < NCH; ++i) {
        int c = tid + kThreads * i;
        if (c < chunks) {
            out[2 * c] = make_float4(acc[i][0], acc[i][1], acc[i][2], acc[i][3]);
            out[2 * c + 1] = make_float4(acc[i][4], acc[i][5], acc[i][6], acc[i][7]);
        }
    }
}

// The same walk for rows of at most 768 chunks (d_model <= 6144), one record at a time with the loads of
// the next P records already in flight: the records of a walker are independent, so nothing but registers
// limits how far ahead their loads may run.  The list entry of the record after those is fetched one
// record early, so that no address waits for it.  A CTA holds SETS independent walkers of 256 threads
// (W = 256; rows of more than 768 chunks get one walker of W = 512 threads; walker v of all takes list
// positions v, v + walkers, ...), each with its own named barrier; with two,
// the second leaves its sums in shared memory and the first adds them to its own, so the CTA writes one
// partial row: half as many rows for the reduce kernel as with one walker per CTA.
template <int DT, int NCH, int P, int SETS, int W>
__global__ void __launch_bounds__(W * SETS, 512 / (W * SETS))
si_decode_partial_ahead_kernel(const uint4 *__restrict__ rec, int n_loaded, int chunks,
                               const uint4 *__restrict__ x, const int32_t *__restrict__ idx,
                               const int32_t *__restrict__ offsets, int list, int k_fixed,
                               float *__restrict__ partial, int32_t *status) {
    __shared__ float red[SETS][2][W / 32][2];
    __shared__ float4 merge[SETS > 1 ? 2 * NCH * W : 1];
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    asm volatile("griddepcontrol.wait;" ::: "memory");                // x and the list may come from the kernel before
    const int base = offsets ? offsets[list] : list * k_fixed;
    const int k = offsets ? offsets[list + 1] - base : k_fixed;
    idx += base;
    const int q = threadIdx.x / W, tid = threadIdx.x % W, lane = tid & 31, warp = tid >> 5;
    const int G = gridDim.x * SETS, vb = blockIdx.x * SETS + q;      // walkers, this one's index
    const int n_mine = k > vb ? (k - vb + G - 1) / G : 0;             // records of this walker
    const int32_t *my = idx + vb;
    int first[P];
#pragma unroll
    for (int st = 0; st < P; ++st) first[st] = st < n_mine ? my[(size_t)st * G] : 0;
    int ahead = P < n_mine ? my[(size_t)P * G] : 0;              // list entry of record j + P
    uint4 xp[NCH];
    float acc[NCH][8];
#pragma unroll
    for (int i = 0; i < NCH; ++i) {
        const int c = tid + W * i;
        xp[i] = c < chunks ? __ldg(x + c) : make_uint4(0, 0, 0, 0);
#pragma unroll
        for (int e = 0; e < 8; ++e) acc[i][e] = 0.f;
    }
    uint4 buf[P][3 * NCH];
    bool ok[P];
    auto fetch = [&](uint4 (&b)[3 * NCH], bool &good, int slot) {
        good = slot >= 0 && slot < n_loaded;
        if (!good && tid == 0 && status) atomicCAS(status, 0, SI_ERR_OUT_OF_RANGE);
        const uint4 *r = rec + (size_t)(good ? slot : 0) * 3 * chunks;
#pragma unroll
        for (int i = 0; i < NCH; ++i) {
            const int c = tid + W * i;
            if (c < chunks) {
                b[3 * i] = __ldg(r + c); b[3 * i + 1] = __ldg(r + chunks + c); b[3 * i + 2] = __ldg(r + 2 * chunks + c);
            } else {
                b[3 * i] = b[3 * i + 1] = b[3 * i + 2] = make_uint4(0, 0, 0, 0);
            }
        }
    };
#pragma unroll
    for (int st = 0; st < P; ++st) {
        ok[st] = false;
        if (st < n_mine) fetch(buf[st], ok[st], first[st]);
    }
    for (int j0 = 0; j0 < n_mine; j0 += P) {
#pragma unroll
        for (int st = 0; st < P; ++st) {
            const int j = j0 + st;
            if (j < n_mine) {                                      // uniform over the walker
                float g = 0.f, u = 0.f;
#pragma unroll
                for (int i = 0; i < NCH; ++i) {
                    float xr[8];
                    unpack8<DT>(xp[i], xr);
                    g += dot8<DT>(buf[st][3 * i], xr); u += dot8<DT>(buf[st][3 * i + 1], xr);
                }
                g = warp_sum(g); u = warp_sum(u);
                float(*rb)[2] = red[q][j & 1];
                if (lane == 0) { rb[warp][0] = g; rb[warp][1] = u; }
                if (SETS == 1) __syncthreads();
                else asm volatile("bar.sync %0, %1;" ::"r"(1 + q), "n"(W) : "memory");   // this walker's 256 threads
                g = u = 0.f;
#pragma unroll
                for (int w = 0; w < W / 32; ++w) { g += rb[w][0]; u += rb[w][1]; }
                const float h = ok[st] ? si_silu_mul(g, u) : 0.f;
#pragma unroll
                for (int i = 0; i < NCH; ++i) {
                    float f[8];
                    unpack8<DT>(buf[st][3 * i + 2], f);
#pragma unroll
                    for (int e = 0; e < 8; ++e) acc[i][e] = fmaf(h, f[e], acc[i][e]);
                }
                const int jn = j + P;
                if (jn < n_mine) fetch(buf[st], ok[st], ahead);
                ahead = jn + 1 < n_mine ? my[(size_t)(jn + 1) * G] : 0;
            }
        }
    }
    if (SETS > 1) {
        if (q == 1) {
#pragma unroll
            for (int i = 0; i < NCH; ++i) {
                merge[(2 * i) * W + tid] = make_float4(acc[i][0], acc[i][1], acc[i][2], acc[i][3]);
                merge[(2 * i + 1) * W + tid] = make_float4(acc[i][4], acc[i][5], acc[i][6], acc[i][7]);
            }
        }
        __syncthreads();
        if (q != 0) return;
#pragma unroll
        for (int i = 0; i < NCH; ++i) {
            const float4 lo = merge[(2 * i) * W + tid], hi = merge[(2 * i + 1) * W + tid];
            acc[i][0] += lo.x; acc[i][1] += lo.y; acc[i][2] += lo.z; acc[i][3] += lo.w;
            acc[i][4] += hi.x; acc[i][5] += hi.y; acc[i][6] += hi.z; acc[i][7] += hi.w;
        }
    }
    float4 *out = reinterpret_cast<float4 *>(partial + (size_t)blockIdx.x * chunks * 8);
#pragma unroll
    for (int i = 0; i < NCH; ++i) {
        const int c = tid + W * i;
        if (c < chunks) {
            out[2 * c] = make_float4(acc[i][0], acc[i][1], acc[i][2], acc[i][3]);
            out[2 * c + 1] = make_float4(acc[i][4], acc[i][5], acc[i][6], acc[i][7]);
        }
    }
}

// y[j] = (x[j] +) sum over the partial rows g = 0..G-1 of partial[g][j].  One block per 32 output columns
// (eight float4 groups); thread (group = tid & 7, row class = tid >> 3) sums rows class, class + 32, ... in
// ascending order, five loads in flight (one round for up to 160 rows).  The 32 classes are then added in
// a fixed tree -- the four classes of a warp by two shuffle steps, the eight warps in warp order -- so the
// result does not depend on scheduling.
template <int DT>
__global__ void __launch_bounds__(256)
si_decode_reduce_kernel(const float *__restrict__ partial, int G, int d,
                             const uint16_t *__restrict__ x, void *__restrict__ y,
                             int y_f32, int residual) {
    __shared__ float4 part[8][8];
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");   // a following kernel may be scheduled (it waits for y itself)
    asm volatile("griddepcontrol.wait;" ::: "memory");                // the partial rows of the preceding kernel
    const int g = threadIdx.x & 7, rc = threadIdx.x >> 3, warp = threadIdx.x >> 5;
    const int col = (blockIdx.x * 8 + g) * 4;
    float4 a = make_float4(0.f, 0.f, 0.f, 0.f);
    if (col < d) {
        for (int r0 = rc; r0 < G; r0 += 32 * 5) {
            float4 v[5];
#pragma unroll
            for (int j = 0; j < 5; ++j) {
                const int r = r0 + 32 * j;
                v[j] = r < G ? __ldg(reinterpret_cast<const float4 *>(partial + (size_t)r * d + col)) : make_float4(0.f, 0.f, 0.f, 0.f);
            }
#pragma unroll
            for (int j = 0; j < 5; ++j) { a.x += v[j].x; a.y += v[j].y; a.z += v[j].z; a.w += v[j].w; }
        }
    }
#pragma unroll
    for (int o = 8; o <= 16; o <<= 1) {
        a.x += __shfl_xor_sync(0xFFFFFFFFu, a.x, o); a.y += __shfl_xor_sync(0xFFFFFFFFu, a.y, o);
        a.z += __shfl_xor_sync(0xFFFFFFFFu, a.z, o); a.w += __shfl_xor_sync(0xFFFFFFFFu, a.w, o);
    }
    if ((threadIdx.x & 31) < 8) part[warp][g] = a;
    __syncthreads();
    if (threadIdx.x >= 8 || col >= d) return;
    a = part[0][g];
#pragma unroll
    for (int w = 1; w < 8; ++w) { const float4 v = part[w][g]; a.x += v.x; a.y += v.y; a.z += v.z; a.w += v.w; }
    if (residual) {
        const uint2 xw = *reinterpret_cast<const uint2 *>(x + col);
        a.x += si_cvt<DT>::lo(xw.x); a.y += si_cvt<DT>::hi(xw.x); a.z += si_cvt<DT>::lo(xw.y); a.w += si_cvt<DT>::hi(xw.y);
    }
    if (y_f32) {
        *reinterpret_cast<float4 *>(reinterpret_cast<float *>(y) + col) = a;
    } else {
        uint2 w;
        w.x = (uint32_t)si_cvt<DT>::from_float(a.x) | ((uint32_t)si_cvt<DT>::from_float(a.y) << 16);
        w.y = (uint32_t)si_cvt<DT>::from_float(a.z) | ((uint32_t)si_cvt<DT>::from_float(a.w) << 16);
        *reinterpret_cast<uint2 *>(reinterpret_cast<uint16_t *>(y) + col) = w;
    }
}

template <int DT>
int launch_simple_step(const si_store *s, int layer, const void *x, const int32_t *idx,
                       const int32_t *offsets, int list, int k, void *y, int y_dtype, unsigned flags,
                       float *partial, int max_ctas, int32_t *status_dev, cudaStream_t stream, int *rows_only = nullptr) {
    const int d = s->d_model, chunks = d / 8;
    const int nch = (chunks + kThreads - 1) / kThreads;
    int G = k < max_ctas ? (k < 1 ? 1 : k) : max_ctas;          // one partial row per CTA
    const uint4 *rec = (const uint4 *)s->records(layer);
    const int nl = s->n_loaded[layer];
    // Both kernels are launched as programmatic dependents: each may be scheduled while its predecessor in
    // the stream finishes and waits for that kernel's results with griddepcontrol.wait before it reads
    // anything.  After a predecessor that never triggers early this is an ordinary launch.
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(G); cfg.blockDim = dim3(kThreads); cfg.dynamicSmemBytes = 0; cfg.stream = stream;
    cfg.attrs = attr; cfg.numAttrs = 1;
    const uint4 *x4 = (const uint4 *)x;
#define SI_LAUNCH_PARTIAL(N)                                                                                       \
    SI_CUDA_TRY(cudaLaunchKernelEx(&cfg, si_decode_partial_kernel<DT, N>, rec, nl, chunks, x4, idx, offsets, list, k, \
                                   partial, status_dev))
#define SI_LAUNCH_AHEAD(N, P, SETS, W)                                                                                        \
    SI_CUDA_TRY(cudaLaunchKernelEx(&cfg, si_decode_partial_ahead_kernel<DT, N, P, SETS, W>, rec, nl, chunks, x4, idx, offsets, \
                                   list, k, partial, status_dev))
    if (nch <= 3) {
        // two walkers of 256 threads per CTA, one CTA per SM slot pair: one partial row per CTA
        G = (G + 1) / 2;
        cfg.gridDim = dim3(G); cfg.blockDim = dim3(2 * kThreads);
        if (nch <= 1) SI_LAUNCH_AHEAD(1, 4, 2, 256);
        else if (nch <= 2) SI_LAUNCH_AHEAD(2, 3, 2, 256);
        else SI_LAUNCH_AHEAD(3, 2, 2, 256);
    } else if (nch <= 4) {
        // rows of up to 1024 chunks (d_model <= 8192): one walker of 512 threads per CTA and SM
        G = (G + 1) / 2;
        cfg.gridDim = dim3(G); cfg.blockDim = dim3(512);
        SI_LAUNCH_AHEAD(2, 3, 1, 512);
    }
    else if (nch <= 8) SI_LAUNCH_PARTIAL(8);
    else return SI_ERR_UNSUPPORTED;
#undef SI_LAUNCH_PARTIAL
#undef SI_LAUNCH_AHEAD
    if (rows_only) {                  // the caller sums the partial rows itself (the sharded path: sum and exchange in one kernel)
        *rows_only = G;
        SI_CUDA_TRY(cudaGetLastError());
        return SI_OK;
    }
    cfg.gridDim = dim3((d + 31) / 32); cfg.blockDim = dim3(256);
    SI_CUDA_TRY(cudaLaunchKernelEx(&cfg, si_decode_reduce_kernel<DT>, (const float *)partial, G, d, (const uint16_t *)x, y,
                                   (int)(y_dtype == SI_F32), (int)((flags & SI_FLAG_RESIDUAL) != 0)));
    SI_CUDA_TRY(cudaGetLastError());
    return SI_OK;
}

}  // namespace

// The first kernel of a single step alone: fp32 partial rows [*rows_out][d_model] in `partial` (room for 2 rows per SM).
int si_decode_partial_launch(const si_store *s, int layer, const void *x, const int32_t *idx, int k, float *partial,
                             int32_t *status_dev, cudaStream_t stream, int *rows_out) {
    return s->dtype == SI_BF16
               ? launch_simple_step<SI_BF16>(s, layer, x, idx, nullptr, 0, k, nullptr, SI_F32, 0, partial, kSimpleCtasPerSm * s->num_sms, status_dev, stream, rows_out)
               : launch_simple_step<SI_F16>(s, layer, x, idx, nullptr, 0, k, nullptr, SI_F32, 0, partial, kSimpleCtasPerSm * s->num_sms, status_dev, stream, rows_out);
}

int si_decode_launch(const si_store *s, int n_steps, const int32_t *layers_host, const void *x,
                     const int32_t *idx, const int32_t *idx_offsets, int k_fixed, void *y,
                     int y_dtype, unsigned flags, void *workspace, size_t ws_bytes,
                     int32_t *status_dev, cudaStream_t stream, const si_decode_extra *ex) {
    si_ws_layout ws = si_ws_carve(s, 1, k_fixed, n_steps);
    if (ws_bytes < ws.total) return SI_ERR_NOMEM;
    if (n_steps <= 0) return SI_ERR_INVALID_ARG;
    for (int st = 0; st < n_steps; ++st) {
        int l = layers_host ? layers_host[st] : st % s->n_layers;
        if (l < 0 || l >= s->n_layers) return SI_ERR_INVALID_ARG;
        if (!s->loaded[l]) return SI_ERR_INVALID_ARG;
    }
    char *wsb = (char *)workspace;
    // one or two steps are served faster by two plain launches each than by starting the persistent
    // kernel: a launch of it costs about 33 us beyond its steps, a plain step 12 us against 5.4 us
    // (replayed from a CUDA graph; launched one by one from the host three steps already favour the
    // persistent kernel, whose single launch costs the host less than six)
    const bool chained = ex && (ex->chain_len > 0 || ex->n_static > 0);
    if (chained && !si_persistent_supported(s)) return SI_ERR_UNSUPPORTED;    // chains and static prefixes live in the persistent kernel
    const bool use_simple = !chained && ((flags & SI_FLAG_SIMPLE_KERNELS) != 0 || !si_persistent_supported(s) || n_steps <= 2);
    if (!use_simple)
        return si_decode_persistent_launch(s, n_steps, layers_host, x, idx, idx_offsets, k_fixed, y, y_dtype, flags,
                                           wsb, ws, status_dev, stream, ex);
    // simple path: one partial + one reduce launch per step.  With CSR lists the true length
    // is read on the device; k_fixed (an upper bound) only sizes the grid.
    const size_t esz = 2, ysz = (y_dtype == SI_F32) ? 4 : 2;
    float *partial = (float *)(wsb + ws.partial_off);
    // CTAs of the partial kernel (one fp32 row of the partial buffer each): as many as can be resident
    int max_ctas = kSimpleCtasPerSm * s->num_sms;
    const size_t rows = ws.partial_bytes / ((size_t)s->d_model * 4);
    if ((size_t)max_ctas > rows) max_ctas = (int)rows;
    for (int st = 0; st < n_steps; ++st) {
        int l = layers_host ? layers_host[st] : st % s->n_layers;
        const int list = ((flags & SI_FLAG_LIST_PER_LAYER) && !idx_offsets) ? l : st;   // which list the step uses
        const void *xs = (const char *)x + (size_t)st * s->d_model * esz;
        void *ys = (char *)y + (size_t)st * s->d_model * ysz;
        int rc = (s->dtype == SI_BF16)
                     ? launch_simple_step<SI_BF16>(s, l, xs, idx, idx_offsets, list, k_fixed, ys, y_dtype, flags, partial, max_ctas, status_dev, stream)
                     : launch_simple_step<SI_F16>(s, l, xs, idx, idx_offsets, list, k_fixed, ys, y_dtype, flags, partial, max_ctas, status_dev, stream);
        if (rc != SI_OK) return rc;
    }
    return SI_OK;
}

// ---------------------------------------------------------------------------------------------
// Entry point for callers that cannot allocate device memory.
//
// The per-step kernels above need scratch for the per-CTA partial outputs.  Here that scratch is
// a fixed array that is part of the library image: it is reserved on every GPU that loads the
// library and stays reserved until the process exits.
namespace {

constexpr int kNoAllocMaxDModel = 8192;
constexpr int kNoAllocMaxCtas = 304;          // 2 CTAs per SM on up to 152 SMs
static __device__ __align__(256) float si_noalloc_scratch[(size_t)kNoAllocMaxCtas * kNoAllocMaxDModel];

// In host code the array's name above is only a handle; the device address has to be asked for,
// once per device, with that device current.
struct NoAllocDevices {
    std::atomic<void *> ptr[64];      // null until the device's address has been looked up
};
NoAllocDevices &noalloc_devices() {
    static NoAllocDevices d;           // zero-initialised; constructed once (thread-safe in C++11)
    return d;
}

// `dev` must be the current device.  Two host threads that make the first call on a device at the
// same time both look the address up and both store the same value.
int noalloc_scratch_for_device(int dev, float **out) {
    if (dev < 0 || dev >= 64) return SI_ERR_UNSUPPORTED;
    NoAllocDevices &d = noalloc_devices();
    void *p = d.ptr[dev].load(std::memory_order_acquire);
    if (!p) {
        SI_CUDA_TRY(cudaGetSymbolAddress(&p, si_noalloc_scratch));
        if (!p) return SI_ERR_CUDA;
        d.ptr[dev].store(p, std::memory_order_release);
    }
    *out = (float *)p;
    return SI_OK;
}

}  // namespace

extern "C" int si_ffn_forward_noalloc(const si_store_t *store, int layer, const void *x, const int32_t *idx,
                                      int k, void *y, int y_dtype, unsigned flags, int32_t *status_dev,
                                      void *stream_) {
    if (!si_store_ok(store) || !x || !y) return SI_ERR_INVALID_ARG;
    if (y_dtype != SI_F32 && y_dtype != store->dtype) return SI_ERR_INVALID_ARG;
    if (layer < 0 || layer >= store->n_layers || k < 0 || !store->loaded[layer]) return SI_ERR_INVALID_ARG;
    if (k > store->n_loaded[layer]) return SI_ERR_OUT_OF_RANGE;
    if (k > 0 && !idx) return SI_ERR_INVALID_ARG;
    if (!si_aligned16(x) || !si_aligned16(y) || (idx && !si_aligned16(idx))) return SI_ERR_ALIGNMENT;
    if (status_dev && (((uintptr_t)status_dev) & 3u)) return SI_ERR_ALIGNMENT;
    // the fixed scratch holds one fp32 row of d_model values per CTA of the partial kernel
    if (store->d_model > kNoAllocMaxDModel || 2 * store->num_sms > kNoAllocMaxCtas) return SI_ERR_TOO_LARGE;
    // the scratch address and the grid size belong to one device: the store's, which must be current
    int dev = -1;
    SI_CUDA_TRY(cudaGetDevice(&dev));
    if (dev != store->device) return SI_ERR_INVALID_ARG;
    float *scratch = nullptr;
    int rc = noalloc_scratch_for_device(dev, &scratch);
    if (rc != SI_OK) return rc;
    cudaStream_t stream = (cudaStream_t)stream_;
    // every CTA of the partial kernel writes its whole row before the reduce kernel reads it, so
    // nothing left over from an earlier call is ever read and nothing needs clearing
    const unsigned f = flags & SI_FLAG_RESIDUAL;
    return store->dtype == SI_BF16
               ? launch_simple_step<SI_BF16>(store, layer, x, idx, nullptr, 0, k, y, y_dtype, f, scratch, 2 * store->num_sms, status_dev, stream)
               : launch_simple_step<SI_F16>(store, layer, x, idx, nullptr, 0, k, y, y_dtype, f, scratch, 2 * store->num_sms, status_dev, stream);
}
