// Persistent batch-1 selective decode for sm_100a.
//
// One CTA per SM runs any number of (token, layer) steps in a single launch.  In each CTA
//   * warp 0 (producer) walks the CTA's share of every step's active list and streams each
//     selected neuron record -- 6*d_model contiguous bytes: gate row | up row | down row --
//     from HBM into a shared-memory ring with one bulk async copy (cp.async.bulk, completion
//     on an mbarrier).  The ring runs ahead across step boundaries, so HBM stays busy while
//     the consumers finish a step and synchronise;
//   * warps 1..8 (consumers) take records two at a time: each thread owns 8*NCH output
//     columns, forms its slice of the two dot products, the 256 threads reduce them
//     (shuffles + one named barrier), apply SiLU(g)*u and accumulate h * down into fp32
//     registers.  At the end of a step each CTA stores its partial y, all CTAs meet at a
//     counter barrier, and every CTA reduces a disjoint slice of columns over the partials
//     in CTA order (deterministic split-K), writing y once.
// List position p of step s goes to CTA (p + rot_s) mod G, rot_s = (number of list entries
// before step s) mod G, so the records are dealt round-robin across steps and no SM is
// persistently the one with an extra record.
//
// Every wait is bounded: on expiry the kernel records SI_ERR_TIMEOUT, raises a grid-wide
// abort flag, lets its outstanding copies land and returns.
#pragma once

#include <cooperative_groups.h>
#include "si_common.cuh"

#define SI_MAX_LAYERS 128

namespace si_persist {

constexpr int kConsumers = 256;
constexpr int kThreads = kConsumers + 32;
constexpr int kMaxStages = 16;
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
    float *partial;               // [2][G][d_model]
    unsigned int *ctrl;           // [0] barrier counter, [1] abort flag (both zero at launch)
    int32_t *status;
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
__device__ __forceinline__ void consumer_bar_sync() { asm volatile("bar.sync 1, %0;" ::"n"(kConsumers) : "memory"); }
__device__ __forceinline__ bool consumer_bar_or(bool v) {
    uint32_t r;
    asm volatile(
        "{\n\t.reg .pred p, q;\n\t"
        "setp.ne.u32 q, %1, 0;\n\t"
        "bar.red.or.pred p, 1, %2, q;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(r) : "r"((uint32_t)v), "n"(kConsumers) : "memory");
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
__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xFFFFFFFFu, v, o);
    return v;
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

template <int DT, int NCH>
__global__ void __launch_bounds__(kThreads, 1)
si_decode_persistent_kernel(const __grid_constant__ Params P) {
    extern __shared__ __align__(128) uint8_t smem[];
    const int rec_bytes = P.d_model * 6;
    const int nstage = P.nstage;
    uint8_t *ring = smem;
    uint64_t *full = reinterpret_cast<uint64_t *>(smem + (size_t)nstage * rec_bytes);
    uint64_t *empty = full + kMaxStages;
    int *meta = reinterpret_cast<int *>(empty + kMaxStages);           // [kMaxStages]
    float *red = reinterpret_cast<float *>(meta + kMaxStages);          // [2][8][4]
    float4 *red4 = reinterpret_cast<float4 *>(red + 64);                // [8]
    volatile int *cta_abort = reinterpret_cast<volatile int *>(red4 + 8);

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int G = gridDim.x, b = blockIdx.x;
    const int d = P.d_model, chunks = P.chunks;

    if (tid == 0) {
        for (int s = 0; s < nstage; ++s) { mbar_init(&full[s], 1); mbar_init(&empty[s], kConsumers / 32); }
        *cta_abort = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncthreads();

    if (warp == 0) {
        // ------------------------------------------------------------------ producer warp
        const uint64_t policy = l2_policy_evict_first();
        uint32_t n = 0;            // ring item counter
        uint32_t armed = 0;        // items armed so far (== n, kept for the drain)
        bool ok = true;
        StepGeom g = step_geom(P, 0, G, b);
        int layer = P.step_layers ? __ldg(P.step_layers) : 0;
        int slot_cur = -1;
        {
            int i = lane;
            if (i < g.cnt) slot_cur = __ldg(P.idx + g.base + g.first + (long long)i * G);
        }
        for (int step = 0; step < P.n_steps && ok; ++step) {
            // x item (its meta word carries the record count of the step)
            if (lane == 0) {
                int st = n % nstage; uint32_t ph = (n / nstage) & 1;
                ok = mbar_wait_bounded(&empty[st], ph ^ 1, cta_abort);
                if (ok) {
                    meta[st] = g.cnt;
                    mbar_arrive_expect_tx(&full[st], (uint32_t)d * 2);
                    bulk_g2s(ring + (size_t)st * rec_bytes, P.x + (size_t)step * d, (uint32_t)d * 2, &full[st], policy);
                }
            }
            ok = __shfl_sync(0xFFFFFFFFu, (int)ok, 0) != 0;
            if (!ok) break;
            ++n;
            const char *rec_base = P.store_base + P.rec_off[layer];
            const int n_loaded = P.n_loaded[layer];
            int i0 = 0;
            do {
                // prefetch the slots of the next batch (this step's next 32, or the next step's first 32)
                StepGeom gn = g; int step_n = step, i0_n = i0 + 32, layer_n = layer;
                if (i0_n >= g.cnt) {
                    step_n = step + 1; i0_n = 0;
                    if (step_n < P.n_steps) {
                        gn = step_geom(P, step_n, G, b);
                        layer_n = P.step_layers ? __ldg(P.step_layers + step_n) : step_n % P.n_layers;
                    }
                }
                int slot_nxt = -1;
                if (step_n < P.n_steps) {
                    int i = i0_n + lane;
                    if (i < gn.cnt) slot_nxt = __ldg(P.idx + gn.base + gn.first + (long long)i * G);
                }
                int nb = g.cnt - i0 < 32 ? g.cnt - i0 : 32;
                for (int j = 0; j < nb && ok; ++j) {
                    int slot = __shfl_sync(0xFFFFFFFFu, slot_cur, j);
                    if (lane == 0) {
                        int st = n % nstage; uint32_t ph = (n / nstage) & 1;
                        ok = mbar_wait_bounded(&empty[st], ph ^ 1, cta_abort);
                        if (ok) {
                            bool valid = slot >= 0 && slot < n_loaded;
                            meta[st] = valid ? 1 : 0;
                            if (valid) {
                                mbar_arrive_expect_tx(&full[st], (uint32_t)rec_bytes);
                                bulk_g2s(ring + (size_t)st * rec_bytes, rec_base + (size_t)slot * rec_bytes,
                                         (uint32_t)rec_bytes, &full[st], policy);
                            } else {
                                if (P.status) atomicCAS(P.status, 0, SI_ERR_OUT_OF_RANGE);
                                mbar_arrive(&full[st]);
                            }
                        }
                    }
                    ok = __shfl_sync(0xFFFFFFFFu, (int)ok, 0) != 0;
                    if (ok) ++n;
                }
                slot_cur = slot_nxt;
                if (step_n != step) { g = gn; layer = layer_n; break; }
                i0 = i0_n;
            } while (ok);
        }
        armed = n;
        if (!ok && lane == 0) {
            // give up: tell the consumers, then let every copy that was started land
            if (!*cta_abort) {
                *cta_abort = 1;
                if (P.status) atomicCAS(P.status, 0, SI_ERR_TIMEOUT);
                atomicExch(P.ctrl + 1, 1u);
            }
        }
        if (lane == 0 && (*cta_abort || !ok)) {
            uint32_t lo = armed > (uint32_t)nstage ? armed - nstage : 0;
            for (uint32_t m = lo; m < armed; ++m) {
                int st = m % nstage; uint32_t ph = (m / nstage) & 1;
                long long t0 = clock64();
                while (!mbar_try_wait(&full[st], ph) && clock64() - t0 < kWaitCycles) {}
            }
        }
        return;
    }

    // ---------------------------------------------------------------------- consumers
    const int ct = tid - 32;                 // 0..255
    const int cw = ct >> 5;                  // consumer warp 0..7
    uint32_t n = 0;
    bool fail = false;
    for (int step = 0; step < P.n_steps; ++step) {
        float xr[NCH][8], acc[NCH][8];
        int cnt;
        {
            int st = n % nstage; uint32_t ph = (n / nstage) & 1;
            fail |= !mbar_wait_bounded(&full[st], ph, cta_abort);
            cnt = fail ? 0 : meta[st];
            const uint4 *xs = reinterpret_cast<const uint4 *>(ring + (size_t)st * rec_bytes);
#pragma unroll
            for (int i = 0; i < NCH; ++i) {
                int c = ct + kConsumers * i;
                uint4 v = c < chunks ? xs[c] : make_uint4(0, 0, 0, 0);
                unpack8<DT>(v, xr[i]);
#pragma unroll
                for (int e = 0; e < 8; ++e) acc[i][e] = 0.f;
            }
            __syncwarp();
            if (lane == 0) mbar_arrive(&empty[st]);
            ++n;
        }
        // cnt must be agreed on by all consumer threads before it steers barriers
        if (consumer_bar_or(fail)) { fail = true; break; }

        int it = 0;
        for (int i = 0; i < cnt; i += 2, ++it) {
            const bool two = i + 1 < cnt;
            const int st0 = n % nstage; const uint32_t ph0 = (n / nstage) & 1;
            const int st1 = (n + 1) % nstage; const uint32_t ph1 = ((n + 1) / nstage) & 1;
            fail |= !mbar_wait_bounded(&full[st0], ph0, cta_abort);
            if (two) fail |= !mbar_wait_bounded(&full[st1], ph1, cta_abort);
            const bool ok0 = !fail && meta[st0] != 0;
            const bool ok1 = !fail && two && meta[st1] != 0;
            const uint4 *r0 = reinterpret_cast<const uint4 *>(ring + (size_t)st0 * rec_bytes);
            const uint4 *r1 = reinterpret_cast<const uint4 *>(ring + (size_t)st1 * rec_bytes);
            float g0 = 0.f, u0 = 0.f, g1 = 0.f, u1 = 0.f;
            uint4 dn0[NCH], dn1[NCH];
#pragma unroll
            for (int q = 0; q < NCH; ++q) {
                int c = ct + kConsumers * q;
                dn0[q] = dn1[q] = make_uint4(0, 0, 0, 0);
                if (c < chunks) {
                    if (ok0) {
                        uint4 a = r0[c], bb = r0[chunks + c];
                        dn0[q] = r0[2 * chunks + c];
                        g0 += dot8<DT>(a, xr[q]); u0 += dot8<DT>(bb, xr[q]);
                    }
                    if (ok1) {
                        uint4 a = r1[c], bb = r1[chunks + c];
                        dn1[q] = r1[2 * chunks + c];
                        g1 += dot8<DT>(a, xr[q]); u1 += dot8<DT>(bb, xr[q]);
                    }
                }
            }
            __syncwarp();
            if (lane == 0) { mbar_arrive(&empty[st0]); if (two) mbar_arrive(&empty[st1]); }
            n += two ? 2 : 1;
            g0 = warp_sum(g0); u0 = warp_sum(u0); g1 = warp_sum(g1); u1 = warp_sum(u1);
            float *buf = red + (it & 1) * 32;
            if (lane == 0) { buf[cw * 4 + 0] = g0; buf[cw * 4 + 1] = u0; buf[cw * 4 + 2] = g1; buf[cw * 4 + 3] = u1; }
            if (consumer_bar_or(fail)) { fail = true; break; }
            g0 = u0 = g1 = u1 = 0.f;
#pragma unroll
            for (int w = 0; w < kConsumers / 32; ++w) {
                g0 += buf[w * 4 + 0]; u0 += buf[w * 4 + 1]; g1 += buf[w * 4 + 2]; u1 += buf[w * 4 + 3];
            }
            const float h0 = ok0 ? si_silu_mul(g0, u0) : 0.f;
            const float h1 = ok1 ? si_silu_mul(g1, u1) : 0.f;
#pragma unroll
            for (int q = 0; q < NCH; ++q) {
                float f0[8], f1[8];
                unpack8<DT>(dn0[q], f0); unpack8<DT>(dn1[q], f1);
#pragma unroll
                for (int e = 0; e < 8; ++e) acc[q][e] = fmaf(h1, f1[e], fmaf(h0, f0[e], acc[q][e]));
            }
        }
        if (fail) break;

        // ---- split-K reduction across CTAs: store partial, barrier, reduce own column slice
        float *mine = P.partial + ((size_t)(step & 1) * G + b) * d;
#pragma unroll
        for (int q = 0; q < NCH; ++q) {
            int c = ct + kConsumers * q;
            if (c < chunks) {
                float4 *o = reinterpret_cast<float4 *>(mine + (size_t)c * 8);
                __stcg(o, make_float4(acc[q][0], acc[q][1], acc[q][2], acc[q][3]));
                __stcg(o + 1, make_float4(acc[q][4], acc[q][5], acc[q][6], acc[q][7]));
            }
        }
        consumer_bar_sync();
        if (ct == 0) {
            __threadfence();
            atomicAdd(P.ctrl, 1u);
            const unsigned target = (unsigned)(step + 1) * (unsigned)G;
            long long t0 = clock64();
            bool okb = true;
            while (true) {
                unsigned v;
                asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(P.ctrl) : "memory");
                if (v >= target) break;
                unsigned ab;
                asm volatile("ld.relaxed.gpu.global.u32 %0, [%1];" : "=r"(ab) : "l"(P.ctrl + 1) : "memory");
                if (ab || clock64() - t0 > kWaitCycles) { okb = false; break; }
            }
            if (!okb) {
                *cta_abort = 1;
                if (P.status) atomicCAS(P.status, 0, SI_ERR_TIMEOUT);
                atomicExch(P.ctrl + 1, 1u);
            }
            __threadfence();
        }
        consumer_bar_sync();
        if (*cta_abort) { fail = true; break; }

        {
            const int ngroups = d / 4;
            const int gpc = (ngroups + G - 1) / G;            // float4 column groups per CTA
            int gp = 1; while (gp < gpc) gp <<= 1;           // padded to a power of two (<= 256)
            const int LP = kConsumers / gp;                  // threads cooperating on one group
            const int gi = ct / LP, pl = ct % LP;
            const int grp = b * gpc + gi;
            const bool active = gi < gpc && grp < ngroups;
            const float *src = P.partial + (size_t)(step & 1) * G * d + (size_t)grp * 4;
            float4 v = make_float4(0.f, 0.f, 0.f, 0.f);
            if (active) {
                for (int gg = pl; gg < G; gg += LP) {
                    float4 t = __ldcg(reinterpret_cast<const float4 *>(src + (size_t)gg * d));
                    v.x += t.x; v.y += t.y; v.z += t.z; v.w += t.w;
                }
            }
            const int wl = LP < 32 ? LP : 32;
            for (int o = wl >> 1; o > 0; o >>= 1) {
                v.x += __shfl_xor_sync(0xFFFFFFFFu, v.x, o); v.y += __shfl_xor_sync(0xFFFFFFFFu, v.y, o);
                v.z += __shfl_xor_sync(0xFFFFFFFFu, v.z, o); v.w += __shfl_xor_sync(0xFFFFFFFFu, v.w, o);
            }
            if (LP > 32) {
                if (lane == 0) red4[cw] = v;
                consumer_bar_sync();
                if (pl == 0) {
                    const int w0 = gi * (LP / 32);
                    v = red4[w0];
                    for (int w = 1; w < LP / 32; ++w) {
                        float4 t = red4[w0 + w];
                        v.x += t.x; v.y += t.y; v.z += t.z; v.w += t.w;
                    }
                }
            }
            if (active && pl == 0) {
                const size_t col = (size_t)step * d + (size_t)grp * 4;
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
    }
    if (fail && ct == 0) {
        if (!*cta_abort) {
            *cta_abort = 1;
            if (P.status) atomicCAS(P.status, 0, SI_ERR_TIMEOUT);
            atomicExch(P.ctrl + 1, 1u);
        }
    }
}

inline size_t smem_bytes(int d_model, int nstage) {
    return (size_t)nstage * d_model * 6 + 2 * kMaxStages * 8 + kMaxStages * 4 + 64 * 4 + 8 * 16 + 64;
}
inline int pick_stages(int d_model) {
    const size_t budget = 227 * 1024 - 2048;
    int n = (int)((budget - smem_bytes(d_model, 0)) / ((size_t)d_model * 6));
    if (n > kMaxStages) n = kMaxStages;
    return n;
}

}  // namespace si_persist

inline bool si_persistent_supported(const si_store *s) {
    return s->n_layers <= SI_MAX_LAYERS && si_persist::pick_stages(s->d_model) >= 3 &&
           s->d_model / 8 <= si_persist::kConsumers * 8;
}

template <int DT, int NCH>
inline int si_decode_persistent_launch_t(const si_persist::Params &P, int G, cudaStream_t stream) {
    auto kern = si_persist::si_decode_persistent_kernel<DT, NCH>;
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
    if (layers_host) {
        int32_t *dst = (int32_t *)(wsb + ws.steps_off);
        SI_CUDA_TRY(cudaMemcpyAsync(dst, layers_host, (size_t)n_steps * 4, cudaMemcpyHostToDevice, stream));
        P.step_layers = dst;
    }
    P.x = (const uint16_t *)x; P.idx = idx; P.idx_offsets = idx_offsets; P.y = y;
    P.y_f32 = y_dtype == SI_F32; P.residual = (flags & SI_FLAG_RESIDUAL) != 0;
    P.partial = (float *)(wsb + ws.partial_off);
    P.ctrl = (unsigned int *)(wsb + ws.ctrl_off);
    P.status = status_dev;
    int G = s->num_sms;
    if (!idx_offsets && k_fixed < G) G = k_fixed < 1 ? 1 : k_fixed;
    SI_CUDA_TRY(cudaMemsetAsync(P.ctrl, 0, 256, stream));
    const int nch = (P.chunks + si_persist::kConsumers - 1) / si_persist::kConsumers;
#define SI_PL(DT)                                                               \
    (nch <= 1 ? si_decode_persistent_launch_t<DT, 1>(P, G, stream)              \
     : nch <= 2 ? si_decode_persistent_launch_t<DT, 2>(P, G, stream)            \
     : nch <= 4 ? si_decode_persistent_launch_t<DT, 4>(P, G, stream)            \
                : si_decode_persistent_launch_t<DT, 8>(P, G, stream))
    return s->dtype == SI_BF16 ? SI_PL(SI_BF16) : SI_PL(SI_F16);
#undef SI_PL
}
