// Tensor-core plumbing shared by the contraction kernels: mbarrier, cp.async, TMA and tcgen05 wrappers (inline
// PTX), shared-memory and instruction descriptors, the parameter block of a multi-token call and the tensor
// map helper.  Everything here is internal to the library.
#pragma once
#include <cuda.h>       // CUtensorMap and the encode function's signature only; the function is looked up at run time

#include "si_common.cuh"

namespace si_tc {

constexpr int kLoaderThreads = 256;              // warps 0..7: gather loads, later the epilogue
constexpr int kLoaderWarps = kLoaderThreads / 32;
constexpr int kGemmThreads = kLoaderThreads + 32; // warp 8: MMA issue + tensor-memory allocation
constexpr int kMaxStages = 6;
constexpr int kChunkK = 64;                      // K elements per pipeline stage (128 bytes per row)
constexpr long long kSpinLimit = 1ll << 24;      // default limit of every wait, in mbarrier probes
constexpr size_t kPartialCap = (size_t)64 << 20; // bytes of fp32 partial tiles per contraction

__device__ __forceinline__ uint32_t smem_u32(const void *p) { return (uint32_t)__cvta_generic_to_shared(p); }
__device__ __forceinline__ void mbar_init(uint64_t *bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count) : "memory");
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
// Bounded wait: false after `limit` unsuccessful probes.
__device__ __forceinline__ bool mbar_wait(uint64_t *bar, uint32_t parity, long long limit) {
    for (long long i = 0; i < limit; ++i)
        if (mbar_try_wait(bar, parity)) return true;
    return false;
}
// The same for threads that have nothing urgent to do when the barrier completes (loader threads waiting for a free
// stage, epilogue threads waiting for the accumulators): they sleep between probes, so that the warps that issue the
// copies and the MMAs get the issue slots.  The limit counts probes all the same.
__device__ __forceinline__ bool mbar_wait_relaxed(uint64_t *bar, uint32_t parity, long long limit, unsigned ns) {
    for (long long i = 0; i < limit; ++i) {
        if (mbar_try_wait(bar, parity)) return true;
        __nanosleep(ns);
    }
    return false;
}
__device__ __forceinline__ void cp_async16(void *dst_smem, const void *src) {
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(smem_u32(dst_smem)), "l"(src) : "memory");
}
// Arrival that fires by itself once all cp.async copies this thread has issued so far have landed: the
// loader never blocks on its own copies, so every stage can be in flight and the producer side is
// decoupled from the consumer (counts as one of the barrier's expected arrivals).
__device__ __forceinline__ void cp_async_arrive_when_landed(uint64_t *bar) {
    asm volatile("cp.async.mbarrier.arrive.noinc.shared::cta.b64 [%0];" ::"r"(smem_u32(bar)) : "memory");
}
__device__ __forceinline__ void cp_async_wait_all() { asm volatile("cp.async.wait_all;" ::: "memory"); }
// Programmatic dependent launch: a kernel launched with the stream-serialization attribute may start
// while its predecessor in the stream still runs; pdl_wait() returns once the predecessor has
// finished and its writes are visible, pdl_launch() lets the successor start being scheduled.  Both
// are no-ops in launches without the attribute.
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void pdl_launch() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }
__device__ __forceinline__ void mbar_arrive_expect_tx(uint64_t *bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(bar)), "r"(bytes) : "memory");
}
// TMA: one 2-D tile of a dense 16-bit matrix (box = 64 columns x box rows, 128-byte swizzle) into shared
// memory; x = first column (a multiple of 64, i.e. of 128 bytes), y = first row; rows past the matrix
// read as zero.  Completion is counted in bytes on the mbarrier.
__device__ __forceinline__ void tma_load_tile(void *dst_smem, const CUtensorMap *map, int x, int y, uint64_t *bar) {
    asm volatile("cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
                 ::"r"(smem_u32(dst_smem)), "l"(map), "r"(x), "r"(y), "r"(smem_u32(bar)) : "memory");
}
// Ask for a tile to be brought into L2 (no shared-memory destination, no completion to wait for).
__device__ __forceinline__ void tma_prefetch_tile(const CUtensorMap *map, int x, int y) {
    asm volatile("cp.async.bulk.prefetch.tensor.2d.L2.global.tile [%0, {%1, %2}];" ::"l"(map), "r"(x), "r"(y) : "memory");
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

__device__ __forceinline__ uint32_t cluster_ctarank() {
    uint32_t r; asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r)); return r;
}
__device__ __forceinline__ void cluster_sync_all() {
    asm volatile("barrier.cluster.arrive.release.aligned;\n\tbarrier.cluster.wait.acquire.aligned;" ::: "memory");
}
// shared::cluster address of the same shared-memory location in CTA `rank` of the cluster
__device__ __forceinline__ uint32_t map_to_cta(uint32_t smem_addr, uint32_t rank) {
    uint32_t r; asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(smem_addr), "r"(rank)); return r;
}
// 16 bytes into the shared memory of a CTA of the cluster (address from map_to_cta)
__device__ __forceinline__ void st_cluster_v4(uint32_t cluster_addr, uint32_t a, uint32_t b, uint32_t c, uint32_t d) {
    asm volatile("st.shared::cluster.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(cluster_addr), "r"(a), "r"(b), "r"(c), "r"(d) : "memory");
}
// `bytes` (a multiple of 16) from this CTA's shared memory into the shared memory of another CTA of the cluster; completion
// is counted in bytes on an mbarrier of that CTA (both addresses from map_to_cta)
__device__ __forceinline__ void bulk_copy_to_cta(uint32_t dst_cluster, const void *src_smem, uint32_t bytes, uint32_t bar_cluster) {
    asm volatile("cp.async.bulk.shared::cluster.shared::cta.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                 ::"r"(dst_cluster), "r"(smem_u32(src_smem)), "r"(bytes), "r"(bar_cluster) : "memory");
}

// ------------------------------------------------------------------------------- parameters
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
    int n_split;                   // K splits = CTAs of the thread-block cluster that works on a tile
    int fmt;                       // 0 f16, 1 bf16
    int nstage;
    int32_t *status;
    const uint32_t *tokbits;       // [T][mask_words] slot bitmaps of the tokens' own lists, or nullptr: all tokens
    int mask_words;                //   use the whole union
    uint16_t *h_out;               // gate/up: H [t_pad_total][nu_pad]
    void *y;                       // down: output [T][d_model]
    int y_f32, residual;
    long long spin_limit;          // probes after which a wait gives up (SI_ERR_TIMEOUT)
    int withhold;                  // diagnostics: the first gate/up CTA never loads the X tile of its first chunk
    int pair_n;                    // (pair kernels) output columns of a pair's down tile: 128 or 256
};

// Tensor map of a dense row-major 16-bit matrix [rows][cols] for tiles of box_rows x 64 columns with the
// 128-byte swizzle the MMA descriptors expect.  base must be 16-byte aligned, row_bytes a multiple of 16.
inline int make_tile_map(CUtensorMap *map, const void *base, size_t cols, size_t rows, size_t row_bytes, int box_rows) {
    typedef CUresult (*encode_fn_t)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *,
                                    const cuuint64_t *, const cuuint32_t *, const cuuint32_t *, CUtensorMapInterleave,
                                    CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);
    static encode_fn_t encode = nullptr;
    if (!encode) {
        void *fn = nullptr;
        cudaDriverEntryPointQueryResult q;
        SI_CUDA_TRY(cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &q));
        if (!fn || q != cudaDriverEntryPointSuccess) return SI_ERR_CUDA;
        encode = (encode_fn_t)fn;
    }
    const cuuint64_t dims[2] = {(cuuint64_t)cols, (cuuint64_t)rows};
    const cuuint64_t strides[1] = {(cuuint64_t)row_bytes};
    const cuuint32_t box[2] = {(cuuint32_t)kChunkK, (cuuint32_t)box_rows};
    const cuuint32_t estr[2] = {1, 1};
    const CUresult r = encode(map, CU_TENSOR_MAP_DATA_TYPE_UINT16, 2, const_cast<void *>(base), dims, strides, box, estr,
                              CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
                              CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    return r == CUDA_SUCCESS ? SI_OK : SI_ERR_CUDA;
}

}  // namespace si_tc

// Kernel shapes of a call with more than 128 tokens (see si_pair_plan in si_gemm_pair.cu)
struct si_pair_plan_t {
    int gateup_w, gateup_sub, gateup_pairs;   // neurons per sub-tile, sub-tiles per tile, CTA pairs launched
    int down_n, down_ksplit, down_ctas;       // output columns per pair tile, pairs sharing a tile (K split), CTAs launched
};
void si_pair_plan(int d_model, int nu_pad, int T, int num_sms, si_pair_plan_t *plan);

// Contractions of calls with more than 128 tokens on pairs of SMs (si_gemm_pair.cu)
bool si_pair_path_applies(const si_store *s, int T);
int si_pair_contractions_launch(const si_store *s, si_tc::GemmParams P, int n_loaded, void *h_buf, size_t h_bytes, cudaStream_t stream);
