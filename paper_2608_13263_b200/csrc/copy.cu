// All-layer K+V gather-copy (the stage-aware asynchronous copy of Sec. 3.3.4): executes the
// inverse plan the planner left in the context.  Destination slots are consecutive inside
// each destination block (blocks are filled completely, Sec. 3.3.3), so every work item
// gathers scattered source rows into one contiguous destination range.
//
// Work decomposition: slab = (K|V, layer); item = `rows` consecutive destination slots of one
// destination block in one slab.  Items are ordered slab-major (all items of a slab before the
// next slab) so that the CTAs running at any moment touch one ~GB slab: TLB- and DRAM-page
// friendly over pools of tens of GB.  Persistent grid: item counts come from device memory.
//
// Two paths over the same decomposition:
//   register path : one warp per row, 16-byte loads (streaming hint) then 16-byte stores
//   bulk path     : per warp a ring of shared-memory stages; each lane issues one
//                   cp.async.bulk global->shared per source row (completion on an mbarrier),
//                   one lane issues a single cp.async.bulk shared->global for the whole
//                   contiguous destination range.  Every wait is bounded.
#include "common.cuh"

#include <cstdio>
#include <cstdlib>

namespace {

struct CopyArgs {
    uint8_t *k_pool, *v_pool;
    const int32_t *dst_src, *dst_blocks;
    vtoken_counts *counts;
    int64_t layer_stride, row_bytes;
    int32_t S, L, rows;        // rows per item (bulk path)
};

__device__ __forceinline__ uint8_t *slab_base(const CopyArgs &a, int slab)
{
    return (slab < a.L ? a.k_pool : a.v_pool) + (int64_t)(slab < a.L ? slab : slab - a.L) * a.layer_stride;
}

// ---- register path -----------------------------------------------------------------------
__device__ __forceinline__ uint4 ld_stream(const uint4 *p)
{
    uint4 v;
    asm volatile("ld.global.cs.v4.u32 {%0,%1,%2,%3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "l"(p));
    return v;
}
__device__ __forceinline__ void st_stream(uint4 *p, const uint4 &v)
{
    asm volatile("st.global.cs.v4.u32 [%0], {%1,%2,%3,%4};" ::"l"(p), "r"(v.x), "r"(v.y), "r"(v.z), "r"(v.w) : "memory");
}

constexpr int REG_NT = 256;
constexpr int REG_UNROLL = 4;   // 16-byte loads in flight per lane per row

__global__ void __launch_bounds__(REG_NT) copy_rows_kernel(CopyArgs a)
{
    const int nblk = a.counts->num_dst_blocks;
    const int64_t rows_per_slab = (int64_t)nblk * a.S;
    const int64_t total = rows_per_slab * 2 * a.L;
    const int lane = vtk_lane();
    const int64_t nwarps = (int64_t)gridDim.x * (REG_NT / 32);
    const int row_vecs = (int)(a.row_bytes >> 4);
    for (int64_t u = (int64_t)blockIdx.x * (REG_NT / 32) + (threadIdx.x >> 5); u < total; u += nwarps) {
        const int slab = (int)(u / rows_per_slab);
        const int64_t ds = u - (int64_t)slab * rows_per_slab;
        const int32_t src = a.dst_src[ds];
        if (src < 0) continue;
        const int j = (int)(ds / a.S);
        const int32_t blk = a.dst_blocks[j];
        if (blk < 0) continue;
        uint8_t *base = slab_base(a, slab);
        const uint4 *sp = reinterpret_cast<const uint4 *>(base + (int64_t)src * a.row_bytes);
        uint4 *dp = reinterpret_cast<uint4 *>(base + ((int64_t)blk * a.S + (ds - (int64_t)j * a.S)) * a.row_bytes);
        for (int c = lane; c < row_vecs; c += 32 * REG_UNROLL) {
            uint4 v[REG_UNROLL];
#pragma unroll
            for (int k = 0; k < REG_UNROLL; ++k)
                if (c + 32 * k < row_vecs) v[k] = ld_stream(sp + c + 32 * k);
#pragma unroll
            for (int k = 0; k < REG_UNROLL; ++k)
                if (c + 32 * k < row_vecs) st_stream(dp + c + 32 * k, v[k]);
        }
    }
}

// ---- bulk path ---------------------------------------------------------------------------
__device__ __forceinline__ uint32_t smem_u32(const void *p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint64_t *bar, uint32_t count)
{
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count));
}
__device__ __forceinline__ void mbar_expect_tx(uint64_t *bar, uint32_t bytes)
{
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(bar)), "r"(bytes) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint64_t *bar, uint32_t parity)
{
    uint32_t ok;
    asm volatile(
        "{\n .reg .pred p;\n mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n selp.u32 %0, 1, 0, p;\n}\n"
        : "=r"(ok) : "r"(smem_u32(bar)), "r"(parity) : "memory");
    return ok != 0;
}
__device__ __forceinline__ uint64_t global_ns()
{
    uint64_t t;
    asm volatile("mov.u64 %0, %globaltimer;" : "=l"(t));
    return t;
}
// Bounded wait: false when the phase did not complete within limit_ns (default two seconds).
__device__ __forceinline__ bool mbar_wait_bounded(uint64_t *bar, uint32_t parity, uint64_t limit_ns = 2000000000ull)
{
    if (mbar_try_wait(bar, parity)) return true;
    const uint64_t t0 = global_ns();
    for (;;) {
        for (int it = 0; it < 64; ++it)
            if (mbar_try_wait(bar, parity)) return true;
        if (global_ns() - t0 > limit_ns) return false;
    }
}
__device__ __forceinline__ void bulk_g2s(void *smem_dst, const void *gsrc, uint32_t bytes, uint64_t *bar)
{
    asm volatile("cp.async.bulk.shared::cta.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                 ::"r"(smem_u32(smem_dst)), "l"(gsrc), "r"(bytes), "r"(smem_u32(bar)) : "memory");
}
__device__ __forceinline__ void bulk_s2g(void *gdst, const void *smem_src, uint32_t bytes)
{
    asm volatile("cp.async.bulk.global.shared::cta.bulk_group [%0], [%1], %2;"
                 ::"l"(gdst), "r"(smem_u32(smem_src)), "r"(bytes) : "memory");
}
__device__ __forceinline__ void bulk_commit() { asm volatile("cp.async.bulk.commit_group;" ::: "memory"); }
template <int N>
__device__ __forceinline__ void bulk_wait_read() { asm volatile("cp.async.bulk.wait_group.read %0;" ::"n"(N) : "memory"); }
__device__ __forceinline__ void bulk_wait_all() { asm volatile("cp.async.bulk.wait_group 0;" ::: "memory"); }

constexpr int BULK_MAX_WARPS = 8;
constexpr int BULK_MAX_STAGES = 8;

// Each warp runs its own pipeline over its items.  At step k it (1) frees and refills the
// stage that item k+depth will use (its previous tenant is item k+depth-stages <= k-2, so at
// most the newest store group may still be reading shared memory), (2) waits for the rows of
// item k, (3) stores them with one bulk copy.
__global__ void __launch_bounds__(BULK_MAX_WARPS * 32) copy_bulk_kernel(CopyArgs a, int stages)
{
    extern __shared__ __align__(128) uint8_t smem[];
    __shared__ uint64_t bars[BULK_MAX_WARPS * BULK_MAX_STAGES];

    const int lane = vtk_lane(), warp = threadIdx.x >> 5, nwarps_cta = blockDim.x >> 5;
    const int rows = a.rows;
    const uint32_t row_bytes = (uint32_t)a.row_bytes;
    const uint32_t stage_bytes = rows * row_bytes;
    uint8_t *my_smem = smem + (size_t)warp * stages * stage_bytes;
    uint64_t *my_bars = bars + warp * BULK_MAX_STAGES;
    if (lane == 0) {
        for (int s = 0; s < stages; ++s) mbar_init(&my_bars[s], 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncwarp();

    const int nblk = a.counts->num_dst_blocks;
    const int parts = (a.S + rows - 1) / rows;                 // items per destination block
    const int64_t items_per_slab = (int64_t)nblk * parts;
    const int64_t total = items_per_slab * 2 * a.L;
    const int64_t gw = (int64_t)blockIdx.x * nwarps_cta + warp;
    const int64_t gstride = (int64_t)gridDim.x * nwarps_cta;
    const int depth = stages - 2;                              // items loading ahead of the one being stored
    bool timed_out = false;

    // issue the loads of this warp's k-th item into stage k % stages; returns nothing, the
    // store side recomputes the item's geometry
    auto issue = [&](int64_t k) {
        const int64_t it = gw + k * gstride;
        if (it >= total) return;
        const int s = (int)(k % stages);
        const int slab = (int)(it / items_per_slab);
        const int64_t rem = it - (int64_t)slab * items_per_slab;
        const int j = (int)(rem / parts), part = (int)(rem - (int64_t)j * parts);
        const int i0 = part * rows;
        const int nrows = min(rows, a.S - i0);
        const int32_t blk = a.dst_blocks[j];
        const uint8_t *base = slab_base(a, slab);
        uint8_t *stg = my_smem + (size_t)s * stage_bytes;
        // all store groups but the newest have finished reading shared memory
        bulk_wait_read<1>();
        __syncwarp();
        unsigned valid_total = 0;
        for (int i = lane; i < ((nrows + 31) & ~31); i += 32) {
            int32_t src = -1;
            if (i < nrows && blk >= 0) src = a.dst_src[(int64_t)j * a.S + i0 + i];
            valid_total += __popc(__ballot_sync(0xffffffffu, src >= 0));
        }
        if (lane == 0) mbar_expect_tx(&my_bars[s], valid_total * row_bytes);   // 0 rows: plain arrive
        __syncwarp();
        for (int i = lane; i < nrows; i += 32) {
            const int32_t src = blk >= 0 ? a.dst_src[(int64_t)j * a.S + i0 + i] : -1;
            if (src >= 0) bulk_g2s(stg + (size_t)i * row_bytes, base + (int64_t)src * a.row_bytes, row_bytes, &my_bars[s]);
        }
    };

    for (int64_t k = 0; k < depth; ++k) issue(k);
    for (int64_t k = 0;; ++k) {
        const int64_t it = gw + k * gstride;
        if (it >= total) break;
        issue(k + depth);
        const int s = (int)(k % stages);
        if (!mbar_wait_bounded(&my_bars[s], (uint32_t)((k / stages) & 1))) { timed_out = true; break; }
        const int slab = (int)(it / items_per_slab);
        const int64_t rem = it - (int64_t)slab * items_per_slab;
        const int j = (int)(rem / parts), part = (int)(rem - (int64_t)j * parts);
        const int i0 = part * rows;
        const int nrows = min(rows, a.S - i0);
        const int32_t blk = a.dst_blocks[j];
        if (blk >= 0) {
            uint8_t *base = slab_base(a, slab);
            uint8_t *stg = my_smem + (size_t)s * stage_bytes;
            uint8_t *dst = base + ((int64_t)blk * a.S + i0) * a.row_bytes;
            // valid rows normally form a prefix (only the tail of a request's last block is empty)
            int nvalid = 0;
            bool prefix = true;
            for (int i0w = 0; i0w < nrows; i0w += 32) {
                const int i = i0w + lane;
                const bool v = i < nrows && a.dst_src[(int64_t)j * a.S + i0 + i] >= 0;
                const unsigned m = __ballot_sync(0xffffffffu, v);
                const int cnt = __popc(m);
                if (m != (cnt == 32 ? 0xffffffffu : ((1u << cnt) - 1u))) prefix = false;   // a hole inside this group
                if (nvalid != i0w && cnt != 0) prefix = false;                             // a hole before this group
                nvalid += cnt;
            }
            if (prefix) {
                if (lane == 0 && nvalid > 0) bulk_s2g(dst, stg, (uint32_t)nvalid * row_bytes);
            } else {
                for (int i = lane; i < nrows; i += 32)
                    if (a.dst_src[(int64_t)j * a.S + i0 + i] >= 0)
                        bulk_s2g(dst + (size_t)i * row_bytes, stg + (size_t)i * row_bytes, row_bytes);
            }
        }
        bulk_commit();   // every lane commits (possibly empty) so group counts stay aligned
    }
    if (timed_out) {
        // give loads still in flight a bounded chance to land before shared memory is released
        for (int s = 0; s < stages; ++s) {
            mbar_wait_bounded(&my_bars[s], 0, 50000000ull);
            mbar_wait_bounded(&my_bars[s], 1, 50000000ull);
        }
        if (lane == 0) atomicOr(&a.counts->error_flags, VTOKEN_FLAG_TIMEOUT);
    }
    bulk_wait_all();
}

}  // namespace

// ---------------------------------------------------------------------------------------
int vtk_configure_copy(vtoken_ctx *ctx)
{
    const int S = ctx->cfg.block_size;
    int variant = ctx->cfg.copy_variant;
    if (const char *e = getenv("VTOKEN_COPY_VARIANT")) { if (variant == 0) variant = atoi(e); }
    // bulk copies need 16-byte multiples (checked at create) and a row that fits a stage
    if (variant == 0) variant = (ctx->row_bytes >= 512 && ctx->row_bytes <= 32768) ? 2 : 1;
    if (variant != 1 && variant != 2) return VTOKEN_EINVAL;

    int ctas_per_sm;
    if (variant == 1) {
        ctx->copy_threads = REG_NT;
        ctx->copy_smem = 0;
        ctas_per_sm = 8;
    } else {
        // tuning knobs: warps per CTA, ring depth, rows per item ("w,s,r"); defaults target
        // about 192 KB of staging per SM
        int warps = 4, stages = 3, rows = 0;
        if (const char *e = getenv("VTOKEN_BULK_TUNE")) sscanf(e, "%d,%d,%d", &warps, &stages, &rows);
        if (rows <= 0) {
            rows = S;
            while (rows > 1 && (int64_t)rows * ctx->row_bytes > 16384) rows = (rows + 1) / 2;
        }
        if (rows > S) rows = S;
        if (warps < 1) warps = 1;
        if (warps > BULK_MAX_WARPS) warps = BULK_MAX_WARPS;
        if (stages < 3) stages = 3;
        if (stages > BULK_MAX_STAGES) stages = BULK_MAX_STAGES;
        int64_t smem = (int64_t)warps * stages * rows * ctx->row_bytes;
        while (smem > 200 * 1024 && warps > 1) { --warps; smem = (int64_t)warps * stages * rows * ctx->row_bytes; }
        while (smem > 200 * 1024 && stages > 3) { --stages; smem = (int64_t)warps * stages * rows * ctx->row_bytes; }
        if (smem > 200 * 1024) return VTOKEN_EINVAL;
        ctx->bulk_warps = warps;
        ctx->bulk_stages = stages;
        ctx->bulk_rows = rows;
        ctx->copy_threads = warps * 32;
        ctx->copy_smem = (int)smem;
        VTK_CUDA(ctx, cudaFuncSetAttribute(copy_bulk_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
        ctas_per_sm = (int)((220 * 1024) / (smem + 1024));
        if (ctas_per_sm < 1) ctas_per_sm = 1;
        if (ctas_per_sm > 8) ctas_per_sm = 8;
    }
    int ctas = ctx->num_sms * ctas_per_sm;
    if (const char *e = getenv("VTOKEN_COPY_CTAS")) { int v = atoi(e); if (v > 0) ctas = v; }
    if (ctx->cfg.max_ctas > 0 && ctas > ctx->cfg.max_ctas) ctas = ctx->cfg.max_ctas;
    ctx->copy_ctas = ctas;
    ctx->copy_variant = variant;
    return VTOKEN_OK;
}

int vtk_launch_copy(vtoken_ctx *ctx, cudaStream_t st)
{
    CopyArgs a;
    a.k_pool = (uint8_t *)ctx->cfg.k_pool;
    a.v_pool = (uint8_t *)ctx->cfg.v_pool;
    a.dst_src = ctx->dst_src;
    a.dst_blocks = ctx->dst_blocks;
    a.counts = ctx->counts;
    a.layer_stride = ctx->layer_stride;
    a.row_bytes = ctx->row_bytes;
    a.S = ctx->cfg.block_size;
    a.L = ctx->cfg.num_layers;
    a.rows = ctx->bulk_rows;
    if (ctx->copy_variant == 1)
        copy_rows_kernel<<<ctx->copy_ctas, ctx->copy_threads, 0, st>>>(a);
    else
        copy_bulk_kernel<<<ctx->copy_ctas, ctx->copy_threads, ctx->copy_smem, st>>>(a, ctx->bulk_stages);
    VTK_CUDA(ctx, cudaGetLastError());
    return VTOKEN_OK;
}
