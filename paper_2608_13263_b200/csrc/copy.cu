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


namespace {

struct CopyArgs {
    uint8_t *k_pool, *v_pool;
    vtk_arr<const int32_t> dst_src, dst_blocks;
    vtk_arr<vtoken_counts> counts;
    int64_t layer_stride, row_bytes;
    int64_t slots_per_layer;   // rows of a slab (the checked build refuses a row outside)
    int32_t S, L, rows;        // rows per item (bulk path)
    int64_t wait_limit_ns;     // bound of every wait on a shared-memory barrier (bulk path)
    int64_t stall_item;        // -1, or the global index of one item whose barrier is armed with bytes that
                               // never arrive: exercises the time-out path without faulting anything
    unsigned int *ticket;      // dynamic item distribution: [0] next item index, [1] warps that have finished
    // gather mode (logical view): rows g_src[0 .. *g_total) of layers [layer_begin, layer_begin + L) go to the
    // dense buffers out_k / out_v, [L][out_capacity][row_bytes]
    vtk_arr<const int32_t> g_src, g_total;
    uint8_t *out_k, *out_v;
    int64_t out_capacity;
    int32_t layer_begin;
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
    vtk_wait_for_predecessor();            // the plan is the previous kernel's output
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
#ifdef VTOKEN_CHECKED
        if ((int64_t)src >= a.slots_per_layer || ((int64_t)blk + 1) * a.S > a.slots_per_layer) {
            atomicOr(&a.counts->error_flags, (uint32_t)VTOKEN_FLAG_CHECK_FAILED);     // a row outside its slab: skipped
            continue;
        }
#endif
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
// at most n (1..10) of this thread's newest store groups may still be reading shared memory
__device__ __forceinline__ void bulk_wait_read_n(int n)
{
    switch (n) {
        case 1: bulk_wait_read<1>(); break;
        case 2: bulk_wait_read<2>(); break;
        case 3: bulk_wait_read<3>(); break;
        case 4: bulk_wait_read<4>(); break;
        case 5: bulk_wait_read<5>(); break;
        case 6: bulk_wait_read<6>(); break;
        case 7: bulk_wait_read<7>(); break;
        case 8: bulk_wait_read<8>(); break;
        case 9: bulk_wait_read<9>(); break;
        default: bulk_wait_read<10>(); break;
    }
}
// every bulk store of this thread has read its shared-memory source (the global writes complete with the kernel)
__device__ __forceinline__ void bulk_wait_all_read() { asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory"); }

constexpr int TAIL_ITEMS_PER_WARP = 2;      // items per warp that are handed out singly at the end of a launch
constexpr int BULK_MAX_WARPS = 16;
constexpr int BULK_MAX_STAGES = 12;
constexpr int BULK_MAX_SMEM = 216 * 1024;   // dynamic shared memory cap: leaves room for the static barrier arrays

// Each warp runs its own pipeline through a ring of `stages` shared-memory buffers.
//
// Work: an item is `rows` consecutive destination slots of one destination block in one slab
// (rows is a power of two that divides S, so its destination is one contiguous byte range).
// Items are numbered slab-major and handed to the warps of the grid in that order (by a ticket
// counter, see DYNAMIC below, or round-robin): at any moment the grid works on a window of
// consecutive items, i.e. on one contiguous destination range of a few MB, which keeps DRAM
// pages and TLB entries hot on the write side.
//
// Step k of a warp's pipeline: (1) free and refill the stage that item k+depth will use -- its
// previous tenant is item k+depth-stages = k-(w+1), w = stages-depth-1, so the w newest store
// groups may still be reading shared memory; each lane issues one cp.async.bulk global->shared
// for its source row, completion bytes counted on the stage's mbarrier -- (2) wait for the rows
// of item k (bounded), (3) one lane stores them with a single cp.async.bulk shared->global.
//
// Nothing on that path waits for a global-memory read of the plan: the entries of an item
// (destination block id, source slot of the lane's row) are fetched `ahead` (1 or 2) items
// early into registers, what the store side needs (destination address, valid-row mask) is
// parked in shared memory at issue time, and item indices advance by additions (no per-step
// division).  `ahead` is a run-time argument on purpose: measured on B200, the build in which
// it is a compile-time constant schedules the issue path 2-3 % slower (6.20 vs 6.32 TB/s on the
// Llama-shaped workload, same box, alternating runs).
//
// DYNAMIC: instead of its fixed share (items gw, gw + gstride, ...) a warp takes the next
// `chunk` consecutive items from a global ticket counter.  SMs do not all move bytes at the same
// rate: an in-kernel timeline on B200 showed the median warp at 6.8 TB/s-equivalent throughout
// while the slowest SM finished 80-190 us after the median one, whatever the kernel's length, so
// fixed shares leave most of the GPU idle at the end of every launch (3.7 % of a 1.35 ms launch,
// 8 % of a 0.7 ms one).  Tickets keep the property that the grid works on one contiguous window
// of items, and they absorb row-less tail items as well.  One atomic per item caps the kernel at
// the throughput of same-address atomics (3.2 TB/s on the largest workload); one per 4 items is
// free.  A chunk's ticket is requested a whole chunk before it is used, so its round trip is off
// the critical path; the last warp to finish resets the counters for the next launch.
//
// GATHER: the same machinery writes the logical view instead of executing a plan: an item is
// `rows` consecutive rows of the dense output, its sources are the slots g_src names, and the
// destination lies in another buffer than the source.  (Always with tickets.)
template <bool DYNAMIC, bool GATHER>
__global__ void __launch_bounds__(BULK_MAX_WARPS * 32) copy_bulk_kernel(CopyArgs a, int stages, int depth, int ahead,
                                                                        int chunk)
{
    extern __shared__ __align__(128) uint8_t smem[];
    __shared__ uint64_t bars[BULK_MAX_WARPS * BULK_MAX_STAGES];
    __shared__ uint64_t park_dst[BULK_MAX_WARPS * BULK_MAX_STAGES];    // destination address of the staged item
    __shared__ uint32_t park_mask[BULK_MAX_WARPS * BULK_MAX_STAGES];   // which of its rows are valid

    const int lane = vtk_lane(), warp = threadIdx.x >> 5, nwarps_cta = blockDim.x >> 5;
    const int rows = a.rows;                                   // power of two, divides S, <= 32
    const int S = a.S;
    const uint32_t row_bytes = (uint32_t)a.row_bytes;
    const uint32_t stage_bytes = rows * row_bytes;
    uint8_t *my_smem = smem + (size_t)warp * stages * stage_bytes;
    uint64_t *my_bars = bars + warp * BULK_MAX_STAGES;
    uint64_t *my_dst = park_dst + warp * BULK_MAX_STAGES;
    uint32_t *my_mask = park_mask + warp * BULK_MAX_STAGES;
    if (lane == 0) {
        for (int s = 0; s < stages; ++s) mbar_init(&my_bars[s], 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncwarp();
    // everything above overlaps the tail of the previous kernel in the stream (normally the
    // planner); its output -- counts, inverse plan -- and the pools are touched only below
    vtk_wait_for_predecessor();

    const int parts = S / rows;                                // items per destination block
    const int g_n = GATHER ? *a.g_total : 0;                   // gather: output rows per slab
    // items per slab, < 2^31 (checked on the host)
    const int per_slab = GATHER ? (g_n + rows - 1) / rows : a.counts->num_dst_blocks * parts;
    const int num_slabs = 2 * a.L;
    const int64_t gw = (int64_t)blockIdx.x * nwarps_cta + warp;
    const int64_t gstride = (int64_t)gridDim.x * nwarps_cta;
    const int stores_in_flight = stages - depth - 1;

    // cursors over this warp's items (gw, gw + gstride, ...) as (slab, item inside the slab)
    struct Cursor { int slab, rem; };
    const int step_slabs = per_slab > 0 ? (int)(gstride / per_slab) : 0;
    const int step_rem = per_slab > 0 ? (int)(gstride % per_slab) : 0;
    Cursor c_fetch;
    c_fetch.slab = per_slab > 0 ? (int)min((int64_t)num_slabs, gw / per_slab) : num_slabs;
    c_fetch.rem = per_slab > 0 ? (int)(gw % per_slab) : 0;

    // plan entries of the next two items to issue: slab, destination slot of the first row
    // (-1: skip the item), source slot of this lane's row (-1: no row)
    struct Entry { int slab; int32_t dst0, src; unsigned idx; };
    Entry e1, e2;
    const unsigned total_items = (unsigned)per_slab * (unsigned)num_slabs;   // < 2^31, checked on the host
    // DYNAMIC: a ticket stands for `chunk` consecutive items (one atomic per chunk keeps the counter
    // far from the throughput of same-address atomics); lane 0 holds the ticket of the NEXT chunk
    // A warp's first chunk is the one with its own index in the grid, without an atomic: 1184 warps asking
    // one address for a ticket at the same instant are served one after the other (about 3 us until the
    // last one has its answer), and nothing can start before.  The counter hands out the chunks behind
    // those (its value + number of warps); those requests are made a chunk ahead, off the critical path.
    // The last items of a launch are handed out one per ticket: with a whole chunk per ticket to the end the
    // warps would finish up to a chunk (about 3 us of a warp's time) apart, which a launch of tens of
    // microseconds feels.  Tickets below n_big stand for `chunk` items, the ones behind them for one item.
    const unsigned tail_items = min(total_items, (unsigned)gstride * (unsigned)TAIL_ITEMS_PER_WARP);
    const unsigned n_big = (total_items - tail_items) / (unsigned)chunk;
    const unsigned big_items = n_big * (unsigned)chunk;
    unsigned ticket = (unsigned)gw, chunk_base = 0, chunk_len = 0, chunk_pos = 0;
    unsigned finished_rank = 0xffffffffu;       // lane 0: how many warps had run out of tickets before this one
    bool exhausted = false;
    auto take_ticket = [&]() { if (lane == 0) ticket = atomicAdd(&a.ticket[0], 1u) + (unsigned)gstride; };
    auto fetch = [&](Entry &e) {           // reads the next item of this warp, moves on
        e.dst0 = -1;
        e.src = -1;
        e.idx = 0;
        if (DYNAMIC) {
            if (chunk_pos == chunk_len && !exhausted) {     // next chunk: its ticket was requested a chunk ago
                const unsigned t = __shfl_sync(0xffffffffu, ticket, 0);
                if (t < n_big) {
                    chunk_base = t * (unsigned)chunk;
                    chunk_len = (unsigned)chunk;
                } else {
                    const unsigned single = t - n_big;
                    chunk_base = single < total_items - big_items ? big_items + single : 0x7fffffffu;
                    chunk_len = 1;
                }
                chunk_pos = 0;
                if (chunk_base < total_items) {
                    take_ticket();
                } else {
                    // out of tickets: say so now, while this warp's last items are still in flight, so that the
                    // counters are back at zero by the time the last warp leaves (see the end of the kernel)
                    exhausted = true;
                    if (lane == 0) finished_rank = atomicAdd(&a.ticket[1], 1u);
                }
            }
            const unsigned i = exhausted ? 0x7fffffffu : chunk_base + chunk_pos;
            ++chunk_pos;
            e.slab = num_slabs;
            if (i < total_items) {
                const unsigned slab = i / (unsigned)per_slab, rem = i - slab * (unsigned)per_slab;
                if (GATHER) {
                    const int i0 = (int)rem * rows;                 // first output row of the item
                    if (lane < rows && i0 + lane < g_n) e.src = a.g_src[i0 + lane];
                    e.dst0 = i0;
                } else {
                    const int j = (int)(rem / (unsigned)parts);
                    const int i0 = ((int)rem - j * parts) * rows;
                    const int32_t blk = a.dst_blocks[j];
                    if (lane < rows) e.src = a.dst_src[(int64_t)j * S + i0 + lane];
                    e.dst0 = blk >= 0 ? blk * S + i0 : -1;
                }
                e.slab = (int)slab;
                e.idx = i;
            }
        } else {
            e.slab = c_fetch.slab;
            if (c_fetch.slab < num_slabs) {
                const int j = (int)((unsigned)c_fetch.rem / (unsigned)parts);
                const int i0 = (c_fetch.rem - j * parts) * rows;
                const int32_t blk = a.dst_blocks[j];
                if (lane < rows) e.src = a.dst_src[(int64_t)j * S + i0 + lane];
                e.dst0 = blk >= 0 ? blk * S + i0 : -1;
                c_fetch.slab += step_slabs;
                c_fetch.rem += step_rem;
                if (c_fetch.rem >= per_slab) { c_fetch.rem -= per_slab; ++c_fetch.slab; }
            }
        }
    };
    fetch(e1);
    if (ahead == 2) fetch(e2);

    int s_issue = 0, issued = 0, stored = 0;
    int stall_countdown = -1;                  // issues left before the item named by the test hook
    if (a.stall_item >= gw && (a.stall_item - gw) % gstride == 0 && (a.stall_item - gw) / gstride < (1 << 30))
        stall_countdown = (int)((a.stall_item - gw) / gstride);
    auto issue = [&]() {
        if (e1.slab >= num_slabs) return;
        const int s = s_issue;
        s_issue = s_issue + 1 == stages ? 0 : s_issue + 1;
        const Entry e = e1;
        if (ahead == 2) {
            e1 = e2;
            fetch(e2);                               // in flight for two steps before it is used
        } else {
            fetch(e1);                               // in flight for one step
        }
        bool valid = e.src >= 0 && e.dst0 >= 0;
#ifdef VTOKEN_CHECKED
        // a source row outside its slab, or a destination range outside the slab / the output buffer: skipped
        if (valid && ((int64_t)e.src >= a.slots_per_layer ||
                      (int64_t)e.dst0 + lane >= (GATHER ? a.out_capacity : a.slots_per_layer))) {
            atomicOr(&a.counts->error_flags, (uint32_t)VTOKEN_FLAG_CHECK_FAILED);
            valid = false;
        }
#endif
        uint8_t *base, *dst_base;
        if (GATHER) {
            const int li = e.slab < a.L ? e.slab : e.slab - a.L;
            base = (e.slab < a.L ? a.k_pool : a.v_pool) + (int64_t)(a.layer_begin + li) * a.layer_stride;
            dst_base = (e.slab < a.L ? a.out_k : a.out_v) + (int64_t)li * a.out_capacity * a.row_bytes;
        } else {
            base = slab_base(a, e.slab);
            dst_base = base;
        }
        uint8_t *stg = my_smem + (size_t)s * stage_bytes;
        bulk_wait_read_n(stores_in_flight);          // the stage's previous store has read its bytes
        const unsigned mask = __ballot_sync(0xffffffffu, valid);
        if (lane == 0) {
            my_mask[s] = mask;
            my_dst[s] = (uint64_t)(dst_base + (int64_t)e.dst0 * a.row_bytes);
            const uint32_t phantom = (DYNAMIC ? (a.stall_item >= 0 && (int64_t)e.idx == a.stall_item)
                                              : stall_countdown == 0) ? 16u : 0u;
            mbar_expect_tx(&my_bars[s], (uint32_t)__popc(mask) * row_bytes + phantom);   // no rows: plain arrive
        }
        __syncwarp();
        if (valid) bulk_g2s(stg + (size_t)lane * row_bytes, base + (int64_t)e.src * a.row_bytes, row_bytes, &my_bars[s]);
        ++issued;
        --stall_countdown;
    };

    bool timed_out = false;
    for (int k = 0; k < depth; ++k) issue();
    int s = 0;
    uint32_t parity = 0;
    for (;;) {
        issue();
        if (stored == issued) break;
        if (!mbar_wait_bounded(&my_bars[s], parity, (uint64_t)a.wait_limit_ns)) { timed_out = true; break; }
        const unsigned mask = my_mask[s];
        if (mask != 0) {
            uint8_t *stg = my_smem + (size_t)s * stage_bytes;
            uint8_t *dst = (uint8_t *)my_dst[s];
            const int nvalid = __popc(mask);
            // valid rows normally form a prefix (only the tail of a request's last block is empty)
            if (mask == (nvalid == 32 ? 0xffffffffu : ((1u << nvalid) - 1u))) {
                if (lane == 0) bulk_s2g(dst, stg, (uint32_t)nvalid * row_bytes);
            } else if ((mask >> lane) & 1u) {
                bulk_s2g(dst + (size_t)lane * row_bytes, stg + (size_t)lane * row_bytes, row_bytes);
            }
        }
        bulk_commit();   // every lane commits (possibly empty) so group counts stay aligned
        ++stored;
        if (++s == stages) { s = 0; parity ^= 1u; }
    }
    if (timed_out) {
        // give loads still in flight a bounded chance to land before shared memory is released
        for (int q = 0; q < stages; ++q) {
            mbar_wait_bounded(&my_bars[q], 0, 50000000ull);
            mbar_wait_bounded(&my_bars[q], 1, 50000000ull);
        }
        if (lane == 0) atomicOr(&a.counts->error_flags, VTOKEN_FLAG_TIMEOUT);
    }
    bulk_wait_all_read();
    if (DYNAMIC && lane == 0) {
        // the last warp of the grid to run out of tickets puts the counters back for the next launch: every
        // other warp has stopped taking tickets by then.  (A warp that timed out may not have run out: it
        // reports in here, so that the count is complete either way.)
        if (finished_rank == 0xffffffffu) finished_rank = atomicAdd(&a.ticket[1], 1u);
        if (finished_rank == (unsigned)gstride - 1u) {
            a.ticket[0] = 0u;
            a.ticket[1] = 0u;
        }
    }
}

}  // namespace

// ---------------------------------------------------------------------------------------
int vtk_configure_copy(vtoken_ctx *ctx)
{
    const int S = ctx->cfg.block_size;
    const vtoken_copy_tuning &tune = ctx->cfg.tuning;
    const bool tuned = tune.enabled != 0;
    int variant = ctx->cfg.copy_variant;
    // bulk copies need 16-byte multiples (checked at create) and a row that fits a stage.  Small rows
    // belong on the bulk path too: the register path spends a warp per row whatever its size (measured
    // on B200 with 256 / 128 / 64 / 16-byte rows: 2.0 / 1.0 / 0.5 / 0.14 TB/s against 6.1 / 4.6 / 2.6 /
    // 0.3 TB/s through the rings, where an item is up to 32 rows)
    if (variant == 0) variant = ctx->row_bytes <= 32768 ? 2 : 1;
    if (variant != 1 && variant != 2) return VTOKEN_EINVAL;
    if (ctx->cfg.wait_limit_ms < 0 || ctx->cfg.wait_limit_ms > 60000) return VTOKEN_EINVAL;
    ctx->wait_limit_ns = ctx->cfg.wait_limit_ms ? (int64_t)ctx->cfg.wait_limit_ms * 1000000ll : 2000000000ll;
    ctx->stall_item = -1;
#ifdef VTOKEN_CHECKED
    if (ctx->cfg.debug_stall_item > 0) ctx->stall_item = ctx->cfg.debug_stall_item - 1;
#else
    if (ctx->cfg.debug_stall_item != 0) return VTOKEN_EINVAL;      // the hook exists in the checked build only
#endif

    int ctas_per_sm;
    if (variant == 1) {
        ctx->copy_threads = REG_NT;
        ctx->copy_smem = 0;
        ctas_per_sm = 8;
    } else {
        // Launch shape: warps per CTA, ring stages per warp, rows per item, items loading ahead of the one
        // being stored, plan entries fetched ahead.  Default: 8 warps x 4 stages x 4 KiB items = 128 KiB of
        // staging per SM, two items loading ahead, one store in flight per warp.  Measured on B200: alone,
        // shapes from 96 to 192 KiB per SM and from 4 to 32 KiB per item land within a few per cent of each
        // other; below 4 KiB per warp-step with only 8 warps per SM the pipeline becomes issue-bound; beside a
        // bandwidth-bound kernel the ring size decides how the two share HBM (see common.cuh).
        int warps = VTK_DEFAULT_WARPS, stages = VTK_DEFAULT_STAGES, rows = 0, depth = 2, ahead = 2;
        if (tuned) {
            if (tune.warps > 0) warps = tune.warps;
            if (tune.stages > 0) stages = tune.stages;
            rows = tune.rows;
            depth = tune.depth;
            ahead = tune.ahead;
        }
        ctx->bulk_ahead = ahead == 1 ? 1 : 2;
        if (rows <= 0) rows = (int)(4096 / ctx->row_bytes);
        // an item is `rows` consecutive destination slots inside one block: a power of two
        // (<= 32, one row per lane) that divides the block size
        {
            int r = 1;
            while (r * 2 <= rows && r * 2 <= 32 && S % (r * 2) == 0) r *= 2;
            rows = r;
        }
        if (warps < 1) warps = 1;
        if (warps > BULK_MAX_WARPS) warps = BULK_MAX_WARPS;
        if (stages < 2) stages = 2;
        if (stages > BULK_MAX_STAGES) stages = BULK_MAX_STAGES;
        int64_t smem = (int64_t)warps * stages * rows * ctx->row_bytes;
        while (smem > BULK_MAX_SMEM && warps > 1) { --warps; smem = (int64_t)warps * stages * rows * ctx->row_bytes; }
        while (smem > BULK_MAX_SMEM && stages > 2) { --stages; smem = (int64_t)warps * stages * rows * ctx->row_bytes; }
        if (smem > BULK_MAX_SMEM) return VTOKEN_EINVAL;
        if (depth < 0) depth = 0;
        if (depth > stages - 2) depth = stages - 2;
        // the kernel indexes the items of a slab with 32-bit integers
        if ((int64_t)ctx->cap_dst_blocks * (S / rows) >= (int64_t)INT32_MAX) return VTOKEN_EINVAL;
        ctx->bulk_depth = depth;
        ctx->bulk_warps = warps;
        ctx->bulk_stages = stages;
        ctx->bulk_rows = rows;
        ctx->copy_threads = warps * 32;
        ctx->copy_smem = (int)smem;
        VTK_CUDA(ctx, cudaFuncSetAttribute(copy_bulk_kernel<false, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, BULK_MAX_SMEM));
        VTK_CUDA(ctx, cudaFuncSetAttribute(copy_bulk_kernel<true, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, BULK_MAX_SMEM));
        VTK_CUDA(ctx, cudaFuncSetAttribute(copy_bulk_kernel<true, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, BULK_MAX_SMEM));
        // tickets are 32-bit: every item of a launch must have an index below 2^31
        ctx->copy_dynamic = (int64_t)ctx->cap_dst_blocks * (S / rows) * 2 * ctx->cfg.num_layers < (int64_t)INT32_MAX;
        if (tuned && tune.fixed_shares) ctx->copy_dynamic = false;
        // one ticket per >= 16 KiB of destination bytes and never fewer than 4 items: measured on B200, one
        // ticket per 8 KiB already runs into the throughput of atomics on one address (4.5 instead of 6.7 TB/s)
        {
            const int64_t item_bytes = (int64_t)rows * ctx->row_bytes;
            int64_t c = (16384 + item_bytes - 1) / item_bytes;
            ctx->copy_chunk = (int)(c < 4 ? 4 : (c > 64 ? 64 : c));
        }
        if (tuned && tune.chunk >= 1 && tune.chunk <= 1024) ctx->copy_chunk = tune.chunk;
        ctas_per_sm = (int)((227 * 1024) / (smem + 2048));
        if (ctas_per_sm < 1) ctas_per_sm = 1;
        if (ctas_per_sm > 8) ctas_per_sm = 8;
    }
    int ctas = ctx->num_sms * ctas_per_sm;
    if (tuned && tune.ctas > 0) ctas = tune.ctas;
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
    a.dst_src = VTK_ARR(ctx, (const int32_t *)ctx->dst_src, (int64_t)ctx->cap_dst_blocks * ctx->cfg.block_size);
    a.dst_blocks = VTK_ARR(ctx, (const int32_t *)ctx->dst_blocks, ctx->cap_dst_blocks);
    a.counts = VTK_ARR(ctx, ctx->counts, 1);
    a.layer_stride = ctx->layer_stride;
    a.row_bytes = ctx->row_bytes;
    a.slots_per_layer = ctx->slots_per_layer;
    a.S = ctx->cfg.block_size;
    a.L = ctx->cfg.num_layers;
    a.rows = ctx->bulk_rows;
    a.wait_limit_ns = ctx->wait_limit_ns;
    a.stall_item = ctx->stall_item;
    a.ticket = ctx->copy_ticket;
    const dim3 grid(ctx->copy_ctas), block(ctx->copy_threads);
    if (ctx->copy_variant == 1)
        VTK_CUDA(ctx, vtk_launch_dependent(ctx, copy_rows_kernel, grid, block, 0, st, a));
    else if (ctx->copy_dynamic)
        VTK_CUDA(ctx, vtk_launch_dependent(ctx, copy_bulk_kernel<true, false>, grid, block, (size_t)ctx->copy_smem, st, a,
                                           ctx->bulk_stages, ctx->bulk_depth, ctx->bulk_ahead, ctx->copy_chunk));
    else
        VTK_CUDA(ctx, vtk_launch_dependent(ctx, copy_bulk_kernel<false, false>, grid, block, (size_t)ctx->copy_smem, st, a,
                                           ctx->bulk_stages, ctx->bulk_depth, ctx->bulk_ahead, 1));
    VTK_CUDA(ctx, cudaGetLastError());
    return VTOKEN_OK;
}

// The row copy of vtoken_gather_logical through the bulk path.  Returns 1 when the kernel was launched,
// 0 when the context has no bulk configuration for these rows (the caller uses its register kernel),
// VTOKEN_ECUDA when the launch failed (the CUDA error is kept in the context).
int vtk_launch_gather_bulk(vtoken_ctx *ctx, const int32_t *g_src, const int32_t *g_total, int32_t layer_begin,
                            int32_t layer_end, void *out_k, void *out_v, int64_t out_capacity, cudaStream_t st)
{
    if (ctx->copy_variant != 2 || !ctx->copy_dynamic || ctx->g_ticket == nullptr) return 0;
    // tickets are 32-bit: every item must have an index below 2^31
    const int64_t items = (ctx->cfg.max_tokens + ctx->bulk_rows - 1) / ctx->bulk_rows * 2 * (layer_end - layer_begin);
    if (items >= (int64_t)INT32_MAX) return 0;
    CopyArgs a;
    a.k_pool = (uint8_t *)ctx->cfg.k_pool;
    a.v_pool = (uint8_t *)ctx->cfg.v_pool;
    a.dst_src = vtk_arr<const int32_t>();
    a.dst_blocks = vtk_arr<const int32_t>();
    a.counts = VTK_ARR(ctx, ctx->rt_counts, 1);   // gather mode reads no count from it: only the time-out flag goes there
    a.layer_stride = ctx->layer_stride;
    a.row_bytes = ctx->row_bytes;
    a.slots_per_layer = ctx->slots_per_layer;
    a.S = ctx->bulk_rows;                 // parts = 1: unused in gather mode
    a.L = layer_end - layer_begin;
    a.rows = ctx->bulk_rows;
    a.wait_limit_ns = ctx->wait_limit_ns;
    a.stall_item = -1;
    a.ticket = ctx->g_ticket;
    a.g_src = VTK_ARR(ctx, g_src, ctx->cfg.max_tokens);
    a.g_total = VTK_ARR(ctx, g_total, 1);
    a.out_k = (uint8_t *)out_k;
    a.out_v = (uint8_t *)out_v;
    a.out_capacity = out_capacity;
    a.layer_begin = layer_begin;
    VTK_CUDA(ctx, vtk_launch_dependent(ctx, copy_bulk_kernel<true, true>, dim3(ctx->copy_ctas), dim3(ctx->copy_threads),
                                       (size_t)ctx->copy_smem, st, a, ctx->bulk_stages, ctx->bulk_depth, ctx->bulk_ahead,
                                       ctx->copy_chunk));
    return 1;
}
