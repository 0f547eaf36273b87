// Repack in waves: plan -> copy -> commit, num_waves times on one stream, where the commit of a
// wave hands the blocks it reclaimed to the pool of the next wave (the paper frees sources after
// the packed layout is committed, Sec. 3.3.4, and defers what the headroom cannot serve,
// Sec. 3.3.2).  Tables and pools ping-pong between the caller's outputs and the workspace so
// that the last wave writes the caller's buffers.  Stream order is the only synchronisation:
// wave k+1 may overwrite blocks wave k has read because its copy kernel runs after wave k's.
#include "common.cuh"

namespace {

constexpr int COMMIT_NT = 256;

struct CommitArgs {
    const int32_t *num_requests;
    int32_t max_requests, wave;
    const int32_t *status_k;          // statuses of this wave
    int32_t *req_status, *req_wave;   // merged over the waves so far
    int32_t *req_append_pos;          // or NULL
    const int32_t *moved;             // tokens this wave moves per request (planner scratch)
    const int32_t *new_bt_offsets;    // block tables this wave proposes
    int32_t S;
    const int32_t *pool, *num_pool;   // P_k and its size
    const int32_t *freed;             // blocks reclaimed by this wave
    vtoken_counts *wave_counts;       // counts of this wave (written by the planner)
    const vtoken_counts *ctx_counts;  // the context's copy: carries the flags raised by the copy kernel
    int32_t *pool_next, *num_pool_next;
    int32_t free_capacity;
    // references dropped by copy-on-write detaches: this wave's list goes behind those of the waves before it
    const int32_t *released_k;        // or NULL
    const vtoken_counts *all_counts;  // counts of the waves so far ([wave + 1])
    int32_t *released_out, *num_released_out;
    int64_t released_capacity;
    int32_t last;                     // 1: the last wave (writes the total)
};

__global__ void __launch_bounds__(COMMIT_NT) wave_commit_kernel(CommitArgs a)
{
    vtk_release_successor();
    vtk_wait_for_predecessor();
    const int gtid = blockIdx.x * COMMIT_NT + threadIdx.x, gsz = gridDim.x * COMMIT_NT;
    int R = *a.num_requests;
    R = R < 0 ? 0 : (R > a.max_requests ? a.max_requests : R);
    for (int r = gtid; r < R; r += gsz) {
        const int s = a.status_k[r];
        if (s == VTOKEN_REPACKED) {
            a.req_status[r] = VTOKEN_REPACKED;
            a.req_wave[r] = a.wave;
            if (a.req_append_pos) {
                // behind the tokens this wave moved: they fill its destination blocks at the end of the list
                const int m = a.moved[r], blocks = a.new_bt_offsets[r + 1] - a.new_bt_offsets[r];
                a.req_append_pos[r] = (blocks - (m + a.S - 1) / a.S) * a.S + m;
            }
        } else if (a.wave == 0) {
            a.req_status[r] = s;
            a.req_wave[r] = -1;
            if (a.req_append_pos) a.req_append_pos[r] = -1;
        } else if (a.req_status[r] != VTOKEN_REPACKED) {
            a.req_status[r] = s;
        }
    }
    // next pool = unconsumed part of this pool (same order) ++ reclaimed blocks (reclaim order)
    int np = *a.num_pool;
    bool over = np > a.free_capacity;
    np = np < 0 ? 0 : (over ? a.free_capacity : np);
    int consumed = a.wave_counts->num_free_consumed;
    consumed = consumed < 0 ? 0 : (consumed > np ? np : consumed);
    const int rest = np - consumed;
    const int nfreed = a.wave_counts->num_freed;
    long long total = (long long)rest + nfreed;
    if (total > a.free_capacity) {
        over = true;
        total = a.free_capacity;
    }
    for (int i = gtid; i < (int)total; i += gsz)
        a.pool_next[i] = i < rest ? a.pool[consumed + i] : a.freed[i - rest];
    if (a.released_k != nullptr) {
        int64_t base = 0;
        for (int k = 0; k < a.wave; ++k) base += a.all_counts[k].num_released;
        const int n = a.wave_counts->num_released;
        for (int i = gtid; i < n && base + i < a.released_capacity; i += gsz) a.released_out[base + i] = a.released_k[i];
        if (gtid == 0 && a.last && a.num_released_out != nullptr) *a.num_released_out = (int32_t)(base + n);
    } else if (gtid == 0 && a.last && a.num_released_out != nullptr) {
        *a.num_released_out = 0;
    }
    if (gtid == 0) {
        *a.num_pool_next = (int)total;
        a.wave_counts->error_flags |= a.ctx_counts->error_flags | (over ? VTOKEN_FLAG_CAPACITY : 0u);
    }
}

struct Layout {                       // workspace carve-up, every part 16-byte aligned
    int64_t freed, released, status, num_pool, pool, bt_offsets, bt_blocks, tt_slots, total;
};

Layout layout_of(const vtoken_ctx *ctx, int32_t free_capacity)
{
    auto up = [](int64_t b) { return (b + 15) & ~(int64_t)15; };
    const vtoken_config &c = ctx->cfg;
    Layout l;
    int64_t o = 0;
    l.freed = o;      o += up(4 * c.max_table_blocks);
    l.released = o;   o += up(4 * c.max_table_blocks);
    l.status = o;     o += up(4 * (int64_t)c.max_requests);
    l.num_pool = o;   o += 16;
    l.pool = o;       o += up(4 * (int64_t)(free_capacity > 1 ? free_capacity : 1));
    l.bt_offsets = o; o += up(4 * ((int64_t)c.max_requests + 1));
    l.bt_blocks = o;  o += up(4 * c.max_table_blocks);
    l.tt_slots = o;   o += up(4 * c.max_tokens);
    l.total = o;
    return l;
}

}  // namespace

extern "C" {

int64_t vtoken_waves_workspace_bytes(const vtoken_ctx *ctx, int32_t free_capacity)
{
    if (!ctx || free_capacity < 0) return 0;
    return layout_of(ctx, free_capacity).total;
}

int vtoken_repack_waves(vtoken_ctx *ctx, const vtoken_plan_in *in, const vtoken_partial_opts *opts,
                        int32_t num_waves, const vtoken_waves_out *out, void *cuda_stream)
{
    if (!ctx || !in || !out || num_waves < 1) return VTOKEN_EINVAL;
    if (!in->num_requests || !in->bt_offsets || !in->bt_blocks || !in->tt_offsets || !in->tt_slots || !in->keep ||
        !in->free_blocks || !in->num_free)
        return VTOKEN_EINVAL;
    if (!out->new_bt_offsets || !out->new_bt_blocks || !out->new_tt_slots || !out->req_status || !out->req_wave ||
        !out->free_out || !out->num_free_out || !out->wave_counts || !out->workspace)
        return VTOKEN_EINVAL;
    if (out->free_capacity < 0 || ((uintptr_t)out->workspace & 15)) return VTOKEN_EINVAL;
    const bool detach = opts && opts->protect != nullptr && opts->detach_den != 0;
    if (detach && !out->released_blocks) return VTOKEN_EINVAL;   // a detach threshold needs the list of dropped references
    if (out->free_capacity > ctx->cfg.max_free_blocks) return VTOKEN_ECAPACITY;
    const Layout l = layout_of(ctx, out->free_capacity);
    if (out->workspace_bytes < l.total) return VTOKEN_ECAPACITY;
    cudaStream_t st = (cudaStream_t)cuda_stream;
    uint8_t *ws = (uint8_t *)out->workspace;
    auto at = [&](int64_t off) { return (int32_t *)(ws + off); };

    // state buffers: index 0 = the caller's outputs, 1 = the workspace
    int32_t *bt_offsets[2] = {out->new_bt_offsets, at(l.bt_offsets)};
    int32_t *bt_blocks[2] = {out->new_bt_blocks, at(l.bt_blocks)};
    int32_t *tt_slots[2] = {out->new_tt_slots, at(l.tt_slots)};
    int32_t *pool[2] = {out->free_out, at(l.pool)};
    int32_t *num_pool[2] = {out->num_free_out, at(l.num_pool)};

    vtoken_plan_in cur = *in;
    for (int32_t k = 0; k < num_waves; ++k) {
        const int w = (num_waves - 1 - k) & 1;       // the last wave writes the caller's buffers
        vtoken_plan_out po;
        po.new_bt_offsets = bt_offsets[w];
        po.new_bt_blocks = bt_blocks[w];
        po.new_tt_slots = tt_slots[w];
        po.freed_blocks = at(l.freed);
        po.req_status = at(l.status);
        po.counts = out->wave_counts + k;
        po.released_blocks = detach ? at(l.released) : nullptr;
        int rc = opts ? vtoken_plan_partial(ctx, &cur, opts, &po, cuda_stream) : vtoken_plan(ctx, &cur, &po, cuda_stream);
        if (rc != VTOKEN_OK) return rc;
        rc = vtk_launch_copy(ctx, st);
        if (rc != VTOKEN_OK) return rc;

        CommitArgs a;
        a.num_requests = in->num_requests;
        a.max_requests = ctx->cfg.max_requests;
        a.wave = k;
        a.status_k = po.req_status;
        a.req_status = out->req_status;
        a.req_wave = out->req_wave;
        a.req_append_pos = out->req_append_pos;
        a.moved = opts ? ctx->req_nsrc : ctx->req_n;      // live tokens in the sources / of the request
        a.new_bt_offsets = po.new_bt_offsets;
        a.S = ctx->cfg.block_size;
        a.pool = cur.free_blocks;
        a.num_pool = cur.num_free;
        a.freed = po.freed_blocks;
        a.wave_counts = po.counts;
        a.ctx_counts = ctx->counts;
        a.pool_next = pool[w];
        a.num_pool_next = num_pool[w];
        a.free_capacity = out->free_capacity;
        a.released_k = detach ? po.released_blocks : nullptr;
        a.all_counts = out->wave_counts;
        a.released_out = out->released_blocks;
        a.num_released_out = out->num_released;
        a.released_capacity = ctx->cfg.max_table_blocks;
        a.last = k == num_waves - 1;
        int64_t span = out->free_capacity > ctx->cfg.max_requests ? out->free_capacity : ctx->cfg.max_requests;
        int blocks = (int)((span + COMMIT_NT - 1) / COMMIT_NT);
        if (blocks < 1) blocks = 1;
        if (blocks > ctx->num_sms * 8) blocks = ctx->num_sms * 8;
        VTK_CUDA(ctx, vtk_launch_dependent(ctx, wave_commit_kernel, dim3(blocks), dim3(COMMIT_NT), 0, st, a));
        VTK_CUDA(ctx, cudaGetLastError());

        cur.bt_offsets = po.new_bt_offsets;
        cur.bt_blocks = po.new_bt_blocks;
        cur.tt_slots = po.new_tt_slots;
        cur.free_blocks = pool[w];
        cur.num_free = num_pool[w];
    }
    return VTOKEN_OK;
}

}  // extern "C"
