// C ABI of libvtoken: argument checks, scratch allocation, launch sequencing.
#include "common.cuh"

#include <cstdlib>
#include <cstring>
#include <new>

namespace {

template <typename T>
int dev_alloc(vtoken_ctx *ctx, T **p, int64_t count)
{
    if (count < 1) count = 1;
    cudaError_t e = cudaMalloc((void **)p, (size_t)count * sizeof(T));
    if (e != cudaSuccess) {
        ctx->last_cuda_error = (int)e;
        *p = nullptr;
        return VTOKEN_ENOMEM;
    }
    ctx->scratch_bytes += count * (int64_t)sizeof(T);
    return VTOKEN_OK;
}

void free_all(vtoken_ctx *ctx)
{
    void *ptrs[] = {ctx->tile_n, ctx->req_part, ctx->req_before, ctx->req_n, ctx->req_dst_base, ctx->req_freed_base, ctx->req_status, ctx->dst_src,
                    ctx->dst_blocks, ctx->counts, ctx->rt_counts, ctx->plan_header, ctx->g_src, ctx->g_total, ctx->g_ids, ctx->g_req, ctx->g_offsets, ctx->tile_mov, ctx->tile_shared, ctx->part_mov, ctx->req_ns, ctx->req_nsrc,
                    ctx->n_b, ctx->slot_bits, ctx->copy_ticket, ctx->g_ticket, ctx->g_tile_n, ctx->g_req_part, ctx->g_req_before, ctx->part_shared, ctx->req_shared, ctx->req_detach,
                    ctx->req_rel_base, ctx->cow,
                    ctx->stage.num_requests, ctx->stage.bt_blocks,
                    ctx->stage.tt_slots, ctx->stage.free_blocks, ctx->stage.keep,
                    ctx->stage.new_bt_offsets, ctx->stage.new_bt_blocks,
                    ctx->stage.new_tt_slots, ctx->stage.freed_blocks, ctx->stage.req_status, ctx->stage.counts,
                    ctx->stage.protect, ctx->stage.released_blocks};
    for (void *p : ptrs)
        if (p) cudaFree(p);
    if (ctx->stage.h_scalars) cudaFreeHost(ctx->stage.h_scalars);
    if (ctx->stage.h_counts) cudaFreeHost(ctx->stage.h_counts);
    if (ctx->stage.planned) cudaEventDestroy(ctx->stage.planned);
    if (ctx->stage.copied) cudaEventDestroy(ctx->stage.copied);
    if (ctx->stage.aux) cudaStreamDestroy(ctx->stage.aux);
}

int ensure_stage(vtoken_ctx *ctx)
{
    if (ctx->stage.ready) return VTOKEN_OK;
    const vtoken_config &c = ctx->cfg;
    int rc = VTOKEN_OK;
    auto A = [&](auto **p, int64_t n) { if (rc == VTOKEN_OK) rc = dev_alloc(ctx, p, n); };
    // The small inputs -- the two scalars, both offset arrays, the selection bytes -- share one device
    // allocation and one pinned host mirror, so that they travel in a single copy: every copy call costs
    // the submitting thread a few microseconds whatever its size, and the GPU waits for the last of them.
    const int64_t rc1 = (int64_t)c.max_requests + 1;
    ctx->stage.small_ints = 2 + 2 * rc1 + (c.max_requests + 3) / 4;
    A(&ctx->stage.num_requests, ctx->stage.small_ints);
    if (rc == VTOKEN_OK) {
        ctx->stage.num_free = ctx->stage.num_requests + 1;
        ctx->stage.bt_offsets = ctx->stage.num_requests + 2;
        ctx->stage.tt_offsets = ctx->stage.bt_offsets + rc1;
        ctx->stage.select = reinterpret_cast<uint8_t *>(ctx->stage.tt_offsets + rc1);
    }
    A(&ctx->stage.bt_blocks, c.max_table_blocks);
    A(&ctx->stage.tt_slots, c.max_tokens);
    A(&ctx->stage.free_blocks, c.max_free_blocks);
    A(&ctx->stage.keep, c.max_tokens);
    A(&ctx->stage.new_bt_offsets, (int64_t)c.max_requests + 1);
    A(&ctx->stage.new_bt_blocks, c.max_table_blocks);
    A(&ctx->stage.new_tt_slots, c.max_tokens);
    A(&ctx->stage.freed_blocks, c.max_table_blocks);
    A(&ctx->stage.req_status, c.max_requests);
    A(&ctx->stage.counts, 1);
    if (rc == VTOKEN_OK) {
        if (cudaMallocHost((void **)&ctx->stage.h_scalars, (size_t)ctx->stage.small_ints * sizeof(int32_t)) != cudaSuccess ||
            cudaMallocHost((void **)&ctx->stage.h_counts, sizeof(vtoken_counts)) != cudaSuccess ||
            cudaStreamCreateWithFlags(&ctx->stage.aux, cudaStreamNonBlocking) != cudaSuccess ||
            cudaEventCreateWithFlags(&ctx->stage.planned, cudaEventDisableTiming) != cudaSuccess ||
            cudaEventCreateWithFlags(&ctx->stage.copied, cudaEventDisableTiming) != cudaSuccess)
            rc = VTOKEN_ECUDA;
    }
    if (rc == VTOKEN_OK) ctx->stage.ready = true;
    return rc;
}

}  // namespace

extern "C" {

int vtoken_create(const vtoken_config *cfg, vtoken_ctx **out_ctx)
{
    if (!cfg || !out_ctx) return VTOKEN_EINVAL;
    *out_ctx = nullptr;
    if (cfg->num_layers < 1 || cfg->num_blocks < 1 || cfg->block_size < 1 || cfg->num_kv_heads < 1 ||
        cfg->head_dim < 1 || cfg->elem_bytes < 1 || !cfg->k_pool || !cfg->v_pool || cfg->max_requests < 1 ||
        cfg->max_tokens < 1 || cfg->max_table_blocks < 1 || cfg->max_free_blocks < 0 || cfg->max_ctas < 0 ||
        cfg->debug_stall_item < 0)
        return VTOKEN_EINVAL;
    const int64_t row_bytes = (int64_t)cfg->num_kv_heads * cfg->head_dim * cfg->elem_bytes;
    const int64_t slots = (int64_t)cfg->num_blocks * cfg->block_size;
    if (row_bytes % 16 != 0) return VTOKEN_EINVAL;
    if (cfg->plan_variant < 0 || cfg->plan_variant > 2) return VTOKEN_EINVAL;
    if (slots >= (int64_t)INT32_MAX) return VTOKEN_EINVAL;            // slots are int32
    if (cfg->max_tokens >= (int64_t)INT32_MAX || cfg->max_table_blocks >= (int64_t)INT32_MAX) return VTOKEN_EINVAL;
    const int64_t stride = cfg->layer_stride_bytes ? cfg->layer_stride_bytes : slots * row_bytes;
    if (stride < slots * row_bytes || stride % 16 != 0) return VTOKEN_EINVAL;
    if (((uintptr_t)cfg->k_pool | (uintptr_t)cfg->v_pool) & 15) return VTOKEN_EINVAL;

    vtoken_ctx *ctx = new (std::nothrow) vtoken_ctx;
    if (!ctx) return VTOKEN_ENOMEM;
    memset(ctx, 0, sizeof(*ctx));
    ctx->cfg = *cfg;
    ctx->row_bytes = row_bytes;
    ctx->layer_stride = stride;
    ctx->slots_per_layer = slots;
    int64_t cap = (cfg->max_tokens + cfg->block_size - 1) / cfg->block_size + cfg->max_requests;
    if (cap > cfg->max_free_blocks) cap = cfg->max_free_blocks;
    if (cap < 1) cap = 1;
    ctx->cap_dst_blocks = (int32_t)cap;

    cudaError_t e = cudaGetDevice(&ctx->device);
    if (e == cudaSuccess) e = cudaDeviceGetAttribute(&ctx->num_sms, cudaDevAttrMultiProcessorCount, ctx->device);
    if (e != cudaSuccess) { delete ctx; return VTOKEN_ECUDA; }

    int rc = VTOKEN_OK;
    auto A = [&](auto **p, int64_t n) { if (rc == VTOKEN_OK) rc = dev_alloc(ctx, p, n); };
    A(&ctx->req_n, cfg->max_requests);
    A(&ctx->req_dst_base, cfg->max_requests);
    A(&ctx->plan_header, 4);
    A(&ctx->tile_n, (cfg->max_tokens + 1023) / 1024 + 1);
    A(&ctx->req_part, (int64_t)cfg->max_requests + 1);
    A(&ctx->req_before, (int64_t)cfg->max_requests + 1);
    A(&ctx->req_freed_base, cfg->max_requests);
    A(&ctx->req_status, cfg->max_requests);
    A(&ctx->dst_src, cap * cfg->block_size);
    A(&ctx->dst_blocks, cap);
    A(&ctx->counts, 1);
    A(&ctx->rt_counts, 1);
    if (rc == VTOKEN_OK && cudaMemset(ctx->rt_counts, 0, sizeof(vtoken_counts)) != cudaSuccess) rc = VTOKEN_ECUDA;
    A(&ctx->g_src, cfg->max_tokens);
    A(&ctx->g_total, 1);
    A(&ctx->g_ids, cfg->max_tokens);
    A(&ctx->g_req, cfg->max_tokens);
    A(&ctx->g_offsets, (int64_t)cfg->max_requests + 1);
    A(&ctx->g_tile_n, (cfg->max_tokens + 1023) / 1024 + 1);
    A(&ctx->g_req_part, (int64_t)cfg->max_requests + 1);
    A(&ctx->g_req_before, (int64_t)cfg->max_requests + 1);
    A(&ctx->tile_mov, (cfg->max_tokens + 1023) / 1024 + 1);
    A(&ctx->tile_shared, (cfg->max_tokens + 1023) / 1024 + 1);
    A(&ctx->part_mov, (int64_t)cfg->max_requests + 1);
    A(&ctx->req_ns, cfg->max_requests);
    A(&ctx->req_nsrc, cfg->max_requests);
    A(&ctx->n_b, (int64_t)cfg->num_blocks + (cfg->num_blocks + 3) / 4);      // n_b, then blk_src (one byte per block)
    if (rc == VTOKEN_OK) ctx->blk_src = reinterpret_cast<uint8_t *>(ctx->n_b + cfg->num_blocks);
    A(&ctx->slot_bits, (slots + 31) / 32);
    A(&ctx->copy_ticket, 2);
    if (rc == VTOKEN_OK && cudaMemset(ctx->copy_ticket, 0, 2 * sizeof(unsigned int)) != cudaSuccess) rc = VTOKEN_ECUDA;
    A(&ctx->g_ticket, 2);
    if (rc == VTOKEN_OK && cudaMemset(ctx->g_ticket, 0, 2 * sizeof(unsigned int)) != cudaSuccess) rc = VTOKEN_ECUDA;
    A(&ctx->part_shared, (int64_t)cfg->max_requests + 1);
    A(&ctx->req_shared, cfg->max_requests);
    A(&ctx->req_detach, cfg->max_requests);
    A(&ctx->req_rel_base, cfg->max_requests);
    A(&ctx->cow, 2 * (int64_t)cfg->max_table_blocks);
    if (rc == VTOKEN_OK && cudaMemset(ctx->counts, 0, sizeof(vtoken_counts)) != cudaSuccess) rc = VTOKEN_ECUDA;
    if (rc == VTOKEN_OK) rc = vtk_configure_copy(ctx);
    if (rc == VTOKEN_OK) rc = vtk_configure_plan(ctx);
    if (rc != VTOKEN_OK) { free_all(ctx); delete ctx; return rc; }
    *out_ctx = ctx;
    return VTOKEN_OK;
}

void vtoken_destroy(vtoken_ctx *ctx)
{
    if (!ctx) return;
    free_all(ctx);
    delete ctx;
}

int vtoken_plan(vtoken_ctx *ctx, const vtoken_plan_in *in, const vtoken_plan_out *out, void *cuda_stream)
{
    if (!ctx || !in || !out) return VTOKEN_EINVAL;
    if (!in->num_requests || !in->bt_offsets || !in->bt_blocks || !in->tt_offsets || !in->tt_slots || !in->keep ||
        !in->free_blocks || !in->num_free)
        return VTOKEN_EINVAL;
    if (!out->new_bt_offsets || !out->new_bt_blocks || !out->new_tt_slots || !out->freed_blocks ||
        !out->req_status || !out->counts)
        return VTOKEN_EINVAL;
    int rc = vtk_launch_plan(ctx, in, out, (cudaStream_t)cuda_stream);
    if (rc == VTOKEN_OK) ctx->has_plan = true;
    return rc;
}

int vtoken_repack(vtoken_ctx *ctx, void *cuda_stream)
{
    if (!ctx) return VTOKEN_EINVAL;
    if (!ctx->has_plan) return VTOKEN_ESTATE;
    return vtk_launch_copy(ctx, (cudaStream_t)cuda_stream);
}

int vtoken_gather_logical(vtoken_ctx *ctx, const int32_t *num_requests, const int32_t *tt_offsets,
                          const int32_t *tt_slots, const uint8_t *keep, const uint8_t *select,
                          int32_t layer_begin, int32_t layer_end, void *out_k, void *out_v,
                          int64_t out_capacity_tokens, int32_t *out_offsets, void *cuda_stream)
{
    if (!ctx || !num_requests || !tt_offsets || !tt_slots || !out_k || !out_v || !out_offsets) return VTOKEN_EINVAL;
    if (layer_begin < 0 || layer_end > ctx->cfg.num_layers || layer_begin >= layer_end) return VTOKEN_EINVAL;
    if (out_capacity_tokens < 0) return VTOKEN_EINVAL;
    if (((uintptr_t)out_k | (uintptr_t)out_v) & 15) return VTOKEN_EINVAL;
    return vtk_launch_gather(ctx, num_requests, tt_offsets, tt_slots, keep, select, layer_begin, layer_end, out_k,
                             out_v, out_capacity_tokens, out_offsets, (cudaStream_t)cuda_stream);
}

int vtoken_read_counts(vtoken_ctx *ctx, vtoken_counts *host_out, void *cuda_stream)
{
    if (!ctx || !host_out) return VTOKEN_EINVAL;
    cudaStream_t st = (cudaStream_t)cuda_stream;
    uint32_t rt_flags = 0;
    VTK_CUDA(ctx, cudaMemcpyAsync(host_out, ctx->counts, sizeof(vtoken_counts), cudaMemcpyDeviceToHost, st));
    VTK_CUDA(ctx, cudaMemcpyAsync(&rt_flags, &ctx->rt_counts->error_flags, sizeof(uint32_t), cudaMemcpyDeviceToHost, st));
    VTK_CUDA(ctx, cudaMemsetAsync(&ctx->rt_counts->error_flags, 0, sizeof(uint32_t), st));   // reported once
    VTK_CUDA(ctx, cudaStreamSynchronize(st));
    host_out->error_flags |= rt_flags;
    return VTOKEN_OK;
}

static int repack_host(vtoken_ctx *ctx, const vtoken_host_tables *h, const vtoken_partial_opts *opts,
                       void *cuda_stream)
{
    if (!ctx || !h) return VTOKEN_EINVAL;
    if (opts && opts->max_source_blocks < 0) return VTOKEN_EINVAL;
    const bool detach = opts && opts->protect != nullptr && opts->detach_den != 0;
    if (detach && !h->released_blocks) return VTOKEN_EINVAL;    // a detach threshold needs the list of dropped references
    if (!h->bt_offsets || !h->bt_blocks || !h->tt_offsets || !h->tt_slots || !h->keep || !h->free_blocks ||
        !h->new_bt_offsets || !h->new_bt_blocks || !h->new_tt_slots || !h->freed_blocks || !h->req_status ||
        !h->counts)
        return VTOKEN_EINVAL;
    const int32_t R = h->num_requests;
    if (R < 0 || h->num_free < 0) return VTOKEN_EINVAL;
    if (R > ctx->cfg.max_requests || h->num_free > ctx->cfg.max_free_blocks) return VTOKEN_ECAPACITY;
    const int64_t T = h->tt_offsets[R], NBT = h->bt_offsets[R];
    if (T < 0 || NBT < 0) return VTOKEN_EINVAL;
    if (T > ctx->cfg.max_tokens || NBT > ctx->cfg.max_table_blocks) return VTOKEN_ECAPACITY;
    int rc = ensure_stage(ctx);
    if (rc != VTOKEN_OK) return rc;
    cudaStream_t st = (cudaStream_t)cuda_stream;
    auto &s = ctx->stage;
    if (opts && opts->protect && !s.protect) {      // device copy of the protect mask, on first use
        rc = dev_alloc(ctx, &s.protect, ctx->cfg.num_blocks);
        if (rc != VTOKEN_OK) return rc;
    }
#define H2D(dst, src, n) VTK_CUDA(ctx, cudaMemcpyAsync(dst, src, (size_t)(n), cudaMemcpyHostToDevice, st))
#define D2H(dst, src, n) VTK_CUDA(ctx, cudaMemcpyAsync(dst, src, (size_t)(n), cudaMemcpyDeviceToHost, st))
    // the token table first: its transfer runs while this thread submits the rest
    if (T) H2D(s.tt_slots, h->tt_slots, T * sizeof(int32_t));
    if (T) H2D(s.keep, h->keep, T);
    {
        // scalars, offsets and selection bytes through the pinned mirror, in one copy
        const int64_t rc1 = (int64_t)ctx->cfg.max_requests + 1;
        int32_t *m = s.h_scalars;
        m[0] = h->num_requests;
        m[1] = h->num_free;
        memcpy(m + 2, h->bt_offsets, (size_t)(R + 1) * sizeof(int32_t));
        memcpy(m + 2 + rc1, h->tt_offsets, (size_t)(R + 1) * sizeof(int32_t));
        if (h->select && R) memcpy(m + 2 + 2 * rc1, h->select, (size_t)R);
        H2D(s.num_requests, m, s.small_ints * sizeof(int32_t));
    }
    if (NBT) H2D(s.bt_blocks, h->bt_blocks, NBT * sizeof(int32_t));
    if (h->num_free) H2D(s.free_blocks, h->free_blocks, h->num_free * sizeof(int32_t));
    if (opts && opts->protect) H2D(s.protect, opts->protect, ctx->cfg.num_blocks);

    vtoken_plan_in in;
    in.num_requests = s.num_requests;
    in.bt_offsets = s.bt_offsets;
    in.bt_blocks = s.bt_blocks;
    in.tt_offsets = s.tt_offsets;
    in.tt_slots = s.tt_slots;
    in.keep = s.keep;
    in.select = h->select ? s.select : nullptr;
    in.thr_num = h->thr_num;
    in.thr_den = h->thr_den;
    in.free_blocks = s.free_blocks;
    in.num_free = s.num_free;
    vtoken_plan_out out;
    out.new_bt_offsets = s.new_bt_offsets;
    out.new_bt_blocks = s.new_bt_blocks;
    out.new_tt_slots = s.new_tt_slots;
    out.freed_blocks = s.freed_blocks;
    out.req_status = s.req_status;
    out.counts = s.counts;
    out.released_blocks = nullptr;
    if (detach) {
        if (!s.released_blocks) {                     // device copy of the released list, on first use
            rc = dev_alloc(ctx, &s.released_blocks, ctx->cfg.max_table_blocks);
            if (rc != VTOKEN_OK) return rc;
        }
        out.released_blocks = s.released_blocks;
    }
    if (opts) {
        vtoken_partial_opts dopts = *opts;
        dopts.protect = opts->protect ? s.protect : nullptr;
        rc = vtoken_plan_partial(ctx, &in, &dopts, &out, st);
    } else {
        rc = vtk_launch_plan(ctx, &in, &out, st);
    }
    if (rc != VTOKEN_OK) return rc;
    ctx->has_plan = true;
    // every table output is final once the plan has run: copy them back on a second stream
    // while the copy kernel moves the K/V rows on the caller's stream
    VTK_CUDA(ctx, cudaEventRecord(s.planned, st));
    rc = vtk_launch_copy(ctx, st);
    if (rc != VTOKEN_OK) return rc;
    cudaStream_t caller = st;
    VTK_CUDA(ctx, cudaStreamWaitEvent(s.aux, s.planned, 0));
    st = s.aux;
    D2H(h->new_bt_offsets, s.new_bt_offsets, (R + 1) * sizeof(int32_t));
    if (NBT) D2H(h->new_bt_blocks, s.new_bt_blocks, NBT * sizeof(int32_t));
    if (T) D2H(h->new_tt_slots, s.new_tt_slots, T * sizeof(int32_t));
    if (NBT) D2H(h->freed_blocks, s.freed_blocks, NBT * sizeof(int32_t));
    if (R) D2H(h->req_status, s.req_status, R * sizeof(int32_t));
    if (detach && NBT) D2H(h->released_blocks, s.released_blocks, NBT * sizeof(int32_t));
    VTK_CUDA(ctx, cudaEventRecord(s.copied, s.aux));
    st = caller;
    VTK_CUDA(ctx, cudaStreamWaitEvent(st, s.copied, 0));
    // the counts are read from the context's copy so that flags raised by the copy kernel are included
    D2H(s.h_counts, ctx->counts, sizeof(vtoken_counts));
#undef H2D
#undef D2H
    VTK_CUDA(ctx, cudaStreamSynchronize(st));
    *h->counts = *s.h_counts;
    return VTOKEN_OK;
}

int vtoken_repack_host(vtoken_ctx *ctx, const vtoken_host_tables *tables, void *cuda_stream)
{
    return repack_host(ctx, tables, nullptr, cuda_stream);
}

int vtoken_repack_host_partial(vtoken_ctx *ctx, const vtoken_host_tables *tables, const vtoken_partial_opts *opts,
                               void *cuda_stream)
{
    if (!opts) return VTOKEN_EINVAL;
    return repack_host(ctx, tables, opts, cuda_stream);
}

const char *vtoken_strerror(int code)
{
    switch (code) {
        case VTOKEN_OK: return "ok";
        case VTOKEN_EINVAL: return "invalid argument (NULL pointer, shape, or alignment)";
        case VTOKEN_ECAPACITY: return "size exceeds a capacity given to vtoken_create";
        case VTOKEN_ECUDA: return "CUDA call failed (see vtoken_last_cuda_error)";
        case VTOKEN_ENOMEM: return "device scratch allocation failed";
        case VTOKEN_ESTATE: return "vtoken_repack called without a plan";
        default: return "unknown vtoken error code";
    }
}

int vtoken_last_cuda_error(const vtoken_ctx *ctx) { return ctx ? ctx->last_cuda_error : 0; }

int vtoken_copy_grid(const vtoken_ctx *ctx, int32_t *ctas, int32_t *threads, int32_t *smem_bytes, int32_t *variant)
{
    if (!ctx) return VTOKEN_EINVAL;
    if (ctas) *ctas = ctx->copy_ctas;
    if (threads) *threads = ctx->copy_threads;
    if (smem_bytes) *smem_bytes = ctx->copy_smem;
    if (variant) *variant = ctx->copy_variant;
    return VTOKEN_OK;
}

int64_t vtoken_scratch_bytes(const vtoken_ctx *ctx) { return ctx ? ctx->scratch_bytes : 0; }

int vtoken_plan_form(const vtoken_ctx *ctx) { return ctx ? ctx->plan_form : VTOKEN_EINVAL; }

namespace {
__global__ void probe_kernel(vtk_arr<int32_t> arr, int64_t index, int32_t *out)
{
    *out = arr[index];          // checked build: outside [0, n) this reads a dummy element and raises the flag
}
}  // namespace

int vtoken_debug_probe(vtoken_ctx *ctx, int64_t index, int32_t *out_value, void *cuda_stream)
{
#ifdef VTOKEN_CHECKED
    if (!ctx || !out_value) return VTOKEN_EINVAL;
    probe_kernel<<<1, 1, 0, (cudaStream_t)cuda_stream>>>(VTK_ARR(ctx, ctx->req_n, ctx->cfg.max_requests), index, out_value);
    VTK_CUDA(ctx, cudaGetLastError());
    return VTOKEN_OK;
#else
    (void)ctx; (void)index; (void)out_value; (void)cuda_stream;
    return VTOKEN_EINVAL;       // the production library has no checked arrays to probe
#endif
}

int vtoken_checked_build(void)
{
#ifdef VTOKEN_CHECKED
    return 1;
#else
    return 0;
#endif
}

}  // extern "C"
