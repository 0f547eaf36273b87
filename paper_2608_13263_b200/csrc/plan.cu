// Relocation planner (Sec. 3.3.3 of the paper) as three small kernels:
//   count  : live tokens per request part                (warp ballot + popc)
//   scan   : candidates, admission against the free list, per-request bases, counts (one CTA)
//   assign : rank of every live token -> destination slot, new tables, reclaimed list,
//            inverse move plan for the copy kernel
// Every request is cut into PLAN_PARTS equal token ranges, one CTA each in count and assign, so
// that a 32k-token request does not serialise on one CTA; a part's first rank is the sum of the
// live counts of the parts before it.  All grids are fixed by the capacities; R, T and num_free
// are read from device memory.  No output order depends on atomics.
#include "common.cuh"

namespace {

constexpr int PLAN_NT = 512;    // threads per CTA of count / assign
constexpr int PLAN_PARTS = VTK_PLAN_PARTS;   // token ranges per request
constexpr int SCAN_NT = 1024;   // threads of the single scan CTA

struct PlanArgs {
    // inputs
    const int32_t *num_requests, *bt_offsets, *bt_blocks, *tt_offsets, *tt_slots;
    const uint8_t *keep, *select;
    uint32_t thr_num, thr_den;
    const int32_t *free_blocks, *num_free;
    // outputs
    int32_t *new_bt_offsets, *new_bt_blocks, *new_tt_slots, *freed_blocks, *out_status;
    vtoken_counts *out_counts;
    // context
    int32_t *req_n, *part_n, *req_dst_base, *req_freed_base, *req_status, *dst_src, *dst_blocks;
    vtoken_counts *counts;
    int32_t S, num_blocks, max_requests, cap_dst_blocks, max_free_blocks;
    int64_t slots_per_layer, max_tokens, max_table_blocks;
};

__device__ __forceinline__ int clamp_requests(const PlanArgs &a)
{
    int R = *a.num_requests;
    return R < 0 ? 0 : (R > a.max_requests ? a.max_requests : R);
}

// token range [p0, p1) of part c of a request spanning [t0, t1): equal parts, multiples of 128
__device__ __forceinline__ void part_range(int64_t t0, int64_t t1, int c, int64_t &p0, int64_t &p1)
{
    const int64_t len = t1 - t0;
    int64_t per = (len + PLAN_PARTS - 1) / PLAN_PARTS;
    per = (per + 127) & ~(int64_t)127;
    p0 = t0 + (int64_t)c * per;
    p1 = p0 + per;
    if (p0 > t1) p0 = t1;
    if (p1 > t1) p1 = t1;
}

__device__ __forceinline__ void raise_flags(const PlanArgs &a, uint32_t flags)
{
    atomicOr(&a.counts->error_flags, flags);
    atomicOr(&a.out_counts->error_flags, flags);
}

// ---- count -----------------------------------------------------------------------------
__global__ void __launch_bounds__(PLAN_NT) plan_count_kernel(PlanArgs a)
{
    vtk_release_successor();
    vtk_wait_for_predecessor();
    const int r = blockIdx.x / PLAN_PARTS, c = blockIdx.x % PLAN_PARTS;
    if (r >= clamp_requests(a)) return;
    int64_t t0, t1, p0, p1;
    vtk_range(a.tt_offsets, r, a.max_tokens, t0, t1);
    part_range(t0, t1, c, p0, p1);
    int n = 0;
    bool bad = false;
    for (int64_t t = p0 + threadIdx.x; t < p1; t += PLAN_NT)
        n += vtk_live(a.tt_slots[t], a.keep, t, a.slots_per_layer, bad) ? 1 : 0;
    __shared__ int warp_n[PLAN_NT / 32];
#pragma unroll
    for (int d = 16; d > 0; d >>= 1) n += __shfl_down_sync(0xffffffffu, n, d);
    if (vtk_lane() == 0) warp_n[threadIdx.x >> 5] = n;
    if (bad) atomicOr(&a.counts->error_flags, VTOKEN_FLAG_BAD_SLOT);
    __syncthreads();
    if (threadIdx.x == 0) {
        int s = 0;
        for (int w = 0; w < PLAN_NT / 32; ++w) s += warp_n[w];
        a.part_n[blockIdx.x] = s;
    }
}

// ---- scan ------------------------------------------------------------------------------
struct Acc {                    // running sums over admitted requests (and table sizes)
    int dst, freed, newbt, moves, admitted, deferred;
};
__device__ __forceinline__ Acc operator+(const Acc &x, const Acc &y)
{
    return Acc{x.dst + y.dst, x.freed + y.freed, x.newbt + y.newbt, x.moves + y.moves,
               x.admitted + y.admitted, x.deferred + y.deferred};
}
__device__ __forceinline__ Acc shfl_up(const Acc &v, int d)
{
    return Acc{__shfl_up_sync(0xffffffffu, v.dst, d), __shfl_up_sync(0xffffffffu, v.freed, d),
               __shfl_up_sync(0xffffffffu, v.newbt, d), __shfl_up_sync(0xffffffffu, v.moves, d),
               __shfl_up_sync(0xffffffffu, v.admitted, d), __shfl_up_sync(0xffffffffu, v.deferred, d)};
}

template <typename T, typename ShflUp>
__device__ __forceinline__ T block_incl_scan(T v, T *warp_tot, T zero, ShflUp shfl)
{
    const int lane = vtk_lane(), warp = threadIdx.x >> 5;
#pragma unroll
    for (int d = 1; d < 32; d <<= 1) {
        T o = shfl(v, d);
        if (lane >= d) v = o + v;
    }
    if (lane == 31) warp_tot[warp] = v;
    __syncthreads();
    if (warp == 0) {
        T w = warp_tot[lane];           // SCAN_NT / 32 == 32 warps
#pragma unroll
        for (int d = 1; d < 32; d <<= 1) {
            T o = shfl(w, d);
            if (lane >= d) w = o + w;
        }
        warp_tot[lane] = w;
    }
    __syncthreads();
    T pre = warp == 0 ? zero : warp_tot[warp - 1];
    T res = pre + v;
    __syncthreads();
    return res;
}

__global__ void __launch_bounds__(SCAN_NT) plan_scan_kernel(PlanArgs a)
{
    __shared__ long long warp_ll[32];
    __shared__ Acc warp_acc[32];
    __shared__ long long carry_need;
    __shared__ Acc carry;
    const int tid = threadIdx.x;
    vtk_release_successor();
    vtk_wait_for_predecessor();
    const int R = clamp_requests(a);
    uint32_t flags = 0;
    if (tid == 0) {
        if (*a.num_requests > a.max_requests || *a.num_requests < 0) flags |= VTOKEN_FLAG_CAPACITY;
        carry_need = 0;
        carry = Acc{0, 0, 0, 0, 0, 0};
    }
    int nf = *a.num_free;
    if (nf > a.max_free_blocks && tid == 0) flags |= VTOKEN_FLAG_CAPACITY;
    nf = nf < 0 ? 0 : (nf > a.cap_dst_blocks ? a.cap_dst_blocks : nf);
    __syncthreads();

    auto shfl_ll = [](long long v, int d) { return __shfl_up_sync(0xffffffffu, v, d); };
    auto shfl_acc = [](const Acc &v, int d) { return shfl_up(v, d); };

    for (int base = 0; base < R; base += SCAN_NT) {
        const int r = base + tid;
        const bool valid = r < R;
        int n = 0, nb = 0;
        if (valid) {
#pragma unroll
            for (int c = 0; c < PLAN_PARTS; ++c) n += a.part_n[r * PLAN_PARTS + c];
            a.req_n[r] = n;
            int64_t lo, hi, t0, t1;
            const bool clipped = vtk_range(a.bt_offsets, r, a.max_table_blocks, lo, hi) |
                                 vtk_range(a.tt_offsets, r, a.max_tokens, t0, t1);
            if (clipped) flags |= VTOKEN_FLAG_CAPACITY;     // tables beyond the create-time capacities
            nb = (int)(hi - lo);
        }
        const int need = (int)(((int64_t)n + a.S - 1) / a.S);       // ceil(T_live / S)
        bool sel = valid && (a.select == nullptr || a.select[r] != 0);
        if (sel && a.thr_den != 0)
            sel = (unsigned long long)n * a.thr_den <
                  (unsigned long long)a.thr_num * (unsigned long long)nb * (unsigned long long)a.S;
        const bool cand = sel && need < nb;                          // strictly fewer blocks afterwards
        // admission: cumulative demand of candidates so far (this one included) fits the free list
        const long long cum = block_incl_scan<long long>(cand ? need : 0, warp_ll, 0LL, shfl_ll) + carry_need;
        const bool adm = cand && cum <= (long long)nf;
        const int status = !sel ? VTOKEN_NOT_SELECTED
                                : (!cand ? VTOKEN_NO_GAIN : (adm ? VTOKEN_REPACKED : VTOKEN_DEFERRED_NO_FREE));
        Acc mine{adm ? need : 0, adm ? nb : 0, valid ? (adm ? need : nb) : 0, adm ? n : 0, adm ? 1 : 0,
                 (cand && !adm) ? 1 : 0};
        const Acc incl = block_incl_scan<Acc>(mine, warp_acc, Acc{0, 0, 0, 0, 0, 0}, shfl_acc) + carry;
        if (valid) {
            a.req_dst_base[r] = incl.dst - mine.dst;
            a.req_freed_base[r] = incl.freed - mine.freed;
            a.new_bt_offsets[r] = incl.newbt - mine.newbt;
            a.req_status[r] = status;
            a.out_status[r] = status;
        }
        __syncthreads();
        if (tid == SCAN_NT - 1) {          // last thread holds the chunk totals
            carry_need = cum;
            carry = incl;
        }
        __syncthreads();
    }
    if (flags) atomicOr(&a.counts->error_flags, flags);
    __syncthreads();
    if (tid == 0) {
        a.new_bt_offsets[R] = carry.newbt;
        vtoken_counts c;
        c.num_moves = carry.moves;
        c.num_dst_blocks = carry.dst;
        c.num_freed = carry.freed;
        c.num_free_consumed = carry.dst;
        c.num_admitted = carry.admitted;
        c.num_deferred = carry.deferred;
        c.error_flags = atomicOr(&a.counts->error_flags, 0u);   // bits raised by the count kernel and above
        c.num_released = 0;
        *a.counts = c;
        *a.out_counts = c;                               // later flags are OR-ed into both copies
    }
}

// ---- assign ----------------------------------------------------------------------------
__global__ void __launch_bounds__(PLAN_NT) plan_assign_kernel(PlanArgs a)
{
    __shared__ int warp_sums[PLAN_NT / 32 + 1];
    vtk_release_successor();
    vtk_wait_for_predecessor();
    const int r = blockIdx.x / PLAN_PARTS, c = blockIdx.x % PLAN_PARTS;
    if (r >= clamp_requests(a)) return;
    const int tid = threadIdx.x;
    const int S = a.S;
    int64_t t0, t1, b0, b1;
    vtk_range(a.tt_offsets, r, a.max_tokens, t0, t1);
    vtk_range(a.bt_offsets, r, a.max_table_blocks, b0, b1);
    const int nb = (int)(b1 - b0);
    const bool adm = a.req_status[r] == VTOKEN_REPACKED;
    const int n = a.req_n[r];
    const int need = (int)(((int64_t)n + S - 1) / S);
    const int dst_base = a.req_dst_base[r];
    const int nbt0 = a.new_bt_offsets[r];
    uint32_t flags = 0;

    // block tables and the reclaimed list: the request's parts share the work in stripes
    const int stripe = c * PLAN_NT + tid, stride = PLAN_PARTS * PLAN_NT;
    if (adm) {
        for (int j = stripe; j < need; j += stride) {
            int blk = a.free_blocks[dst_base + j];
            if ((int64_t)nbt0 + j < a.max_table_blocks) a.new_bt_blocks[nbt0 + j] = blk;
            if (blk < 0 || blk >= a.num_blocks) { flags |= VTOKEN_FLAG_BAD_FREE; blk = -1; }
            a.dst_blocks[dst_base + j] = blk;
        }
        const int f0 = a.req_freed_base[r];
        for (int j = stripe; j < nb && (int64_t)f0 + j < a.max_table_blocks; j += stride) {
            const int blk = a.bt_blocks[b0 + j];
            if (blk < 0 || blk >= a.num_blocks) flags |= VTOKEN_FLAG_BAD_BLOCK;
            a.freed_blocks[f0 + j] = blk;
        }
        // unused tail of the last destination block
        for (int i = n + stripe; i < need * S; i += stride) a.dst_src[(int64_t)dst_base * S + i] = -1;
    } else {
        for (int j = stripe; j < nb && (int64_t)nbt0 + j < a.max_table_blocks; j += stride)
            a.new_bt_blocks[nbt0 + j] = a.bt_blocks[b0 + j];
    }

    // token table: rank of each live token in logical order -> destination slot
    int64_t p0, p1;
    part_range(t0, t1, c, p0, p1);
    int carry = 0;                                       // live tokens of the parts before this one
    for (int cc = 0; cc < c; ++cc) carry += a.part_n[r * PLAN_PARTS + cc];
    for (int64_t tb = p0; tb < p1; tb += PLAN_NT) {
        const int64_t t = tb + tid;
        int32_t slot = -1;
        bool live = false, bad = false;
        if (t < p1) {
            slot = a.tt_slots[t];
            live = vtk_live(slot, a.keep, t, a.slots_per_layer, bad);
        }
        int total;
        const int i = carry + vtk_block_rank<PLAN_NT>(live, warp_sums, total);
        carry += total;
        if (t < p1) {
            int32_t out = -1;
            if (live) {
                if (adm) {
                    const int j = i / S, off = i - j * S;
                    const int blk = a.free_blocks[dst_base + j];
                    out = blk * S + off;                    // slot = block_id * S + offset
                    a.dst_src[(int64_t)(dst_base + j) * S + off] = slot;
                } else {
                    out = slot;
                }
            }
            a.new_tt_slots[t] = out;
        }
    }
    if (flags) raise_flags(a, flags);
}

}  // namespace

int vtk_launch_plan(vtoken_ctx *ctx, const vtoken_plan_in *in, const vtoken_plan_out *out, cudaStream_t st)
{
    PlanArgs a;
    a.num_requests = in->num_requests;
    a.bt_offsets = in->bt_offsets;
    a.bt_blocks = in->bt_blocks;
    a.tt_offsets = in->tt_offsets;
    a.tt_slots = in->tt_slots;
    a.keep = in->keep;
    a.select = in->select;
    a.thr_num = in->thr_num;
    a.thr_den = in->thr_den;
    a.free_blocks = in->free_blocks;
    a.num_free = in->num_free;
    a.new_bt_offsets = out->new_bt_offsets;
    a.new_bt_blocks = out->new_bt_blocks;
    a.new_tt_slots = out->new_tt_slots;
    a.freed_blocks = out->freed_blocks;
    a.out_status = out->req_status;
    a.out_counts = out->counts;
    a.req_n = ctx->req_n;
    a.part_n = ctx->part_n;
    a.req_dst_base = ctx->req_dst_base;
    a.req_freed_base = ctx->req_freed_base;
    a.req_status = ctx->req_status;
    a.dst_src = ctx->dst_src;
    a.dst_blocks = ctx->dst_blocks;
    a.counts = ctx->counts;
    a.S = ctx->cfg.block_size;
    a.num_blocks = ctx->cfg.num_blocks;
    a.max_requests = ctx->cfg.max_requests;
    a.cap_dst_blocks = ctx->cap_dst_blocks;
    a.max_free_blocks = ctx->cfg.max_free_blocks;
    a.slots_per_layer = ctx->slots_per_layer;
    a.max_tokens = ctx->cfg.max_tokens;
    a.max_table_blocks = ctx->cfg.max_table_blocks;

    VTK_CUDA(ctx, cudaMemsetAsync(ctx->counts, 0, sizeof(vtoken_counts), st));
    const dim3 parts(ctx->cfg.max_requests * PLAN_PARTS);
    VTK_CUDA(ctx, vtk_launch_dependent(plan_count_kernel, parts, dim3(PLAN_NT), 0, st, a));
    VTK_CUDA(ctx, vtk_launch_dependent(plan_scan_kernel, dim3(1), dim3(SCAN_NT), 0, st, a));
    VTK_CUDA(ctx, vtk_launch_dependent(plan_assign_kernel, parts, dim3(PLAN_NT), 0, st, a));
    VTK_CUDA(ctx, cudaGetLastError());
    return VTOKEN_OK;
}
