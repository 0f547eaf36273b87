// Input-precondition checker: every violated precondition of the planner's inputs as a bit
// (unique mapping I2 of the paper's Sec. 3.5 among them).  A debugging aid for integrators: the
// fast path assumes these preconditions and does not check them.  Each bit is defined by
// counting, so the parallel evaluation below gives the same answer in any order.
#include "common.cuh"

namespace {

constexpr int CK_NT = 256;
constexpr int CK_PARTS = VTK_PLAN_PARTS;

enum : uint32_t {
    CK_OFFSETS = 1u, CK_BLOCK_RANGE = 2u, CK_BLOCK_TWICE = 4u, CK_FREE_RANGE = 8u, CK_FREE_TWICE_OR_HELD = 16u,
    CK_SLOT_RANGE = 32u, CK_FOREIGN_SLOT = 64u, CK_SLOT_TWICE = 128u
};
// owner[b]: -1 nobody, r >= 0 held by request r only, -2 on the free list, -3 held by several requests
constexpr int32_t OWNER_NONE = -1, OWNER_FREE = -2, OWNER_SHARED = -3;

struct CheckArgs {
    const int32_t *num_requests, *bt_offsets, *bt_blocks, *tt_offsets, *tt_slots, *free_blocks, *num_free;
    const uint8_t *protect;
    int32_t *owner;
    uint32_t *slot_bits, *out_bits;
    int32_t max_requests, max_free_blocks, num_blocks, S;
    int64_t slots;
};

__device__ __forceinline__ int ck_requests(const CheckArgs &a)
{
    int R = *a.num_requests;
    return R < 0 ? 0 : (R > a.max_requests ? a.max_requests : R);
}

__global__ void __launch_bounds__(CK_NT) check_offsets_kernel(CheckArgs a)
{
    const int R = ck_requests(a);
    bool bad = false;
    for (int r = blockIdx.x * CK_NT + threadIdx.x; r < R; r += gridDim.x * CK_NT)
        bad |= a.bt_offsets[r + 1] < a.bt_offsets[r] || a.tt_offsets[r + 1] < a.tt_offsets[r];
    if (bad) atomicOr(a.out_bits, CK_OFFSETS);
}

// one CTA per request: who holds which block
__global__ void __launch_bounds__(CK_NT) check_blocks_kernel(CheckArgs a)
{
    const int r = blockIdx.x;
    if (r >= ck_requests(a) || (*a.out_bits & CK_OFFSETS)) return;     // ranges are meaningless then
    uint32_t f = 0;
    for (int j = a.bt_offsets[r] + threadIdx.x; j < a.bt_offsets[r + 1]; j += CK_NT) {
        const int32_t b = a.bt_blocks[j];
        if (b < 0 || b >= a.num_blocks) { f |= CK_BLOCK_RANGE; continue; }
        const int32_t old = atomicCAS(&a.owner[b], OWNER_NONE, r);
        if (old == OWNER_NONE) continue;
        if (!(a.protect && a.protect[b])) f |= CK_BLOCK_TWICE;
        if (old != r && old != OWNER_SHARED) atomicExch(&a.owner[b], OWNER_SHARED);
    }
    if (f) atomicOr(a.out_bits, f);
}

__global__ void __launch_bounds__(CK_NT) check_free_kernel(CheckArgs a)
{
    if (*a.out_bits & CK_OFFSETS) return;
    int nf = *a.num_free;
    nf = nf < 0 ? 0 : (nf > a.max_free_blocks ? a.max_free_blocks : nf);
    uint32_t f = 0;
    for (int j = blockIdx.x * CK_NT + threadIdx.x; j < nf; j += gridDim.x * CK_NT) {
        const int32_t b = a.free_blocks[j];
        if (b < 0 || b >= a.num_blocks) { f |= CK_FREE_RANGE; continue; }
        if (atomicCAS(&a.owner[b], OWNER_NONE, OWNER_FREE) != OWNER_NONE) f |= CK_FREE_TWICE_OR_HELD;
    }
    if (f) atomicOr(a.out_bits, f);
}

// one CTA per request part: every slot in range, in a block of its request, named once
__global__ void __launch_bounds__(CK_NT) check_slots_kernel(CheckArgs a)
{
    const int r = blockIdx.x / CK_PARTS, c = blockIdx.x % CK_PARTS;
    if (r >= ck_requests(a) || (*a.out_bits & CK_OFFSETS)) return;
    const int64_t t0 = a.tt_offsets[r], t1 = a.tt_offsets[r + 1];
    const int64_t per = (t1 - t0 + CK_PARTS - 1) / CK_PARTS;
    const int64_t p0 = min(t1, t0 + c * per), p1 = min(t1, p0 + per);
    uint32_t f = 0;
    for (int64_t t = p0 + threadIdx.x; t < p1; t += CK_NT) {
        const int32_t s = a.tt_slots[t];
        if (s < 0) continue;
        if ((int64_t)s >= a.slots) { f |= CK_SLOT_RANGE; continue; }
        const int32_t b = s / a.S;
        const int32_t o = a.owner[b];
        if (o == OWNER_NONE || o == OWNER_FREE || (o >= 0 && o != r)) f |= CK_FOREIGN_SLOT;
        const uint32_t bit = 1u << (s & 31);
        if ((atomicOr(&a.slot_bits[s >> 5], bit) & bit) && !(a.protect && a.protect[b])) f |= CK_SLOT_TWICE;
    }
    if (f) atomicOr(a.out_bits, f);
}

}  // namespace

extern "C" int vtoken_check_tables(vtoken_ctx *ctx, const vtoken_plan_in *in, const uint8_t *protect,
                                   uint32_t *out_bits, void *cuda_stream)
{
    if (!ctx || !in || !out_bits) return VTOKEN_EINVAL;
    if (!in->num_requests || !in->bt_offsets || !in->bt_blocks || !in->tt_offsets || !in->tt_slots ||
        !in->free_blocks || !in->num_free)
        return VTOKEN_EINVAL;
    cudaStream_t st = (cudaStream_t)cuda_stream;
    CheckArgs a;
    a.num_requests = in->num_requests;
    a.bt_offsets = in->bt_offsets;
    a.bt_blocks = in->bt_blocks;
    a.tt_offsets = in->tt_offsets;
    a.tt_slots = in->tt_slots;
    a.free_blocks = in->free_blocks;
    a.num_free = in->num_free;
    a.protect = protect;
    a.owner = ctx->n_b;
    a.slot_bits = ctx->slot_bits;
    a.out_bits = out_bits;
    a.max_requests = ctx->cfg.max_requests;
    a.max_free_blocks = ctx->cfg.max_free_blocks;
    a.num_blocks = ctx->cfg.num_blocks;
    a.S = ctx->cfg.block_size;
    a.slots = ctx->slots_per_layer;
    const int R = ctx->cfg.max_requests;
    VTK_CUDA(ctx, cudaMemsetAsync(out_bits, 0, sizeof(uint32_t), st));
    VTK_CUDA(ctx, cudaMemsetAsync(ctx->n_b, 0xFF, sizeof(int32_t) * (size_t)ctx->cfg.num_blocks, st));   // OWNER_NONE
    VTK_CUDA(ctx, cudaMemsetAsync(ctx->slot_bits, 0, sizeof(uint32_t) * (size_t)((ctx->slots_per_layer + 31) / 32), st));
    check_offsets_kernel<<<(R + CK_NT - 1) / CK_NT, CK_NT, 0, st>>>(a);
    check_blocks_kernel<<<R, CK_NT, 0, st>>>(a);
    int fgrid = (ctx->cfg.max_free_blocks + CK_NT - 1) / CK_NT;
    fgrid = fgrid < 1 ? 1 : (fgrid > ctx->num_sms * 8 ? ctx->num_sms * 8 : fgrid);
    check_free_kernel<<<fgrid, CK_NT, 0, st>>>(a);
    check_slots_kernel<<<R * CK_PARTS, CK_NT, 0, st>>>(a);
    VTK_CUDA(ctx, cudaGetLastError());
    return VTOKEN_OK;
}
