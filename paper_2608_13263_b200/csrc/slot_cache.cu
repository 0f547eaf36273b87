// Cached slot-translation arrays (Sec. 3.2 last paragraph and Sec. 4 of the paper): the slots of a
// request's active tokens in token-id order, kept on the device and refreshed only after
// structural changes.  A request that merely grew gets its new entries appended; a request that
// saw an eviction or a relocation is rebuilt; every other request costs one CTA that reads three
// words and leaves.
#include "common.cuh"

namespace {

constexpr int SC_NT = 512;

__device__ __forceinline__ int sc_requests(const int32_t *num_requests, int max_requests)
{
    int R = *num_requests;
    return R < 0 ? 0 : (R > max_requests ? max_requests : R);
}

__global__ void __launch_bounds__(256) slot_cache_mark_kernel(uint8_t *dirty, const int32_t *num_victims,
                                                              int32_t max_victims, const int32_t *victim_req,
                                                              const int32_t *req_status, const int32_t *num_requests,
                                                              int32_t max_requests)
{
    vtk_release_successor();
    vtk_wait_for_predecessor();
    const int R = sc_requests(num_requests, max_requests);
    const int gtid = blockIdx.x * blockDim.x + threadIdx.x, gsz = gridDim.x * blockDim.x;
    if (victim_req != nullptr && num_victims != nullptr) {
        int n = *num_victims;
        n = n < 0 ? 0 : (n > max_victims ? max_victims : n);
        for (int i = gtid; i < n; i += gsz) {
            const int r = victim_req[i];
            if (r >= 0 && r < R) dirty[r] = 1;          // same value from every writer
        }
    }
    if (req_status != nullptr)
        for (int r = gtid; r < R; r += gsz)
            if (req_status[r] == VTOKEN_REPACKED) dirty[r] = 1;
}

__global__ void __launch_bounds__(SC_NT) slot_cache_update_kernel(const int32_t *num_requests, int32_t max_requests,
                                                                  const int32_t *tt_offsets, const int32_t *tt_slots,
                                                                  const uint8_t *keep, const int32_t *tt_len,
                                                                  uint8_t *dirty, int32_t *cache_slots,
                                                                  int32_t *cache_ids, int32_t *cache_len,
                                                                  int32_t *cache_seen, int32_t *stats,
                                                                  int64_t slots_per_layer, vtoken_counts *counts)
{
    vtk_release_successor();
    vtk_wait_for_predecessor();
    __shared__ int warp_sums[SC_NT / 32 + 1];
    const int r = blockIdx.x;
    if (r >= sc_requests(num_requests, max_requests)) return;
    const int64_t base = tt_offsets[r];
    const int cap = tt_offsets[r + 1] - tt_offsets[r];
    int len = tt_len[r];
    len = len < 0 ? 0 : (len > cap ? cap : len);
    const bool rebuild = dirty[r] != 0;
    int first, fill;
    if (rebuild) {
        first = 0;
        fill = 0;
    } else {
        first = cache_seen[r];
        fill = cache_len[r];
        if (first < 0) first = 0;
        if (len <= first) return;                        // nothing changed: the whole CTA leaves
    }
    const int tid = threadIdx.x;
    bool bad = false;
    for (int tb = first; tb < len; tb += SC_NT) {
        const int t = tb + tid;
        int32_t slot = -1;
        bool live = false;
        if (t < len) {
            slot = tt_slots[base + t];
            live = vtk_live(slot, keep, base + t, slots_per_layer, bad);
        }
        int total;
        const int i = fill + vtk_block_rank<SC_NT>(live, warp_sums, total);
        if (live) {
            cache_slots[base + i] = slot;
            if (cache_ids != nullptr) cache_ids[base + i] = t;
        }
        fill += total;
    }
    __syncthreads();                                     // every thread has read the request's state
    if (tid == 0) {
        cache_len[r] = fill;
        cache_seen[r] = len;
        dirty[r] = 0;
        if (stats != nullptr) atomicAdd(&stats[rebuild ? 0 : 1], 1);
    }
    if (bad) atomicOr(&counts->error_flags, VTOKEN_FLAG_BAD_SLOT);
}

}  // namespace

extern "C" {

int vtoken_slot_cache_mark(vtoken_ctx *ctx, uint8_t *dirty, const int32_t *num_victims, int32_t max_victims,
                           const int32_t *victim_req, const int32_t *req_status, const int32_t *num_requests,
                           void *cuda_stream)
{
    if (!ctx || !dirty || !num_requests || max_victims < 0) return VTOKEN_EINVAL;
    if (max_victims > 0 && (!victim_req || !num_victims)) return VTOKEN_EINVAL;
    const int64_t span = max_victims > ctx->cfg.max_requests ? max_victims : ctx->cfg.max_requests;
    int grid = (int)((span + 255) / 256);
    if (grid > ctx->num_sms * 8) grid = ctx->num_sms * 8;
    VTK_CUDA(ctx, vtk_launch_dependent(ctx, slot_cache_mark_kernel, dim3(grid), dim3(256), 0, (cudaStream_t)cuda_stream,
                                       dirty,
                                       max_victims > 0 ? num_victims : nullptr, max_victims,
                                       max_victims > 0 ? victim_req : nullptr, req_status, num_requests,
                                       ctx->cfg.max_requests));
    VTK_CUDA(ctx, cudaGetLastError());
    return VTOKEN_OK;
}

int vtoken_slot_cache_update(vtoken_ctx *ctx, const int32_t *num_requests, const int32_t *tt_offsets,
                             const int32_t *tt_slots, const uint8_t *keep, const int32_t *tt_len, uint8_t *dirty,
                             int32_t *cache_slots, int32_t *cache_ids, int32_t *cache_len, int32_t *cache_seen,
                             int32_t *stats, void *cuda_stream)
{
    if (!ctx || !num_requests || !tt_offsets || !tt_slots || !tt_len || !dirty || !cache_slots || !cache_len ||
        !cache_seen)
        return VTOKEN_EINVAL;
    cudaStream_t st = (cudaStream_t)cuda_stream;
    if (stats) VTK_CUDA(ctx, cudaMemsetAsync(stats, 0, 2 * sizeof(int32_t), st));
    VTK_CUDA(ctx, vtk_launch_dependent(ctx, slot_cache_update_kernel,
                                       dim3(ctx->cfg.max_requests), dim3(SC_NT), 0, st, num_requests,
                                       ctx->cfg.max_requests, tt_offsets, tt_slots, keep, tt_len, dirty, cache_slots,
                                       cache_ids, cache_len, cache_seen, stats, ctx->slots_per_layer, ctx->rt_counts));
    VTK_CUDA(ctx, cudaGetLastError());
    return VTOKEN_OK;
}

}  // extern "C"
