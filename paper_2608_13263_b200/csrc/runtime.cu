// Device-side token-table runtime: the interfaces of the token table (Sec. 3.2 of the paper:
// evict_token, sync_new_tokens, apply_moves) as batch kernels over device-resident tables.
// The slot-mapping build (Sec. 3.4) lives with the logical gather, whose planner it shares.
//
// A request's token table occupies tt_slots[tt_offsets[r] .. tt_offsets[r+1]) -- its capacity;
// tt_len[r] entries are registered, the rest hold -1 / keep 0, which every other kernel of the
// library already treats as "not live".  phys_len[r] is the append position in its block list.
#include "common.cuh"

namespace {

constexpr int RT_NT = 256;

__device__ __forceinline__ int rt_requests(const int32_t *num_requests, int max_requests)
{
    int R = *num_requests;
    return R < 0 ? 0 : (R > max_requests ? max_requests : R);
}

// Per-block liveness that the counted variants keep current (Sec. 3.3.1 of the paper).
struct Liveness {
    int32_t *n_b;                      // [num_blocks] live tokens per physical block
    unsigned long long *live_total;    // sum of n_b, or NULL
    const int32_t *tt_slots;           // evict only: where the victim's K/V sits
    int64_t slots;                     // num_blocks * S
    int32_t S;
};

// Clears one byte of the keep mask atomically and returns its previous value, so that a token
// named twice in a batch (or already evicted) is counted once.  The mask must be allocated in
// multiples of four bytes: the atomic works on the aligned word that holds the byte.
__device__ __forceinline__ uint32_t clear_keep_byte(uint8_t *p)
{
    const uintptr_t a = (uintptr_t)p;
    const unsigned shift = (unsigned)(a & 3u) * 8u;
    const unsigned old = atomicAnd((unsigned *)(a & ~(uintptr_t)3), ~(0xFFu << shift));
    return (old >> shift) & 0xFFu;
}

// evict_token over a batch of victims: metadata only, the KV bytes stay where they are
template <bool COUNTED>
__global__ void __launch_bounds__(RT_NT) evict_kernel(const int32_t *num_victims, int32_t max_victims,
                                                      const int32_t *victim_req, const int32_t *victim_tok,
                                                      const int32_t *num_requests, int32_t max_requests,
                                                      const int32_t *tt_offsets, const int32_t *tt_len,
                                                      uint8_t *keep, vtoken_counts *counts, Liveness lv)
{
    vtk_release_successor();
    vtk_wait_for_predecessor();
    int n = *num_victims;
    n = n < 0 ? 0 : (n > max_victims ? max_victims : n);
    const int R = rt_requests(num_requests, max_requests);
    bool bad = false;
    for (int i = blockIdx.x * RT_NT + threadIdx.x; i < n; i += gridDim.x * RT_NT) {
        const int r = victim_req[i], t = victim_tok[i];
        if (r < 0 || r >= R || t < 0 || t >= tt_len[r]) { bad = true; continue; }
        const int64_t e = (int64_t)tt_offsets[r] + t;
        if (COUNTED) {
            // the block loses a live token only if this thread is the one that deactivates it
            const int32_t s = lv.tt_slots[e];
            if (clear_keep_byte(keep + e) != 0 && s >= 0 && (int64_t)s < lv.slots) {
                atomicSub(&lv.n_b[s / lv.S], 1);
                if (lv.live_total) atomicAdd(lv.live_total, ~0ull);          // minus one
            }
        } else {
            keep[e] = 0;
        }
    }
    if (bad || (threadIdx.x == 0 && blockIdx.x == 0 && *num_victims > max_victims))
        atomicOr(&counts->error_flags, VTOKEN_FLAG_BAD_VICTIM);
}

// sync_new_tokens: one CTA per request; the tokens it can register are a prefix of the ones asked
// for (table capacity and block-list room only shrink it), so the count has a closed form.
template <bool COUNTED>
__global__ void __launch_bounds__(RT_NT) sync_kernel(const int32_t *num_requests, int32_t max_requests, int32_t S,
                                                     const int32_t *tt_offsets, int32_t *tt_slots, uint8_t *keep,
                                                     int32_t *tt_len, int32_t *phys_len, const int32_t *bt_offsets,
                                                     const int32_t *bt_blocks, const int32_t *new_len,
                                                     int32_t num_blocks, vtoken_counts *counts, Liveness lv)
{
    vtk_release_successor();
    vtk_wait_for_predecessor();
    const int r = blockIdx.x;
    if (r >= rt_requests(num_requests, max_requests)) return;
    const int64_t base = tt_offsets[r];
    const int cap = tt_offsets[r + 1] - tt_offsets[r];
    const int len = tt_len[r], phys = phys_len[r];
    const int b0 = bt_offsets[r];
    const long long room = (long long)(bt_offsets[r + 1] - b0) * S;
    const int want = new_len[r] - len;
    if (want <= 0) return;
    long long can = want;
    if (can > cap - len) can = cap - len;
    if (can > room - phys) can = room - phys;
    if (can < 0) can = 0;
    uint32_t flags = can < want ? VTOKEN_FLAG_APPEND_STOPPED : 0u;
    int counted = 0;
    for (int i = threadIdx.x; i < (int)can; i += RT_NT) {
        const int p = phys + i;                              // position in the block list
        const int blk = bt_blocks[b0 + p / S];
        const bool ok = blk >= 0 && blk < num_blocks;
        if (!ok) flags |= VTOKEN_FLAG_BAD_BLOCK;             // registered without a physical copy: slot -1, not kept
        tt_slots[base + len + i] = ok ? blk * S + p % S : -1;   // slot = block_id * S + offset
        keep[base + len + i] = ok ? 1 : 0;
        if (COUNTED && ok) {                                 // one more live token in that block
            atomicAdd(&lv.n_b[blk], 1);
            ++counted;
        }
    }
    if (COUNTED && lv.live_total) {
#pragma unroll
        for (int d = 16; d > 0; d >>= 1) counted += __shfl_down_sync(0xffffffffu, counted, d);
        if (vtk_lane() == 0 && counted) atomicAdd(lv.live_total, (unsigned long long)counted);
    }
    __syncthreads();     // every thread has read tt_len / phys_len before they change
    if (threadIdx.x == 0) {
        tt_len[r] = len + (int)can;
        phys_len[r] = phys + (int)can;
    }
    if (flags) atomicOr(&counts->error_flags, flags);
}

// apply_moves: commit of a repack.  Entries take their new slot, liveness follows the slot, a
// repacked request appends behind the tokens the repack moved: its block list is now the blocks
// that stayed followed by the destination blocks, which the moved tokens fill densely.
__global__ void __launch_bounds__(RT_NT) apply_moves_kernel(const int32_t *num_requests, int32_t max_requests,
                                                            int32_t S, const int32_t *tt_offsets, int32_t *tt_slots,
                                                            uint8_t *keep, int32_t *phys_len,
                                                            const int32_t *new_tt_slots, const int32_t *req_status,
                                                            const int32_t *new_bt_offsets, const int32_t *append_pos)
{
    vtk_release_successor();
    vtk_wait_for_predecessor();
    const int r = blockIdx.x;
    if (r >= rt_requests(num_requests, max_requests)) return;
    const int64_t t0 = tt_offsets[r], t1 = tt_offsets[r + 1];
    int n = 0, moved = 0;                          // entries with a slot; entries whose slot changed
    constexpr int U = 4;                           // loads of four entries in flight before the first store
    for (int64_t tb = t0 + threadIdx.x; tb < t1; tb += (int64_t)RT_NT * U) {
        int32_t s_new[U], s_old[U];
#pragma unroll
        for (int u = 0; u < U; ++u) {
            const int64_t t = tb + (int64_t)u * RT_NT;
            s_new[u] = t < t1 ? __ldg(new_tt_slots + t) : -1;
            s_old[u] = t < t1 ? tt_slots[t] : -1;
        }
#pragma unroll
        for (int u = 0; u < U; ++u) {
            const int64_t t = tb + (int64_t)u * RT_NT;
            if (t < t1) {
                moved += s_new[u] >= 0 && s_new[u] != s_old[u];       // destinations are never sources
                tt_slots[t] = s_new[u];
                keep[t] = s_new[u] >= 0 ? 1 : 0;
                n += s_new[u] >= 0;
            }
        }
    }
    __shared__ int warp_n[RT_NT / 32], warp_m[RT_NT / 32];
#pragma unroll
    for (int d = 16; d > 0; d >>= 1) {
        n += __shfl_down_sync(0xffffffffu, n, d);
        moved += __shfl_down_sync(0xffffffffu, moved, d);
    }
    if (vtk_lane() == 0) {
        warp_n[threadIdx.x >> 5] = n;
        warp_m[threadIdx.x >> 5] = moved;
    }
    __syncthreads();
    if (threadIdx.x == 0 && phys_len != nullptr && req_status != nullptr && req_status[r] == VTOKEN_REPACKED) {
        int sn = 0, sm = 0;
        for (int w = 0; w < RT_NT / 32; ++w) { sn += warp_n[w]; sm += warp_m[w]; }
        if (append_pos != nullptr) {
            phys_len[r] = append_pos[r];           // worked out by the repack in waves, wave by wave
        } else if (new_bt_offsets != nullptr) {
            const int blocks = new_bt_offsets[r + 1] - new_bt_offsets[r];
            phys_len[r] = (blocks - (sm + S - 1) / S) * S + sm;
        } else {
            phys_len[r] = sn;                      // whole-request plans: nothing stayed
        }
    }
}

}  // namespace

extern "C" {

int vtoken_evict_tokens(vtoken_ctx *ctx, const int32_t *num_victims, int32_t max_victims,
                        const int32_t *victim_req, const int32_t *victim_tok, const int32_t *num_requests,
                        const int32_t *tt_offsets, const int32_t *tt_len, uint8_t *keep, void *cuda_stream)
{
    if (!ctx || !num_victims || !victim_req || !victim_tok || !num_requests || !tt_offsets || !tt_len || !keep)
        return VTOKEN_EINVAL;
    if (max_victims < 0) return VTOKEN_EINVAL;
    if (max_victims == 0) return VTOKEN_OK;
    int grid = (max_victims + RT_NT - 1) / RT_NT;
    if (grid > ctx->num_sms * 8) grid = ctx->num_sms * 8;
    VTK_CUDA(ctx, vtk_launch_dependent(ctx, evict_kernel<false>, dim3(grid), dim3(RT_NT), 0, (cudaStream_t)cuda_stream,
                                       num_victims, max_victims, victim_req, victim_tok, num_requests,
                                       ctx->cfg.max_requests, tt_offsets, tt_len, keep, ctx->rt_counts, Liveness{}));
    VTK_CUDA(ctx, cudaGetLastError());
    return VTOKEN_OK;
}

int vtoken_evict_tokens_counted(vtoken_ctx *ctx, const int32_t *num_victims, int32_t max_victims,
                                const int32_t *victim_req, const int32_t *victim_tok, const int32_t *num_requests,
                                const int32_t *tt_offsets, const int32_t *tt_len, const int32_t *tt_slots,
                                uint8_t *keep, int32_t *n_b, int64_t *live_total, void *cuda_stream)
{
    if (!ctx || !num_victims || !victim_req || !victim_tok || !num_requests || !tt_offsets || !tt_len || !tt_slots ||
        !keep || !n_b)
        return VTOKEN_EINVAL;
    if (max_victims < 0 || ((uintptr_t)keep & 3)) return VTOKEN_EINVAL;
    if (max_victims == 0) return VTOKEN_OK;
    int grid = (max_victims + RT_NT - 1) / RT_NT;
    if (grid > ctx->num_sms * 8) grid = ctx->num_sms * 8;
    const Liveness lv{n_b, (unsigned long long *)live_total, tt_slots, ctx->slots_per_layer, ctx->cfg.block_size};
    VTK_CUDA(ctx, vtk_launch_dependent(ctx, evict_kernel<true>, dim3(grid), dim3(RT_NT), 0, (cudaStream_t)cuda_stream,
                                       num_victims, max_victims, victim_req, victim_tok, num_requests,
                                       ctx->cfg.max_requests, tt_offsets, tt_len, keep, ctx->rt_counts, lv));
    VTK_CUDA(ctx, cudaGetLastError());
    return VTOKEN_OK;
}

int vtoken_sync_new_tokens(vtoken_ctx *ctx, const int32_t *num_requests, const int32_t *tt_offsets,
                           int32_t *tt_slots, uint8_t *keep, int32_t *tt_len, int32_t *phys_len,
                           const int32_t *bt_offsets, const int32_t *bt_blocks, const int32_t *new_len,
                           void *cuda_stream)
{
    if (!ctx || !num_requests || !tt_offsets || !tt_slots || !keep || !tt_len || !phys_len || !bt_offsets ||
        !bt_blocks || !new_len)
        return VTOKEN_EINVAL;
    VTK_CUDA(ctx, vtk_launch_dependent(ctx, sync_kernel<false>,
                                       dim3(ctx->cfg.max_requests), dim3(RT_NT), 0, (cudaStream_t)cuda_stream,
                                       num_requests, ctx->cfg.max_requests, ctx->cfg.block_size, tt_offsets, tt_slots,
                                       keep, tt_len, phys_len, bt_offsets, bt_blocks, new_len, ctx->cfg.num_blocks,
                                       ctx->rt_counts, Liveness{}));
    VTK_CUDA(ctx, cudaGetLastError());
    return VTOKEN_OK;
}

int vtoken_sync_new_tokens_counted(vtoken_ctx *ctx, const int32_t *num_requests, const int32_t *tt_offsets,
                                   int32_t *tt_slots, uint8_t *keep, int32_t *tt_len, int32_t *phys_len,
                                   const int32_t *bt_offsets, const int32_t *bt_blocks, const int32_t *new_len,
                                   int32_t *n_b, int64_t *live_total, void *cuda_stream)
{
    if (!ctx || !num_requests || !tt_offsets || !tt_slots || !keep || !tt_len || !phys_len || !bt_offsets ||
        !bt_blocks || !new_len || !n_b)
        return VTOKEN_EINVAL;
    const Liveness lv{n_b, (unsigned long long *)live_total, nullptr, ctx->slots_per_layer, ctx->cfg.block_size};
    VTK_CUDA(ctx, vtk_launch_dependent(ctx, sync_kernel<true>,
                                       dim3(ctx->cfg.max_requests), dim3(RT_NT), 0, (cudaStream_t)cuda_stream,
                                       num_requests, ctx->cfg.max_requests, ctx->cfg.block_size, tt_offsets, tt_slots,
                                       keep, tt_len, phys_len, bt_offsets, bt_blocks, new_len, ctx->cfg.num_blocks,
                                       ctx->rt_counts, lv));
    VTK_CUDA(ctx, cudaGetLastError());
    return VTOKEN_OK;
}

int vtoken_apply_moves(vtoken_ctx *ctx, const int32_t *num_requests, const int32_t *tt_offsets,
                       int32_t *tt_slots, uint8_t *keep, int32_t *phys_len, const int32_t *new_tt_slots,
                       const int32_t *req_status, const int32_t *new_bt_offsets, const int32_t *append_pos,
                       void *cuda_stream)
{
    if (!ctx || !num_requests || !tt_offsets || !tt_slots || !keep || !new_tt_slots) return VTOKEN_EINVAL;
    if (phys_len && !req_status) return VTOKEN_EINVAL;
    VTK_CUDA(ctx, vtk_launch_dependent(ctx, apply_moves_kernel,
                                       dim3(ctx->cfg.max_requests), dim3(RT_NT), 0, (cudaStream_t)cuda_stream,
                                       num_requests, ctx->cfg.max_requests, ctx->cfg.block_size, tt_offsets, tt_slots,
                                       keep, phys_len, new_tt_slots, req_status, new_bt_offsets, append_pos));
    VTK_CUDA(ctx, cudaGetLastError());
    return VTOKEN_OK;
}

}  // extern "C"
