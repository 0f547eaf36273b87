// Internal definitions shared by the translation units of libvtoken (never installed).
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

#include <type_traits>

#include "vtoken.h"

#define VTK_PLAN_PARTS 8   // token ranges per request in the planner

// ---------------------------------------------------------------------------------------
// Context: configuration, derived sizes and every scratch buffer (allocated once).
// ---------------------------------------------------------------------------------------
struct vtoken_ctx {
    vtoken_config cfg;
    int64_t row_bytes;         // H * D * elem_bytes
    int64_t layer_stride;      // bytes between layers
    int64_t slots_per_layer;   // NB * S
    int32_t cap_dst_blocks;    // destination blocks a plan can ever use
    int device, num_sms;
    int last_cuda_error;
    bool has_plan;

    // planner scratch (DEVICE)
    int32_t *req_n;            // [max_requests] live tokens (partial planner)
    int32_t *plan_header;      // [4] R, T, num_free, first entry as the first kernel of a plan read them (one load downstream)
    int32_t *part_n;           // [max_requests * VTK_PLAN_PARTS] live tokens per request part: only the context-free
                               // gather entry point (per-request index kernels) sets it, from its static scratch
    int32_t *req_dst_base;     // [max_requests] first destination block (index into the free list)
    int32_t *req_freed_base;   // [max_requests] first entry in freed_blocks
    int32_t *req_status;       // [max_requests]
    int32_t *dst_src;          // [cap_dst_blocks * S] inverse plan: source slot of each destination slot, -1 = none
    int32_t *dst_blocks;       // [cap_dst_blocks] physical id of each destination block, -1 = skip
    vtoken_counts *counts;     // one struct: counts of the last plan, flags of the plan and its copy
    vtoken_counts *rt_counts;  // one struct, only error_flags is used: flags raised by every call outside plan / repack
                               // (logical gather, slot mapping, digest, token-table runtime, slot cache).  Those calls
                               // belong to the compute stream and may overlap a plan in flight on a side stream, whose
                               // scan kernel stores `counts` as a whole
    int32_t *tile_n;           // [ceil(max_tokens / 1024) + 1] live tokens per tile of the token table, then scanned
    int32_t *req_part;         // [max_requests + 1] live tokens between a request's tile start and its first entry
    int32_t *req_before;       // [max_requests + 1] live (partial planner: moving) tokens of the table before the request's first entry
    int32_t *tile_mov, *tile_shared;   // [like tile_n] partial planner: moving tokens / live tokens in protected blocks per tile
    int32_t *part_mov;         // [max_requests + 1] partial planner: like req_part, moving tokens

    // partial-plan scratch (DEVICE)
    int32_t *req_ns;           // [max_requests] source blocks of the request
    int32_t *req_nsrc;         // [max_requests] live tokens in its source blocks
    int32_t *n_b;              // [num_blocks] live tokens per physical block
    uint8_t *blk_src;          // [num_blocks] 1 = the block is a source of its request (behind n_b in one allocation)
    int32_t *part_shared;      // [max_requests + 1] like req_part, live tokens in protected blocks
    int32_t *req_shared;       // [max_requests] protected entries of the request's block table
    int32_t *req_detach;       // [max_requests] 1 = the request leaves its protected blocks (copy-on-write detach)
    int32_t *req_rel_base;     // [max_requests] first entry in released_blocks
    int plan_form;             // whole-request planner of this context: 1 three kernels (plan.cu), 2 two kernels (plan_small.cu)
    unsigned long long *cow;   // [2 * max_table_blocks] detach per shared block: every request's hash from a protected
                               // block of its table to its own live tokens there ((block id + 1) << 32 | count)
    uint32_t *slot_bits;       // [ceil(num_blocks * S / 32)] one bit per slot (vtoken_check_tables)

    // gather_logical scratch (DEVICE)
    int32_t *g_src;            // [max_tokens] source slot of each output row
    int32_t *g_total;          // [1] output rows
    int32_t *g_ids;            // [max_tokens] logical id of each output row (digest)
    int32_t *g_req;            // [max_tokens] request of each output row (digest)
    int32_t *g_offsets;        // [max_requests + 1] first output row of each request (digest)
    unsigned int *g_ticket;    // [2] work tickets of the gather's row copy (zero between launches)
    int32_t *g_tile_n, *g_req_part, *g_req_before;   // like tile_n / req_part / req_before, owned by the gather family
                                                     // (logical gather, slot mapping, digest): these calls run on the
                                                     // compute stream while a plan may be in flight on a side stream

    // device staging of vtoken_repack_host (DEVICE), allocated on first use
    struct {
        bool ready;
        int32_t *num_requests, *num_free;
        int32_t *bt_offsets, *bt_blocks, *tt_offsets, *tt_slots, *free_blocks;
        uint8_t *keep, *select;
        uint8_t *protect;              // [num_blocks], vtoken_repack_host_partial only (allocated on first use)
        int32_t *released_blocks;      // [max_table_blocks], vtoken_repack_host_partial with a detach threshold (first use)
        int32_t *new_bt_offsets, *new_bt_blocks, *new_tt_slots, *freed_blocks, *req_status;
        vtoken_counts *counts;
        int32_t *h_scalars;            // HOST, pinned mirror of the small inputs of the call in flight: {num_requests,
                                       // num_free}, bt_offsets, tt_offsets, select (same layout as on the device)
        int64_t small_ints;            // its size in 32-bit words
        vtoken_counts *h_counts;       // HOST, pinned: landing place of the counts
        cudaStream_t aux;              // carries the output copies while the copy kernel runs
        cudaEvent_t planned, copied;   // plan done on the caller's stream; outputs copied on aux
    } stage;
    int64_t scratch_bytes;

    // launch shape of the copy kernel
    int copy_variant;          // 1 register path, 2 bulk-copy path
    int copy_ctas, copy_threads, copy_smem;
    int64_t wait_limit_ns, stall_item;   // bound of in-kernel waits; test hook (see copy.cu)
    bool copy_dynamic;         // bulk path: items handed out by a ticket counter instead of fixed shares
    int copy_chunk;            // consecutive items per ticket
    unsigned int *copy_ticket; // [2] DEVICE: next item, finished warps (zero between launches)
    int bulk_warps, bulk_stages, bulk_rows, bulk_depth, bulk_ahead;   // bulk path: warps per CTA, ring size, rows per item, loads ahead
};

// ---------------------------------------------------------------------------------------
// Device arrays as the kernels see them.  In the production build vtk_arr<T> is a bare pointer.
// In the checked build (-DVTOKEN_CHECKED, libvtoken_checked.so) it also carries the number of
// elements the array holds and the address of a flag word of the context: an index outside
// [0, n) raises VTOKEN_FLAG_CHECK_FAILED there and the access goes to a dummy element instead
// -- it is skipped, nothing faults, the kernel goes on.  The tests run against both builds and
// require the flag to stay clear: the place of a memory sanitizer, which also catches what a
// comparison of results cannot (a read beyond an array, a stray write into scratch).
// ---------------------------------------------------------------------------------------
#ifdef VTOKEN_CHECKED
static __device__ __align__(16) unsigned long long vtk_dummy[4];
#endif

template <typename T>
struct vtk_arr {
    T *p;
#ifdef VTOKEN_CHECKED
    int64_t n;
    uint32_t *flag;
    __host__ __device__ vtk_arr() : p(nullptr), n(0), flag(nullptr) {}
    __host__ __device__ vtk_arr(T *p_, int64_t n_, uint32_t *flag_) : p(p_), n(n_), flag(flag_) {}
    __device__ __forceinline__ T &bad() const
    {
        if (flag) atomicOr(flag, (uint32_t)VTOKEN_FLAG_CHECK_FAILED);
        return *reinterpret_cast<T *>(vtk_dummy);
    }
    __device__ __forceinline__ T &operator[](int64_t i) const { return (p == nullptr || i < 0 || i >= n) ? bad() : p[i]; }
    // `count` elements from element i on as a bare pointer (vector accesses)
    __device__ __forceinline__ T *at(int64_t i, int64_t count = 1) const
    {
        return (p == nullptr || i < 0 || i + count > n) ? &bad() : p + i;
    }
#else
    __host__ __device__ vtk_arr() : p(nullptr) {}
    __host__ __device__ vtk_arr(T *p_, int64_t, uint32_t *) : p(p_) {}
    __device__ __forceinline__ T &operator[](int64_t i) const { return p[i]; }
    __device__ __forceinline__ T *at(int64_t i, int64_t = 1) const { return p + i; }
#endif
    __device__ __forceinline__ T &operator*() const { return (*this)[0]; }
    __device__ __forceinline__ T *operator->() const { return at(0); }
    __host__ __device__ __forceinline__ bool null() const { return p == nullptr; }
};

// the flag word the checked build reports to: the context's word for the calls outside plan / repack,
// which no kernel overwrites and vtoken_read_counts reports (and clears)
#define VTK_CHECK_FLAG(ctx) (&(ctx)->rt_counts->error_flags)
// binds `n` elements at `ptr` (capacity known to the context) for a kernel
#define VTK_ARR(ctx, ptr, n) \
    vtk_arr<typename std::remove_pointer<typename std::decay<decltype(ptr)>::type>::type>((ptr), (int64_t)(n), VTK_CHECK_FLAG(ctx))

// host launchers, one per translation unit
int vtk_launch_plan(vtoken_ctx *ctx, const vtoken_plan_in *in, const vtoken_plan_out *out, cudaStream_t st);
int vtk_launch_plan_small(vtoken_ctx *ctx, const vtoken_plan_in *in, const vtoken_plan_out *out, cudaStream_t st);
int vtk_configure_plan(vtoken_ctx *ctx);         // once per context: which form of the whole-request planner it uses
int vtk_launch_copy(vtoken_ctx *ctx, cudaStream_t st);
int vtk_configure_copy(vtoken_ctx *ctx);
// > 0: launched; 0: the context has no bulk configuration for these rows; < 0: VTOKEN_* error
int vtk_launch_gather_bulk(vtoken_ctx *ctx, const int32_t *g_src, const int32_t *g_total, int32_t layer_begin,
                            int32_t layer_end, void *out_k, void *out_v, int64_t out_capacity, cudaStream_t st);
int vtk_launch_gather(vtoken_ctx *ctx, const int32_t *num_requests, const int32_t *tt_offsets,
                      const int32_t *tt_slots, const uint8_t *keep, const uint8_t *select,
                      int32_t layer_begin, int32_t layer_end, void *out_k, void *out_v,
                      int64_t out_capacity_tokens, int32_t *out_offsets, cudaStream_t st);

#define VTK_CUDA(ctx, call)                                  \
    do {                                                     \
        cudaError_t e__ = (call);                            \
        if (e__ != cudaSuccess) {                            \
            (ctx)->last_cuda_error = (int)e__;               \
            return VTOKEN_ECUDA;                             \
        }                                                    \
    } while (0)

// ---------------------------------------------------------------------------------------
// Programmatic dependent launch: a kernel launched through vtk_launch_dependent may become
// resident while its predecessor in the stream is still running (its launch latency and its
// prologue overlap the predecessor's tail); it must call vtk_wait_for_predecessor() before it
// touches anything an earlier kernel wrote or still reads -- the wait returns once the
// predecessor grid has completed and its writes are visible.  Every thread of such a kernel
// calls the wait before it can exit, so the grid cannot complete before its predecessor did and
// the ordering stays transitive along the stream.  vtk_release_successor() lets the next
// kernel in the stream start its own launch early.
// ---------------------------------------------------------------------------------------
__device__ __forceinline__ void vtk_wait_for_predecessor() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void vtk_release_successor() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }

// Ring shape of the bulk-copy kernel (warps per CTA x stages per warp, 4 KiB per stage).  Default 8 x 4 =
// 128 KiB per SM: alone it copies as fast as 8 x 6 (6.69 TB/s on the steady-state workload), beside a
// bandwidth-bound read kernel the two together move 7.07 TB/s instead of 6.27 (repack 2.26 + reader 4.81
// instead of 1.98 + 4.29), and 99 KiB of every SM's shared memory stay free for the other kernel.
// (8 x 3 = 96 KiB came out bimodal from run to run, alone and beside the reader: not offered.)
constexpr int VTK_DEFAULT_WARPS = 8, VTK_DEFAULT_STAGES = 4;

// cfg.plain_launches turns the launch attribute off (the device side is then a no-op)
template <typename... P, typename... A>
inline cudaError_t vtk_launch_dependent(const vtoken_ctx *ctx, void (*kernel)(P...), dim3 grid, dim3 block, size_t smem,
                                        cudaStream_t st, A... args)
{
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid;
    cfg.blockDim = block;
    cfg.dynamicSmemBytes = smem;
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = ctx->cfg.plain_launches ? 0 : 1;
    return cudaLaunchKernelEx(&cfg, kernel, P(args)...);
}

// ---------------------------------------------------------------------------------------
// device helpers
// ---------------------------------------------------------------------------------------
__device__ __forceinline__ int vtk_lane() { return threadIdx.x & 31; }

__device__ __forceinline__ int vtk_warp_incl_scan(int v)
{
#pragma unroll
    for (int d = 1; d < 32; d <<= 1) {
        int o = __shfl_up_sync(0xffffffffu, v, d);
        if (vtk_lane() >= d) v += o;
    }
    return v;
}

// Exclusive rank of `flag` among the flags of a CTA of NT threads (NT multiple of 32, <= 1024)
// in thread order, plus the CTA total.  warp_sums: shared int[NT/32 + 1].  Two barriers.
template <int NT>
__device__ __forceinline__ int vtk_block_rank(bool flag, int *warp_sums, int &total)
{
    const unsigned ballot = __ballot_sync(0xffffffffu, flag);
    const int lane = vtk_lane(), warp = threadIdx.x >> 5;
    const int in_warp = __popc(ballot & ((1u << lane) - 1u));
    if (lane == 0) warp_sums[warp] = __popc(ballot);
    __syncthreads();
    if (warp == 0) {
        int v = (lane < NT / 32) ? warp_sums[lane] : 0;
        int incl = vtk_warp_incl_scan(v);
        if (lane < NT / 32) warp_sums[lane] = incl - v;
        if (lane == 31) warp_sums[NT / 32] = incl;
    }
    __syncthreads();
    const int rank = warp_sums[warp] + in_warp;
    total = warp_sums[NT / 32];
    __syncthreads();   // warp_sums is reused by the next call
    return rank;
}

// Range [off[r], off[r+1]) of request r in a CSR table, clipped to the create-time capacity of that
// table: entries at or beyond `cap` (and ranges that run backwards) do not exist for the planners,
// whose output buffers are sized by the capacities.  Returns true when something was clipped.
template <typename Off>
__device__ __forceinline__ bool vtk_range(const Off &off, int r, int64_t cap, int64_t &lo, int64_t &hi)
{
    const int64_t a = off[r], b = off[r + 1];
    lo = a < 0 ? 0 : (a > cap ? cap : a);
    hi = b < lo ? lo : (b > cap ? cap : b);
    return lo != a || hi != b;
}

// Inclusive scan over the values of a CTA of 1024 threads in thread order; `shfl` is the type's
// shuffle-up, warp_tot shared T[32].  Three barriers; the result may be used at once.
template <typename T, typename ShflUp>
__device__ __forceinline__ T vtk_block_incl_scan(T v, T *warp_tot, T zero, ShflUp shfl)
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
        T w = warp_tot[lane];
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


// ---------------------------------------------------------------------------------------
// Flat tiling of the token table, shared by the planners: a tile is VTK_TILE consecutive table
// entries whatever request they belong to, one CTA of VTK_TILE_NT threads, four entries per thread.
// ---------------------------------------------------------------------------------------
constexpr int VTK_TILE_NT = 256;
constexpr int VTK_TILE_TOK = 4;
constexpr int VTK_TILE = VTK_TILE_NT * VTK_TILE_TOK;

// first table entry of request r (r == R: one past the last entry), clipped to the table capacity
template <typename Off>
__device__ __forceinline__ int64_t vtk_clipped_offset(const Off &off, int r, int64_t cap)
{
    const int64_t o = off[r];
    return o < 0 ? 0 : (o > cap ? cap : o);
}

// The thread's four entries [t, t + 4) of the token table below T: slots, and one bit per live entry.
// Entries in front of `first` (the first request's first entry) belong to no request and count as dead.
// vec: tt_slots is 16-byte and keep 4-byte aligned (t is a multiple of four).  keep == nullptr: every entry
// with a slot counts as kept.
// element i of a bare pointer or of a vtk_arr, `count` elements as a bare pointer
template <typename T> __device__ __forceinline__ T *vtk_at(T *p, int64_t i, int64_t = 1) { return p + i; }
template <typename T> __device__ __forceinline__ T *vtk_at(const vtk_arr<T> &a, int64_t i, int64_t count = 1) { return a.at(i, count); }
template <typename T> __device__ __forceinline__ bool vtk_null(T *p) { return p == nullptr; }
template <typename T> __device__ __forceinline__ bool vtk_null(const vtk_arr<T> &a) { return a.null(); }

template <typename Slots, typename Keep>
__device__ __forceinline__ unsigned vtk_load_entries(const Slots &tt_slots, const Keep &keep, int vec, int64_t t,
                                                     int64_t first, int64_t T, int64_t slots_per_layer,
                                                     int32_t (&slot)[VTK_TILE_TOK], bool &bad)
{
    uint8_t kp[VTK_TILE_TOK] = {0, 0, 0, 0};
#pragma unroll
    for (int k = 0; k < VTK_TILE_TOK; ++k) slot[k] = -1;
    if (vec && t + VTK_TILE_TOK <= T) {
        const int4 s4 = *reinterpret_cast<const int4 *>(vtk_at(tt_slots, t, VTK_TILE_TOK));
        const uchar4 k4 = !vtk_null(keep) ? *reinterpret_cast<const uchar4 *>(vtk_at(keep, t, VTK_TILE_TOK))
                                          : make_uchar4(1, 1, 1, 1);
        slot[0] = s4.x; slot[1] = s4.y; slot[2] = s4.z; slot[3] = s4.w;
        kp[0] = k4.x; kp[1] = k4.y; kp[2] = k4.z; kp[3] = k4.w;
    } else {
#pragma unroll
        for (int k = 0; k < VTK_TILE_TOK; ++k)
            if (t + k < T) { slot[k] = tt_slots[t + k]; kp[k] = !vtk_null(keep) ? keep[t + k] : 1; }
    }
    unsigned bits = 0;
#pragma unroll
    for (int k = 0; k < VTK_TILE_TOK; ++k) {
        if (slot[k] < 0 || t + k < first) continue;
        if ((int64_t)slot[k] >= slots_per_layer) { bad = true; continue; }
        if (kp[k] != 0) bits |= 1u << k;
    }
    return bits;
}

// The requests that own the first and the last entry of the tile [base, min(base + VTK_TILE, T)) --
// owner of an entry: the last request whose first entry is at or before it; -1: the entry lies in
// front of the first request -- each found by one warp (warps 0 and 1, all lanes) with a 32-way
// search over the offsets; tile_req[2] is shared memory, valid after the caller's next barrier.
template <typename Off>
__device__ __forceinline__ void vtk_tile_owners(const Off &off, int R, int64_t cap, int64_t base, int64_t T,
                                                int *tile_req)
{
    const int warp = threadIdx.x >> 5, lane = vtk_lane();
    if (warp >= 2) return;
    const int64_t last = (base + VTK_TILE < T ? base + VTK_TILE : T) - 1;
    const int64_t key = warp == 0 ? base : last;
    int lo = -1, hi = R;                    // offset(lo) <= key (or lo == -1); offset(hi) > key: offset(R) = T
    while (hi - lo > 1) {
        const int step = (hi - lo - 1 + 31) / 32;
        const int probe = lo + 1 + lane * step;
        const bool le = probe < hi && vtk_clipped_offset(off, probe, cap) <= key;
        const int n_le = __popc(__ballot_sync(0xffffffffu, le));
        const int first_gt = lo + 1 + n_le * step;          // first probe beyond the key, if it was probed
        if (n_le > 0) lo = lo + 1 + (n_le - 1) * step;
        if (first_gt < hi) hi = first_gt;
    }
    if (lane == 0) tile_req[warp] = lo;
}

// The request that owns entry t of the tile whose owners are in tile_req (-1: none).
template <typename Off>
__device__ __forceinline__ int vtk_entry_owner(const Off &off, int64_t cap, const int *tile_req, int64_t t)
{
    int lo = tile_req[0], hi = (tile_req[1] > tile_req[0] ? tile_req[1] : tile_req[0]) + 1;
    while (hi - lo > 1) {                   // offset(lo) <= t (or lo == -1); offset(hi) > t
        const int mid = (lo + hi) >> 1;
        if (vtk_clipped_offset(off, mid, cap) <= t) lo = mid; else hi = mid;
    }
    return lo;
}

// A token is live when it owns a slot inside the pool and the policy kept it.
template <typename Keep>
__device__ __forceinline__ bool vtk_live(int32_t slot, const Keep &keep, int64_t t, int64_t slots_per_layer,
                                         bool &bad_slot)
{
    if (slot < 0) return false;
    if ((int64_t)slot >= slots_per_layer) { bad_slot = true; return false; }
    return vtk_null(keep) || keep[t] != 0;
}
