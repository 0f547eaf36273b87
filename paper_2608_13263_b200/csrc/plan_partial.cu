// Eligibility metadata and partial relocation plans (Sec. 3.3.1 - 3.3.3 of the paper): per-block
// liveness n_b, the global waste ratio F as a trigger, and a planner that evacuates only the
// low-utilisation, unprotected source blocks of a request (at most B of them) and leaves the
// others -- fully live blocks, shared-prefix blocks -- where they are.
//
// Kernels (all grids fixed by the capacities, counts read from device memory).  The token table is
// walked in flat tiles of 1024 entries that ignore request boundaries (see plan.cu); per-request
// numbers are differences of running counts at the request's two boundaries:
//   tiles<0>: live tokens per tile and in front of every request boundary inside its tile;
//             n_b[block] += 1 per live token (integer atomics: the sums do not depend on their
//             order); with a detach threshold also the live tokens that sit in protected blocks
//   blocks  : per request, which entries of its block table are sources (rank among eligible
//             entries in table order < B); marks blk_src[block]; decides copy-on-write detach
//   tiles<1>: live tokens that move (they sit in a source block of their request), per tile and
//             in front of every request boundary
//   scan    : running counts at every tile start, live and moving tokens per request, global
//             trigger F > theta, candidates (sources release more blocks than the destinations
//             they need), admission against the free list, bases and counts
//   assign  : new token table (moving tokens ranked in logical order: running count at the token
//             minus running count at the request's first entry), inverse move plan; one extra CTA
//             per request writes the new block table (kept blocks in old order, then
//             destinations), the reclaimed and the released list
// The inverse plan has the same form as the whole-request planner's, so vtoken_repack runs it
// unchanged.
//
// Copy-on-write detach (optional): a request whose own live tokens fill too little of its
// protected (shared) blocks leaves all of them -- they become sources for this request only, its
// tokens there are copied out with the rest, and the blocks are listed as released references
// instead of reclaimed blocks.  "Source" is therefore a per-request notion for protected blocks
// (req_detach[r]) and a per-block one (blk_src[b]) for the others.
//
// Detach decided per shared block on all holders' tokens (opts->detach_rule 2): a protected block whose
// n_b is below the threshold is left by every planned holder.  The blocks kernel marks it blk_src = 2
// (every holder writes the same value), after which its tokens move like those of any other source and
// the block-table writers list it under released instead of reclaimed; no owner of an entry is needed.
//
// Detach decided per shared block on the request's own tokens (opts->detach_rule 1): the request leaves
// exactly the protected blocks that its own live tokens fill below the threshold.  That needs the census n_rb (live
// tokens of request r stored in block b) for every protected entry of every block table, and every
// token must find the count of its own (request, block) pair.  Each request owns the range
// [2 * bt_offsets[r], 2 * bt_offsets[r + 1]) of one scratch array as a private open-addressing hash
// from block id to count (twice as many places as it can have protected entries, so a probe
// sequence always ends): cleared by a memset node, filled with the protected entries by one more
// kernel in front of tiles<0>, counted into by tiles<0> (integer atomics), read by blocks, tiles<1>
// and assign.  A token in a protected block that its request's table does not list finds nothing
// and stays where it is.
#include "common.cuh"

#include <cstring>

namespace {

constexpr int PP_NT = 512;                 // threads of a blocks CTA (one per request)
constexpr int PP_SCAN_NT = 1024;
constexpr int TILE_NT = VTK_TILE_NT, TILE_TOK = VTK_TILE_TOK, TILE = VTK_TILE;

struct PArgs {
    vtk_arr<const int32_t> num_requests, bt_offsets, bt_blocks, tt_offsets, tt_slots;
    vtk_arr<const uint8_t> keep, select, protect;
    uint32_t thr_num, thr_den, util_num, util_den, theta_num, theta_den, detach_num, detach_den;
    uint32_t rule;                   // detach rule: 0 per request, 1 per protected block on the request's own tokens (the
                                     // census in cow), 2 per protected block on all holders' tokens (n_b; blk_src == 2)
    int32_t max_sources;
    vtk_arr<const int32_t> free_blocks, num_free;
    vtk_arr<int32_t> new_bt_offsets, new_bt_blocks, new_tt_slots, freed_blocks, released_blocks, out_status;
    vtk_arr<vtoken_counts> out_counts;
    vtk_arr<int32_t> req_n, req_ns, req_nsrc, req_dst_base, req_freed_base, req_status;
    vtk_arr<int32_t> req_shared, req_detach, req_rel_base;
    // flat tiling: counts per tile ([num_tiles + 1]; live and moving become running counts in the scan
    // kernel; the sign bit of a live count says "a slot outside the pool in this tile") and counts
    // between the start of the tile that holds a request's first entry and that entry ([max_requests + 1])
    vtk_arr<int32_t> tile_live, tile_mov, tile_shared, part_live, part_mov, part_shared;
    vtk_arr<int32_t> req_before;     // [max_requests + 1] moving tokens of the table before the request's first entry
    vtk_arr<int32_t> dst_src, dst_blocks, n_b;
    vtk_arr<uint8_t> blk_src;        // 1: source of its request; 2: protected block that every planned holder leaves
    vtk_arr<unsigned long long> cow; // [2 * max_table_blocks] per-request hashes: (block id + 1) << 32 | own live tokens
    vtk_arr<vtoken_counts> counts;
    int32_t S, num_blocks, max_requests, cap_dst_blocks, max_free_blocks;
    int32_t num_tiles, vec_in, vec_out;
    int64_t slots_per_layer, max_tokens, max_table_blocks;
};

__device__ __forceinline__ int pp_requests(const PArgs &a)
{
    int R = *a.num_requests;
    return R < 0 ? 0 : (R > a.max_requests ? a.max_requests : R);
}

__device__ __forceinline__ int64_t pp_offset(const PArgs &a, int r)
{
    return vtk_clipped_offset(a.tt_offsets, r, a.max_tokens);
}

__device__ __forceinline__ int pp_block_sum(int n, int *warp_n)
{
#pragma unroll
    for (int d = 16; d > 0; d >>= 1) n += __shfl_down_sync(0xffffffffu, n, d);
    if (vtk_lane() == 0) warp_n[threadIdx.x >> 5] = n;
    __syncthreads();
    int s = 0;
    if (threadIdx.x == 0)
        for (int w = 0; w < (int)(blockDim.x >> 5); ++w) s += warp_n[w];
    return s;   // valid in thread 0
}

// ---- the per-request census of own live tokens in protected blocks -------------------------------
// The hash of request r: `size` places from `base` on (size == 0: the request has no block table).
struct CowTable {
    int64_t base, size;
};
__device__ __forceinline__ CowTable pp_cow_table(const PArgs &a, int r)
{
    int64_t b0, b1;
    vtk_range(a.bt_offsets, r, a.max_table_blocks, b0, b1);
    return CowTable{2 * b0, 2 * (b1 - b0)};
}
__device__ __forceinline__ int64_t pp_cow_first(const CowTable &h, int32_t b)
{
    return (int64_t)(((uint32_t)b * 2654435761u) % (uint64_t)h.size);
}
// Place of block b in the table (nullptr: not there).  INSERT: take the first free place on the way.
template <bool INSERT>
__device__ __forceinline__ unsigned long long *pp_cow_find(const PArgs &a, const CowTable &h, int32_t b)
{
    if (h.size <= 0) return nullptr;
    const unsigned long long tag = (unsigned long long)(uint32_t)(b + 1) << 32;
    int64_t i = pp_cow_first(h, b);
    for (int64_t probes = 0; probes < h.size; ++probes) {           // bounded: at most once around the table
        unsigned long long *p = &a.cow[h.base + i];
        unsigned long long e = *p;
        if (INSERT && e == 0) {
            e = atomicCAS(p, 0ull, tag);
            if (e == 0) return p;
        }
        if ((e >> 32) == (tag >> 32)) return p;
        if (e == 0) return nullptr;
        i = i + 1 == h.size ? 0 : i + 1;
    }
    return nullptr;
}
// does request r leave protected block b?  (its own live tokens there fill less than the threshold)
__device__ __forceinline__ bool pp_cow_leaves(const PArgs &a, const CowTable &h, int32_t b)
{
    const unsigned long long *p = pp_cow_find<false>(a, h, b);
    if (!p) return false;
    return (*p & 0xffffffffull) * a.detach_den < (unsigned long long)a.detach_num * (unsigned long long)a.S;
}

// one CTA per request: its protected table entries enter its hash
__global__ void __launch_bounds__(256) pp_cow_insert_kernel(PArgs a)
{
    vtk_release_successor();
    vtk_wait_for_predecessor();
    const int r = blockIdx.x;
    if (r >= pp_requests(a)) return;
    int64_t b0, b1;
    vtk_range(a.bt_offsets, r, a.max_table_blocks, b0, b1);
    const CowTable h{2 * b0, 2 * (b1 - b0)};
    for (int64_t j = b0 + threadIdx.x; j < b1; j += 256) {
        const int32_t blk = a.bt_blocks[j];
        if (blk < 0 || blk >= a.num_blocks) continue;              // flagged by the blocks kernel
        if (a.protect[blk] != 0) pp_cow_find<true>(a, h, blk);
    }
}

// ---- tiles: live / moving tokens per tile and in front of request boundaries, per-block liveness ----
// What decides whether a live token of the request at hand moves out of a protected block.
struct Owner {
    bool detach;         // the request leaves protected blocks (all of them, or those the census names)
    CowTable cow;        // per-block rule: its census
};
__device__ __forceinline__ Owner pp_owner(const PArgs &a, int r)
{
    Owner o{false, CowTable{0, 0}};
    if (r < 0) return o;
    o.detach = a.req_detach[r] != 0;
    if (o.detach && a.rule == 1) o.cow = pp_cow_table(a, r);
    return o;
}
// does a live token of that request in block b move?  (b is a source of its request, or the request
// leaves protected blocks and b is one of those it leaves)
__device__ __forceinline__ bool pp_moves(const PArgs &a, const Owner &o, int32_t b)
{
    if (a.blk_src[b] != 0) return true;
    if (!o.detach || a.protect[b] == 0) return false;
    return a.rule == 1 ? pp_cow_leaves(a, o.cow, b) : true;
}

// Bits of the thread's live entries that move.  Without a detach threshold that is a property of the
// block alone; with one, protected blocks move for the requests that leave them, so the owner of
// every entry is needed: r is the owner of entry t (-1: none) and is stepped over request boundaries.
__device__ __forceinline__ unsigned pp_moving_bits(const PArgs &a, unsigned bits, const int32_t (&slot)[TILE_TOK],
                                                   bool may_detach, int R, int64_t t, int r)
{
    unsigned mov = 0;
    if (bits == 0) return 0;                // nothing live (also: entries outside the table, whose owner would
                                            // have to be searched from the first request on)
    int64_t next = may_detach ? pp_offset(a, r + 1 <= R ? r + 1 : R) : 0;
    Owner o = may_detach ? pp_owner(a, r) : Owner{false, CowTable{0, 0}};
#pragma unroll
    for (int k = 0; k < TILE_TOK; ++k) {
        if (!((bits >> k) & 1u)) continue;
        if (may_detach && t + k >= next && r + 1 < R) {      // owners are stepped at live entries only
            while (r + 1 < R && pp_offset(a, r + 1) <= t + k) ++r;
            next = pp_offset(a, r + 1);
            o = pp_owner(a, r);
        }
        if (pp_moves(a, o, slot[k] / a.S)) mov |= 1u << k;
    }
    return mov;
}

// mode 0: live tokens per tile, n_b (and, with a detach threshold, the live tokens in protected
// blocks, or -- per-block rule -- the census of every request's own live tokens in its protected
// blocks); mode 1: live tokens that move.
template <int MODE>
__global__ void __launch_bounds__(TILE_NT) pp_tiles_kernel(PArgs a)
{
    __shared__ int warp_n[TILE_NT / 32], warp_sh[TILE_NT / 32];
    __shared__ int tile_req[2];
    vtk_release_successor();
    vtk_wait_for_predecessor();
    const int R = pp_requests(a);
    const int64_t T = pp_offset(a, R);
    const int lane = vtk_lane(), warp = threadIdx.x >> 5;
    // (rule 2 needs no owners: the blocks its holders leave are marked in blk_src like any other source)
    const bool may_detach = !a.protect.null() && a.detach_den != 0 && a.rule != 2;
    // A CTA counts over the entries [base, limit): a whole tile, or (the CTAs behind the tiles, one per
    // request boundary) the entries between the start of the boundary's tile and the boundary.
    const bool is_tile = (int)blockIdx.x < a.num_tiles;
    const int rb = (int)blockIdx.x - a.num_tiles;
    int64_t base, limit;
    if (is_tile) {
        base = (int64_t)blockIdx.x * TILE;
        limit = T;
        if (base >= T) return;
    } else {
        if (rb > R) return;
        limit = pp_offset(a, rb);
        base = limit / TILE * TILE;
        if (base == limit) return;                       // nothing in front of it: never read
    }
    bool bad = false;
    int32_t slot[TILE_TOK];
    const int64_t t = base + threadIdx.x * TILE_TOK;
    const unsigned bits = vtk_load_entries(a.tt_slots, a.keep, a.vec_in, t, pp_offset(a, 0), limit, a.slots_per_layer, slot, bad);
    int n = 0, n_sh = 0;
    if (MODE == 0) {
        const bool census = may_detach && a.rule == 1 && is_tile;        // uniform over the CTA
        int r = -1;
        int64_t next = 0;
        CowTable h{0, 0};
        if (census) {
            vtk_tile_owners(a.tt_offsets, R, a.max_tokens, base, limit, tile_req);
            __syncthreads();
            if (t < limit && bits != 0) {
                r = vtk_entry_owner(a.tt_offsets, a.max_tokens, tile_req, t);
                next = pp_offset(a, r + 1 <= R ? r + 1 : R);
                if (r >= 0) h = pp_cow_table(a, r);
            }
        }
#pragma unroll
        for (int k = 0; k < TILE_TOK; ++k) {
            if (!((bits >> k) & 1u)) continue;
            if (census && t + k >= next && r + 1 < R) {      // owners are stepped at live entries only
                while (r + 1 < R && pp_offset(a, r + 1) <= t + k) ++r;
                next = pp_offset(a, r + 1);
                h = pp_cow_table(a, r);
            }
            const int blk = slot[k] / a.S;
            if (is_tile) atomicAdd(&a.n_b[blk], 1);          // the tile CTAs see every entry exactly once
            ++n;
            if (may_detach) {
                const bool prot = a.protect[blk] != 0;
                n_sh += prot;
                if (census && prot && r >= 0) {
                    unsigned long long *p = pp_cow_find<false>(a, h, blk);
                    if (p) atomicAdd(p, 1ull);                  // the count lives in the low half
                }
            }
        }
    } else {
        int r = -1;
        if (may_detach) {                                      // uniform over the CTA
            vtk_tile_owners(a.tt_offsets, R, a.max_tokens, base, limit, tile_req);
            __syncthreads();
            if (t < limit) r = vtk_entry_owner(a.tt_offsets, a.max_tokens, tile_req, t);
        }
        n = __popc(pp_moving_bits(a, bits, slot, may_detach, R, t, r));
    }
#pragma unroll
    for (int d = 16; d > 0; d >>= 1) {
        n += __shfl_down_sync(0xffffffffu, n, d);
        n_sh += __shfl_down_sync(0xffffffffu, n_sh, d);
    }
    if (lane == 0) { warp_n[warp] = n; warp_sh[warp] = n_sh; }
    const int any_bad = __syncthreads_or(bad);
    if (threadIdx.x == 0) {
        int s = 0, sh = 0;
#pragma unroll
        for (int w = 0; w < TILE_NT / 32; ++w) { s += warp_n[w]; sh += warp_sh[w]; }
        if (MODE == 0) {
            if (is_tile) a.tile_live[blockIdx.x] = s | (any_bad ? (int)0x80000000 : 0);   // flag in the sign bit
            else a.part_live[rb] = s;
            if (may_detach) (is_tile ? a.tile_shared[blockIdx.x] : a.part_shared[rb]) = sh;
        } else {
            (is_tile ? a.tile_mov[blockIdx.x] : a.part_mov[rb]) = s;
        }
    }
}

// ---- blocks: source selection per request ------------------------------------------------------
__global__ void __launch_bounds__(PP_NT) pp_blocks_kernel(PArgs a)
{
    vtk_release_successor();
    vtk_wait_for_predecessor();
    __shared__ int warp_sums[PP_NT / 32 + 1];
    const int r = blockIdx.x;
    if (r >= pp_requests(a)) return;
    int64_t b0, b1;
    vtk_range(a.bt_offsets, r, a.max_table_blocks, b0, b1);
    int carry = 0;               // eligible entries before this chunk
    int shared = 0;              // protected entries seen by this thread (per-block rule: those the request leaves)
    uint32_t flags = 0;
    const bool per_block = !a.protect.null() && a.detach_den != 0 && a.rule != 0;
    const CowTable h{2 * b0, 2 * (b1 - b0)};
    for (int64_t jb = b0; jb < b1; jb += PP_NT) {
        const int64_t j = jb + threadIdx.x;
        bool eligible = false;
        int blk = -1;
        if (j < b1) {
            blk = a.bt_blocks[j];
            if (blk < 0 || blk >= a.num_blocks) {
                flags |= VTOKEN_FLAG_BAD_BLOCK;
                blk = -1;
            } else {
                eligible = !(!a.protect.null() && a.protect[blk] != 0);
                if (!eligible) {
                    bool leaves = true;                    // rule 0: decided below for all protected entries at once
                    if (a.rule == 1 && per_block) leaves = pp_cow_leaves(a, h, blk);
                    if (a.rule == 2 && per_block) {
                        // everything stored in the block, whoever holds it: every holder finds the same answer
                        leaves = (unsigned long long)a.n_b[blk] * a.detach_den <
                                 (unsigned long long)a.detach_num * (unsigned long long)a.S;
                        if (leaves) a.blk_src[blk] = 2;
                    }
                    shared += leaves ? 1 : 0;
                }
                if (eligible && a.util_den != 0)
                    eligible = (unsigned long long)a.n_b[blk] * a.util_den <
                               (unsigned long long)a.util_num * (unsigned long long)a.S;
            }
        }
        int total;
        const int rank = carry + vtk_block_rank<PP_NT>(eligible, warp_sums, total);
        carry += total;
        if (eligible && (a.max_sources <= 0 || rank < a.max_sources)) a.blk_src[blk] = 1;
    }
    int ns = (a.max_sources > 0 && carry > a.max_sources) ? a.max_sources : carry;
    if (per_block) {
        // block by block: the protected entries the request leaves are sources, the others stay
        __syncthreads();
        const int ns_leaving = pp_block_sum(shared, warp_sums);         // valid in thread 0
        if (threadIdx.x == 0) {
            a.req_detach[r] = ns_leaving > 0 ? 1 : 0;
            a.req_shared[r] = ns_leaving;
            ns += ns_leaving;
        }
    } else if (!a.protect.null() && a.detach_den != 0) {
        // copy-on-write detach: the request leaves its protected blocks when its own live tokens
        // fill less than detach_num / detach_den of them; then every one of them is a source
        __syncthreads();
        const int ns_shared = pp_block_sum(shared, warp_sums);          // valid in thread 0
        // the request's live tokens in protected blocks: the tiles between its two boundaries, corrected
        // at both ends by the counts in front of the boundaries
        const int64_t o0 = pp_offset(a, r), o1 = pp_offset(a, r + 1);
        int in_tiles = 0;
        for (int64_t i = o0 / TILE + threadIdx.x; i < o1 / TILE; i += PP_NT) in_tiles += a.tile_shared[i];
        __syncthreads();
        in_tiles = pp_block_sum(in_tiles, warp_sums);                   // valid in thread 0
        if (threadIdx.x == 0) {
            long long n_shared = (long long)in_tiles + (o1 % TILE != 0 ? a.part_shared[r + 1] : 0) -
                                 (o0 % TILE != 0 ? a.part_shared[r] : 0);
            if (n_shared < 0) n_shared = 0;                             // offsets that run backwards
            const bool detach = ns_shared > 0 &&
                                (unsigned long long)n_shared * a.detach_den <
                                    (unsigned long long)a.detach_num * (unsigned long long)ns_shared * (unsigned long long)a.S;
            a.req_detach[r] = detach ? 1 : 0;
            a.req_shared[r] = detach ? ns_shared : 0;
            ns += detach ? ns_shared : 0;
        }
    }
    if (threadIdx.x == 0) a.req_ns[r] = ns;
    if (flags) atomicOr(&a.counts->error_flags, flags);
}

// ---- scan ----------------------------------------------------------------------------------------
struct PAcc {
    int dst, freed, newbt, moves, admitted, deferred, released;
};
__device__ __forceinline__ PAcc operator+(const PAcc &x, const PAcc &y)
{
    return PAcc{x.dst + y.dst, x.freed + y.freed, x.newbt + y.newbt, x.moves + y.moves, x.admitted + y.admitted,
                x.deferred + y.deferred, x.released + y.released};
}
__device__ __forceinline__ PAcc pp_shfl_up(const PAcc &v, int d)
{
    return PAcc{__shfl_up_sync(0xffffffffu, v.dst, d),      __shfl_up_sync(0xffffffffu, v.freed, d),
                __shfl_up_sync(0xffffffffu, v.newbt, d),    __shfl_up_sync(0xffffffffu, v.moves, d),
                __shfl_up_sync(0xffffffffu, v.admitted, d), __shfl_up_sync(0xffffffffu, v.deferred, d),
                __shfl_up_sync(0xffffffffu, v.released, d)};
}
__global__ void __launch_bounds__(PP_SCAN_NT) pp_scan_kernel(PArgs a)
{
    vtk_release_successor();
    vtk_wait_for_predecessor();
    __shared__ long long warp_ll[32];
    __shared__ PAcc warp_acc[32];
    __shared__ long long carry_need, tot_live, tot_blocks;
    __shared__ PAcc carry;
    __shared__ int carry_live, carry_mov;
    const int tid = threadIdx.x;
    const int R = pp_requests(a);
    uint32_t flags = 0;
    if (tid == 0) {
        if (*a.num_requests > a.max_requests || *a.num_requests < 0) flags |= VTOKEN_FLAG_CAPACITY;
        carry_need = 0;
        carry_live = 0;
        carry_mov = 0;
        tot_live = 0;
        tot_blocks = 0;
        carry = PAcc{0, 0, 0, 0, 0, 0, 0};
    }
    int nf = *a.num_free;
    if (nf > a.max_free_blocks && tid == 0) flags |= VTOKEN_FLAG_CAPACITY;
    nf = nf < 0 ? 0 : (nf > a.cap_dst_blocks ? a.cap_dst_blocks : nf);
    __syncthreads();
    auto shfl_ll = [](long long v, int d) { return __shfl_up_sync(0xffffffffu, v, d); };
    auto shfl_acc = [](const PAcc &v, int d) { return pp_shfl_up(v, d); };

    // live and moving tokens before every tile (in place: an entry becomes the sum of the tiles before
    // it; one entry past the last tile holds the total)
    const int64_t T = pp_offset(a, R);
    const int tiles = (int)((T + TILE - 1) / TILE);
    for (int base = 0; base <= tiles; base += PP_SCAN_NT) {
        const int i = base + tid;
        const int raw = i < tiles ? a.tile_live[i] : 0;
        if (raw < 0) flags |= VTOKEN_FLAG_BAD_SLOT;
        const long long v = ((long long)(raw & 0x7fffffff) << 32) | (unsigned)(i < tiles ? a.tile_mov[i] : 0);
        // both counts in one 64-bit scan: live in the high half, moving in the low half (each < 2^31)
        const long long incl = vtk_block_incl_scan<long long>(v, warp_ll, 0LL, shfl_ll) +
                               (((long long)carry_live << 32) | (unsigned)carry_mov);
        if (i <= tiles) {
            a.tile_live[i] = (int)((incl - v) >> 32);
            a.tile_mov[i] = (int)((incl - v) & 0xffffffffll);
        }
        __syncthreads();
        if (tid == PP_SCAN_NT - 1) {
            carry_live = (int)(incl >> 32);
            carry_mov = (int)(incl & 0xffffffffll);
        }
        __syncthreads();
    }
    // tokens before table entry o = tokens before its tile + those between the tile's start and o
    auto live_before = [&](int r) {
        const int64_t o = pp_offset(a, r);
        return a.tile_live[o / TILE] + (o % TILE != 0 ? a.part_live[r] : 0);
    };
    auto mov_before = [&](int r) {
        const int64_t o = pp_offset(a, r);
        return a.tile_mov[o / TILE] + (o % TILE != 0 ? a.part_mov[r] : 0);
    };

    // pass 1: live and moving tokens per request, and the totals behind F = 1 - live / (N * S)
    long long my_live = 0, my_blocks = 0;
    for (int r = tid; r < R; r += PP_SCAN_NT) {
        const int mb = mov_before(r);
        int n = live_before(r + 1) - live_before(r), nsrc = mov_before(r + 1) - mb;
        if (n < 0) n = 0;                                   // offsets that run backwards
        if (nsrc < 0) nsrc = 0;
        a.req_before[r] = mb;
        a.req_n[r] = n;
        a.req_nsrc[r] = nsrc;
        int64_t lo, hi, t0, t1;
        if (vtk_range(a.bt_offsets, r, a.max_table_blocks, lo, hi) | vtk_range(a.tt_offsets, r, a.max_tokens, t0, t1))
            flags |= VTOKEN_FLAG_CAPACITY;                  // tables beyond the create-time capacities
        my_live += n;
        my_blocks += hi - lo;
    }
    const long long live_incl = vtk_block_incl_scan<long long>(my_live, warp_ll, 0LL, shfl_ll);
    if (tid == PP_SCAN_NT - 1) tot_live = live_incl;
    const long long blocks_incl = vtk_block_incl_scan<long long>(my_blocks, warp_ll, 0LL, shfl_ll);
    if (tid == PP_SCAN_NT - 1) tot_blocks = blocks_incl;
    __syncthreads();
    bool triggered = true;                      // F > theta  <=>  (N*S - live) * den > num * N*S
    if (a.theta_den != 0) {
        const unsigned long long cap = (unsigned long long)tot_blocks * (unsigned long long)a.S;
        triggered = tot_blocks > 0 && (cap - (unsigned long long)tot_live) * a.theta_den > (unsigned long long)a.theta_num * cap;
    }

    // pass 2: candidates, admission, bases
    for (int base = 0; base < R; base += PP_SCAN_NT) {
        const int r = base + tid;
        const bool valid = r < R;
        const bool may_detach = !a.protect.null() && a.detach_den != 0;
        int n = 0, nsrc = 0, nb = 0, ns = 0, nrel = 0;
        if (valid) {
            n = a.req_n[r];
            nsrc = a.req_nsrc[r];
            ns = a.req_ns[r];
            nrel = may_detach ? a.req_shared[r] : 0;     // protected sources: released, not reclaimed
            int64_t lo, hi;
            vtk_range(a.bt_offsets, r, a.max_table_blocks, lo, hi);
            nb = (int)(hi - lo);
        }
        const int need = (int)(((int64_t)nsrc + a.S - 1) / a.S);   // ceil(T_live / S) over the source blocks
        bool sel = valid && triggered && (a.select.null() || a.select[r] != 0);
        if (sel && a.thr_den != 0)
            sel = (unsigned long long)n * a.thr_den <
                  (unsigned long long)a.thr_num * (unsigned long long)nb * (unsigned long long)a.S;
        const bool cand = sel && need < ns;                        // sources release more than they consume
        const long long cum = vtk_block_incl_scan<long long>(cand ? need : 0, warp_ll, 0LL, shfl_ll) + carry_need;
        const bool adm = cand && cum <= (long long)nf;
        const int status = !sel ? VTOKEN_NOT_SELECTED
                                : (!cand ? VTOKEN_NO_GAIN : (adm ? VTOKEN_REPACKED : VTOKEN_DEFERRED_NO_FREE));
        PAcc mine{adm ? need : 0, adm ? ns - nrel : 0, valid ? (adm ? nb - ns + need : nb) : 0, adm ? nsrc : 0,
                  adm ? 1 : 0, (cand && !adm) ? 1 : 0, adm ? nrel : 0};
        const PAcc incl = vtk_block_incl_scan<PAcc>(mine, warp_acc, PAcc{0, 0, 0, 0, 0, 0, 0}, shfl_acc) + carry;
        if (valid) {
            a.req_dst_base[r] = incl.dst - mine.dst;
            a.req_freed_base[r] = incl.freed - mine.freed;
            a.req_rel_base[r] = incl.released - mine.released;
            a.new_bt_offsets[r] = incl.newbt - mine.newbt;
            a.req_status[r] = status;
            a.out_status[r] = status;
        }
        __syncthreads();
        if (tid == PP_SCAN_NT - 1) {
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
        c.error_flags = atomicOr(&a.counts->error_flags, 0u);   // bits raised by the kernels before and above
        c.num_released = carry.released;
        *a.counts = c;
        *a.out_counts = c;
    }
}

// ---- assign --------------------------------------------------------------------------------------
__global__ void __launch_bounds__(TILE_NT) pp_assign_kernel(PArgs a)
{
    vtk_release_successor();
    vtk_wait_for_predecessor();
    __shared__ int warp_sums[TILE_NT / 32 + 1];
    __shared__ int tile_req[2];
    const int R = pp_requests(a);
    const int tid = threadIdx.x, lane = vtk_lane(), warp = tid >> 5;
    const int S = a.S;
    const bool any_detach = !a.protect.null() && a.detach_den != 0;
    const bool may_detach = any_detach && a.rule != 2;      // owners of entries are needed (see pp_tiles_kernel)
    uint32_t flags = 0;

    if ((int)blockIdx.x >= a.num_tiles) {
        // block table, reclaimed and released list of one request
        const int r = (int)blockIdx.x - a.num_tiles;
        if (r >= R) return;
        int64_t b0, b1;
        vtk_range(a.bt_offsets, r, a.max_table_blocks, b0, b1);
        const int nb = (int)(b1 - b0);
        const int64_t cap_bt = a.max_table_blocks;               // every table write below stays inside its buffer
        const bool adm = a.req_status[r] == VTOKEN_REPACKED;
        const bool detach = adm && any_detach && a.req_detach[r] != 0;
        const int nsrc = a.req_nsrc[r], ns = a.req_ns[r];
        const int need = (int)(((int64_t)nsrc + S - 1) / S);
        const int dst_base = a.req_dst_base[r];
        const int nbt0 = a.new_bt_offsets[r];
        if (adm) {
            // destinations follow the kept blocks in the new block table
            for (int j = tid; j < need; j += TILE_NT) {
                int blk = a.free_blocks[dst_base + j];
                if ((int64_t)nbt0 + (nb - ns) + j < cap_bt) a.new_bt_blocks[nbt0 + (nb - ns) + j] = blk;
                if (blk < 0 || blk >= a.num_blocks) { flags |= VTOKEN_FLAG_BAD_FREE; blk = -1; }
                a.dst_blocks[dst_base + j] = blk;
            }
            for (int i = nsrc + tid; i < need * S; i += TILE_NT) a.dst_src[(int64_t)dst_base * S + i] = -1;
            // kept blocks in old order, unprotected sources to the reclaimed list and the protected blocks the
            // request leaves to the released list, each in old order
            const int f0 = a.req_freed_base[r];
            const int l0 = detach ? a.req_rel_base[r] : 0;
            const CowTable h{2 * b0, 2 * (b1 - b0)};
            int carry_src = 0, carry_rel = 0;
            for (int64_t jb = b0; jb < b1; jb += TILE_NT) {
                const int64_t j = jb + tid;
                int blk = -1;
                bool src = false, rel = false;
                if (j < b1) {
                    blk = a.bt_blocks[j];
                    if (blk >= 0 && blk < a.num_blocks) {
                        src = a.blk_src[blk] == 1;
                        if (a.rule == 2) rel = detach && a.blk_src[blk] == 2;
                        else rel = detach && a.protect[blk] != 0 && (a.rule == 0 || pp_cow_leaves(a, h, blk));
                    }
                }
                int total;
                const int rank_src = carry_src + vtk_block_rank<TILE_NT>(src, warp_sums, total);
                carry_src += total;
                int rank_rel = 0;
                if (detach) {                                   // uniform over the CTA
                    rank_rel = carry_rel + vtk_block_rank<TILE_NT>(rel, warp_sums, total);
                    carry_rel += total;
                }
                if (j < b1) {
                    const int64_t kept = (int64_t)nbt0 + (j - b0) - rank_src - rank_rel;   // entries before it that stay
                    if (src) { if ((int64_t)f0 + rank_src < cap_bt) a.freed_blocks[f0 + rank_src] = blk; }
                    else if (rel) { if ((int64_t)l0 + rank_rel < cap_bt) a.released_blocks[l0 + rank_rel] = blk; }
                    else if (kept < cap_bt) a.new_bt_blocks[kept] = blk;
                }
            }
        } else {
            for (int j = tid; j < nb && (int64_t)nbt0 + j < cap_bt; j += TILE_NT)
                a.new_bt_blocks[nbt0 + j] = a.bt_blocks[b0 + j];
        }
        if (flags) {
            atomicOr(&a.counts->error_flags, flags);
            atomicOr(&a.out_counts->error_flags, flags);
        }
        return;
    }

    // token table: moving tokens ranked in logical order -> destination slot; the others keep theirs
    const int64_t T = pp_offset(a, R);
    const int64_t base = (int64_t)blockIdx.x * TILE;
    if (base >= T) return;
    const int64_t t = base + tid * TILE_TOK;
    int32_t slot[TILE_TOK];
    bool bad = false;
    const unsigned bits = vtk_load_entries(a.tt_slots, a.keep, a.vec_in, t, pp_offset(a, 0), T, a.slots_per_layer, slot, bad);
    vtk_tile_owners(a.tt_offsets, R, a.max_tokens, base, T, tile_req);
    __syncthreads();
    int r = t < T ? vtk_entry_owner(a.tt_offsets, a.max_tokens, tile_req, t) : -1;
    // Live entries that sit in a source block of their request, by the rule the tile counts in tile_mov
    // were taken with (admission was not known then): inside an admitted request every one of them
    // moves, and ranks are only used there.
    const unsigned mov = pp_moving_bits(a, bits, slot, may_detach, R, t, r);
    const int cnt = __popc(mov);
    const int incl = vtk_warp_incl_scan(cnt);
    if (lane == 31) warp_sums[warp] = incl;
    __syncthreads();
    int before = a.tile_mov[blockIdx.x] + incl - cnt;        // such tokens of the whole table before entry t
    for (int w = 0; w < warp; ++w) before += warp_sums[w];
    if (t >= T) return;

    int64_t next = pp_offset(a, r + 1);                      // r + 1 <= R
    int req_before = 0, nsrc = 0, dst_base = 0;
    bool adm = false;
    auto load_request = [&]() {
        req_before = a.req_before[r];
        nsrc = a.req_nsrc[r];
        dst_base = a.req_dst_base[r];
        adm = a.req_status[r] == VTOKEN_REPACKED;
    };
    if (r >= 0) load_request();
    int32_t out[TILE_TOK];
    bool owned = true;
#pragma unroll
    for (int k = 0; k < TILE_TOK; ++k) {
        out[k] = -1;
        if (t + k >= T) { owned = false; continue; }
        if (t + k >= next && r + 1 < R) {                     // a request boundary inside the thread's entries
            while (r + 1 < R && pp_offset(a, r + 1) <= t + k) ++r;
            next = pp_offset(a, r + 1);
            load_request();
        }
        if (r < 0) { owned = false; continue; }               // in front of the first request: left untouched
        if (!((bits >> k) & 1u)) continue;                    // dead or unmapped: -1
        if (!adm || !((mov >> k) & 1u)) { out[k] = slot[k]; continue; }   // its block stays in place
        const int i = before + __popc(mov & ((1u << k) - 1u)) - req_before;   // rank among the request's movers
        if (i < 0 || i >= nsrc) continue;                     // only with inconsistent offsets
        const int j = i / S, off = i - j * S;
        const int blk = a.free_blocks[dst_base + j];
        out[k] = blk * S + off;
        a.dst_src[(int64_t)(dst_base + j) * S + off] = slot[k];
    }
    if (owned && a.vec_out) {
        *reinterpret_cast<int4 *>(a.new_tt_slots.at(t, TILE_TOK)) = make_int4(out[0], out[1], out[2], out[3]);
    } else {
        const int64_t first = pp_offset(a, 0);
#pragma unroll
        for (int k = 0; k < TILE_TOK; ++k)
            if (t + k < T && t + k >= first) a.new_tt_slots[t + k] = out[k];
    }
}

// ---- histogram of block utilisation ------------------------------------------------------------
constexpr int PP_HIST_BINS = 1024;      // bins a CTA keeps in shared memory (block sizes up to 1023)

__global__ void __launch_bounds__(256) pp_hist_kernel(const int32_t *num_requests, int32_t max_requests,
                                                      const int32_t *bt_offsets, const int32_t *bt_blocks,
                                                      const int32_t *n_b, int32_t S, int32_t num_blocks,
                                                      unsigned long long *hist, vtoken_counts *counts)
{
    vtk_release_successor();
    vtk_wait_for_predecessor();
    // a handful of bins takes every increment: counted per CTA in shared memory first, one global
    // atomic per non-empty bin and CTA afterwards (integer sums: the order does not matter)
    __shared__ unsigned int bins[PP_HIST_BINS];
    const bool local = S < PP_HIST_BINS;
    if (local)
        for (int k = threadIdx.x; k <= S; k += 256) bins[k] = 0;
    __syncthreads();
    int R = *num_requests;
    R = R < 0 ? 0 : (R > max_requests ? max_requests : R);
    const int total = bt_offsets[R];
    bool bad = false;
    for (int j = blockIdx.x * 256 + threadIdx.x; j < total; j += gridDim.x * 256) {
        const int blk = bt_blocks[j];
        if (blk < 0 || blk >= num_blocks) { bad = true; continue; }
        int k = n_b[blk];
        if (k > S) k = S;
        if (local) atomicAdd(&bins[k], 1u);
        else atomicAdd(&hist[k], 1ull);
    }
    if (bad) atomicOr(&counts->error_flags, VTOKEN_FLAG_BAD_BLOCK);
    __syncthreads();
    if (local)
        for (int k = threadIdx.x; k <= S; k += 256)
            if (bins[k] != 0) atomicAdd(&hist[k], (unsigned long long)bins[k]);
}

__global__ void __launch_bounds__(1024) pp_summary_kernel(const int32_t *num_requests, int32_t max_requests,
                                                          const int32_t *bt_offsets, const int32_t *tt_offsets,
                                                          int64_t max_tokens, const int32_t *tile_live,
                                                          long long *summary)
{
    vtk_release_successor();
    vtk_wait_for_predecessor();
    // one CTA: total live tokens over all tiles (the sign bit of a count is a flag), allocated blocks
    __shared__ long long warp_s[32];
    int R = *num_requests;
    R = R < 0 ? 0 : (R > max_requests ? max_requests : R);
    const int64_t T = vtk_clipped_offset(tt_offsets, R, max_tokens);
    const int tiles = (int)((T + TILE - 1) / TILE);
    long long s = 0;
    for (int i = threadIdx.x; i < tiles; i += 1024) s += tile_live[i] & 0x7fffffff;
#pragma unroll
    for (int d = 16; d > 0; d >>= 1) s += __shfl_down_sync(0xffffffffu, s, d);
    if (vtk_lane() == 0) warp_s[threadIdx.x >> 5] = s;
    __syncthreads();
    if (threadIdx.x < 32) {
        s = warp_s[threadIdx.x];
#pragma unroll
        for (int d = 16; d > 0; d >>= 1) s += __shfl_down_sync(0xffffffffu, s, d);
        if (threadIdx.x == 0) {
            summary[0] = s;
            summary[1] = bt_offsets[R];
        }
    }
}

void fill_args(PArgs &a, vtoken_ctx *ctx)
{
    const vtoken_config &c = ctx->cfg;
    const int64_t tiles_cap = (c.max_tokens + TILE - 1) / TILE + 1, r1 = (int64_t)c.max_requests + 1;
    a.req_n = VTK_ARR(ctx, ctx->req_n, c.max_requests);
    a.tile_live = VTK_ARR(ctx, ctx->tile_n, tiles_cap);
    a.tile_mov = VTK_ARR(ctx, ctx->tile_mov, tiles_cap);
    a.tile_shared = VTK_ARR(ctx, ctx->tile_shared, tiles_cap);
    a.part_live = VTK_ARR(ctx, ctx->req_part, r1);
    a.part_mov = VTK_ARR(ctx, ctx->part_mov, r1);
    a.req_before = VTK_ARR(ctx, ctx->req_before, r1);
    a.req_ns = VTK_ARR(ctx, ctx->req_ns, c.max_requests);
    a.req_nsrc = VTK_ARR(ctx, ctx->req_nsrc, c.max_requests);
    a.req_dst_base = VTK_ARR(ctx, ctx->req_dst_base, c.max_requests);
    a.req_freed_base = VTK_ARR(ctx, ctx->req_freed_base, c.max_requests);
    a.req_status = VTK_ARR(ctx, ctx->req_status, c.max_requests);
    a.dst_src = VTK_ARR(ctx, ctx->dst_src, (int64_t)ctx->cap_dst_blocks * c.block_size);
    a.dst_blocks = VTK_ARR(ctx, ctx->dst_blocks, ctx->cap_dst_blocks);
    a.n_b = VTK_ARR(ctx, ctx->n_b, c.num_blocks);
    a.blk_src = VTK_ARR(ctx, ctx->blk_src, c.num_blocks);
    a.part_shared = VTK_ARR(ctx, ctx->part_shared, r1);
    a.req_shared = VTK_ARR(ctx, ctx->req_shared, c.max_requests);
    a.req_detach = VTK_ARR(ctx, ctx->req_detach, c.max_requests);
    a.req_rel_base = VTK_ARR(ctx, ctx->req_rel_base, c.max_requests);
    a.cow = VTK_ARR(ctx, ctx->cow, 2 * (int64_t)c.max_table_blocks);
    a.rule = 0;
    a.counts = VTK_ARR(ctx, ctx->counts, 1);
    a.S = ctx->cfg.block_size;
    a.num_blocks = ctx->cfg.num_blocks;
    a.max_requests = ctx->cfg.max_requests;
    a.cap_dst_blocks = ctx->cap_dst_blocks;
    a.max_free_blocks = ctx->cfg.max_free_blocks;
    a.slots_per_layer = ctx->slots_per_layer;
    a.max_tokens = ctx->cfg.max_tokens;
    a.max_table_blocks = ctx->cfg.max_table_blocks;
    a.num_tiles = (int32_t)((ctx->cfg.max_tokens + TILE - 1) / TILE);
    a.vec_in = a.vec_out = 0;
}

}  // namespace

extern "C" {

int vtoken_plan_partial(vtoken_ctx *ctx, const vtoken_plan_in *in, const vtoken_partial_opts *opts,
                        const vtoken_plan_out *out, void *cuda_stream)
{
    if (!ctx || !in || !opts || !out) return VTOKEN_EINVAL;
    if (!in->num_requests || !in->bt_offsets || !in->bt_blocks || !in->tt_offsets || !in->tt_slots || !in->keep ||
        !in->free_blocks || !in->num_free)
        return VTOKEN_EINVAL;
    if (!out->new_bt_offsets || !out->new_bt_blocks || !out->new_tt_slots || !out->freed_blocks ||
        !out->req_status || !out->counts)
        return VTOKEN_EINVAL;
    if (opts->max_source_blocks < 0 || opts->detach_rule > 2) return VTOKEN_EINVAL;
    if (opts->protect != nullptr && opts->detach_den != 0 && !out->released_blocks) return VTOKEN_EINVAL;
    cudaStream_t st = (cudaStream_t)cuda_stream;
    PArgs a{};
    fill_args(a, ctx);
    const vtoken_config &c = ctx->cfg;
    a.num_requests = VTK_ARR(ctx, in->num_requests, 1);
    a.bt_offsets = VTK_ARR(ctx, in->bt_offsets, (int64_t)c.max_requests + 1);
    a.bt_blocks = VTK_ARR(ctx, in->bt_blocks, c.max_table_blocks);
    a.tt_offsets = VTK_ARR(ctx, in->tt_offsets, (int64_t)c.max_requests + 1);
    a.tt_slots = VTK_ARR(ctx, in->tt_slots, c.max_tokens);
    a.keep = VTK_ARR(ctx, in->keep, c.max_tokens);
    a.select = VTK_ARR(ctx, in->select, c.max_requests);
    a.protect = VTK_ARR(ctx, opts->protect, c.num_blocks);
    a.thr_num = in->thr_num;
    a.thr_den = in->thr_den;
    a.util_num = opts->util_num;
    a.util_den = opts->util_den;
    a.theta_num = opts->theta_num;
    a.theta_den = opts->theta_den;
    a.detach_num = opts->detach_num;
    a.detach_den = opts->detach_den;
    a.rule = (opts->protect != nullptr && opts->detach_den != 0) ? opts->detach_rule : 0u;
    a.max_sources = opts->max_source_blocks;
    a.free_blocks = VTK_ARR(ctx, in->free_blocks, c.max_free_blocks);
    a.num_free = VTK_ARR(ctx, in->num_free, 1);
    a.new_bt_offsets = VTK_ARR(ctx, out->new_bt_offsets, (int64_t)c.max_requests + 1);
    a.new_bt_blocks = VTK_ARR(ctx, out->new_bt_blocks, c.max_table_blocks);
    a.new_tt_slots = VTK_ARR(ctx, out->new_tt_slots, c.max_tokens);
    a.freed_blocks = VTK_ARR(ctx, out->freed_blocks, c.max_table_blocks);
    a.released_blocks = VTK_ARR(ctx, out->released_blocks, c.max_table_blocks);
    a.out_status = VTK_ARR(ctx, out->req_status, c.max_requests);
    a.out_counts = VTK_ARR(ctx, out->counts, 1);

    a.vec_in = ((uintptr_t)in->tt_slots % 16 == 0 && (uintptr_t)in->keep % 4 == 0) ? 1 : 0;
    a.vec_out = ((uintptr_t)out->new_tt_slots % 16 == 0) ? 1 : 0;
#ifdef VTOKEN_CHECKED
    a.vec_in = a.vec_out = 0;      // one checked access per entry instead of one per four
#endif

    const int R = ctx->cfg.max_requests;
    const dim3 tiles_grid(a.num_tiles + R + 1);
    VTK_CUDA(ctx, cudaMemsetAsync(ctx->counts, 0, sizeof(vtoken_counts), st));
    // n_b and blk_src share one allocation: one node clears both
    VTK_CUDA(ctx, cudaMemsetAsync(ctx->n_b, 0, (sizeof(int32_t) + 1) * (size_t)ctx->cfg.num_blocks, st));
    if (a.rule == 1) {
        VTK_CUDA(ctx, cudaMemsetAsync(ctx->cow, 0, sizeof(unsigned long long) * 2 * (size_t)c.max_table_blocks, st));
        VTK_CUDA(ctx, vtk_launch_dependent(ctx, pp_cow_insert_kernel, dim3(R), dim3(256), 0, st, a));
    }
    VTK_CUDA(ctx, vtk_launch_dependent(ctx, pp_tiles_kernel<0>, tiles_grid, dim3(TILE_NT), 0, st, a));
    VTK_CUDA(ctx, vtk_launch_dependent(ctx, pp_blocks_kernel, dim3(R), dim3(PP_NT), 0, st, a));
    VTK_CUDA(ctx, vtk_launch_dependent(ctx, pp_tiles_kernel<1>, tiles_grid, dim3(TILE_NT), 0, st, a));
    VTK_CUDA(ctx, vtk_launch_dependent(ctx, pp_scan_kernel, dim3(1), dim3(PP_SCAN_NT), 0, st, a));
    VTK_CUDA(ctx, vtk_launch_dependent(ctx, pp_assign_kernel, dim3(a.num_tiles + R), dim3(TILE_NT), 0, st, a));
    VTK_CUDA(ctx, cudaGetLastError());
    ctx->has_plan = true;
    return VTOKEN_OK;
}

int vtoken_block_liveness(vtoken_ctx *ctx, const int32_t *num_requests, const int32_t *bt_offsets,
                          const int32_t *bt_blocks, const int32_t *tt_offsets, const int32_t *tt_slots,
                          const uint8_t *keep, int32_t *n_b, uint64_t *hist, int64_t *summary, void *cuda_stream)
{
    if (!ctx || !num_requests || !bt_offsets || !bt_blocks || !tt_offsets || !tt_slots || !n_b) return VTOKEN_EINVAL;
    cudaStream_t st = (cudaStream_t)cuda_stream;
    PArgs a{};                                   // the planning options stay zero: only the counting pass runs
    fill_args(a, ctx);
    const vtoken_config &c = ctx->cfg;
    a.num_requests = VTK_ARR(ctx, num_requests, 1);
    a.bt_offsets = VTK_ARR(ctx, bt_offsets, (int64_t)c.max_requests + 1);
    a.bt_blocks = VTK_ARR(ctx, bt_blocks, c.max_table_blocks);
    a.tt_offsets = VTK_ARR(ctx, tt_offsets, (int64_t)c.max_requests + 1);
    a.tt_slots = VTK_ARR(ctx, tt_slots, c.max_tokens);
    a.keep = VTK_ARR(ctx, keep, c.max_tokens);
    a.n_b = VTK_ARR(ctx, n_b, c.num_blocks);
    const int R = ctx->cfg.max_requests;
    VTK_CUDA(ctx, cudaMemsetAsync(n_b, 0, sizeof(int32_t) * (size_t)ctx->cfg.num_blocks, st));
    a.vec_in = ((uintptr_t)tt_slots % 16 == 0 && (uintptr_t)keep % 4 == 0) ? 1 : 0;
#ifdef VTOKEN_CHECKED
    a.vec_in = 0;
#endif
    VTK_CUDA(ctx, vtk_launch_dependent(ctx, pp_tiles_kernel<0>, dim3(a.num_tiles + R + 1), dim3(TILE_NT), 0, st, a));
    if (hist) {
        VTK_CUDA(ctx, cudaMemsetAsync(hist, 0, sizeof(uint64_t) * (size_t)(ctx->cfg.block_size + 1), st));
        VTK_CUDA(ctx, vtk_launch_dependent(ctx, pp_hist_kernel, dim3(ctx->num_sms * 4), dim3(256), 0, st, num_requests, R,
                                           bt_offsets, bt_blocks, (const int32_t *)n_b, ctx->cfg.block_size,
                                           ctx->cfg.num_blocks, (unsigned long long *)hist, ctx->counts));
    }
    if (summary)
        VTK_CUDA(ctx, vtk_launch_dependent(ctx, pp_summary_kernel, dim3(1), dim3(1024), 0, st, num_requests, R, bt_offsets,
                                           tt_offsets, ctx->cfg.max_tokens, (const int32_t *)ctx->tile_n,
                                           (long long *)summary));
    VTK_CUDA(ctx, cudaGetLastError());
    return VTOKEN_OK;
}

}  // extern "C"
