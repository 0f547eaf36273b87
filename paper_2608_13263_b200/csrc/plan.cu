// Relocation planner (Sec. 3.3.3 of the paper) as three small kernels over a flat tiling of the
// token table:
//   tiles  : live tokens per tile of 1024 consecutive table entries (four per thread, vector
//            loads), and for every request the live tokens between the start of its first tile and
//            its first entry
//   scan   : running live count at every tile start; live tokens per request as a difference of
//            two running counts; candidates, admission against the free list, per-request bases,
//            counts (one CTA)
//   assign : rank of every live token inside its request = running count at the token minus the
//            running count at the request's first entry -> destination slot, new token table,
//            inverse move plan for the copy kernel; extra CTAs (one per request) write the new
//            block tables and the reclaimed list
// The tiling ignores request boundaries, so the work per CTA is the same whatever the mix of
// request lengths (512 short requests or 32 long ones), and every CTA keeps four table entries
// per thread in flight.  All grids are fixed by the capacities; R, T and num_free are read from
// device memory.  No output order depends on atomics.
#include "common.cuh"

namespace {

constexpr int TILE_NT = VTK_TILE_NT;             // threads per CTA of tiles / assign
constexpr int TILE_TOK = VTK_TILE_TOK;           // table entries per thread
constexpr int TILE = VTK_TILE;                   // entries per tile
constexpr int SCAN_NT = 1024;                    // threads of the single scan CTA

struct PlanArgs {
    // inputs
    vtk_arr<const int32_t> num_requests, bt_offsets, bt_blocks, tt_offsets, tt_slots;
    vtk_arr<const uint8_t> keep, select;
    uint32_t thr_num, thr_den;
    vtk_arr<const int32_t> free_blocks, num_free;
    // outputs
    vtk_arr<int32_t> new_bt_offsets, new_bt_blocks, new_tt_slots, freed_blocks, out_status;
    vtk_arr<vtoken_counts> out_counts;
    // context
    vtk_arr<int32_t> req_n, req_dst_base, req_freed_base, req_status, dst_src, dst_blocks;
    vtk_arr<int32_t> tile_n;  // [num_tiles + 1] live tokens per tile (sign bit: a slot outside the pool); after the
                              // scan: live tokens before the tile
    vtk_arr<int32_t> req_part;    // [max_requests + 1] live tokens between the start of the tile that holds the
                                  // request's first entry and that entry
    vtk_arr<int32_t> req_before;  // [max_requests + 1] live tokens before the request's first entry
    vtk_arr<int32_t> header;      // [4] R, T, num_free, first entry as the tiles kernel read them: one load for the
                                  // kernels behind it instead of a chain of dependent ones
    vtk_arr<vtoken_counts> counts;
    int32_t S, num_blocks, max_requests, cap_dst_blocks, max_free_blocks, num_tiles;
    int32_t vec_in, vec_out;   // tt_slots 16-byte / keep 4-byte aligned; new_tt_slots 16-byte aligned
    int64_t slots_per_layer, max_tokens, max_table_blocks;
};

__device__ __forceinline__ int clamp_requests(const PlanArgs &a)
{
    int R = *a.num_requests;
    return R < 0 ? 0 : (R > a.max_requests ? a.max_requests : R);
}

__device__ __forceinline__ int64_t clipped_offset(const PlanArgs &a, int r)
{
    return vtk_clipped_offset(a.tt_offsets, r, a.max_tokens);
}

__device__ __forceinline__ void raise_flags(const PlanArgs &a, uint32_t flags)
{
    atomicOr(&a.counts->error_flags, flags);
    atomicOr(&a.out_counts->error_flags, flags);
}

// ---- tiles -----------------------------------------------------------------------------
constexpr int TILES_PER_CTA = 4;                 // tiles a counting CTA takes: the loads of all of them are in flight
                                                 // together, and the grid of a 2 M-entry table is one wave

__host__ __device__ __forceinline__ int tile_ctas(int num_tiles) { return (num_tiles + TILES_PER_CTA - 1) / TILES_PER_CTA; }

__global__ void __launch_bounds__(TILE_NT) plan_tiles_kernel(PlanArgs a)
{
    __shared__ int warp_n[TILES_PER_CTA][TILE_NT / 32];
    __shared__ unsigned int bad_tiles;
    vtk_release_successor();
    vtk_wait_for_predecessor();
    const int R = clamp_requests(a);
    const int64_t T = clipped_offset(a, R);
    const int64_t first = clipped_offset(a, 0);
    const int lane = vtk_lane(), warp = threadIdx.x >> 5;
    if (blockIdx.x == 0 && threadIdx.x == 0) {
        a.header[0] = R;
        a.header[1] = (int32_t)T;
        a.header[2] = *a.num_free;
        a.header[3] = (int32_t)first;
    }
    if (threadIdx.x == 0) bad_tiles = 0u;
    const int n_tile_ctas = tile_ctas(a.num_tiles);
    if ((int)blockIdx.x < n_tile_ctas) {
        // TILES_PER_CTA consecutive tiles, every entry of the table exactly once
        const int tile0 = (int)blockIdx.x * TILES_PER_CTA;
        if ((int64_t)tile0 * TILE >= T) return;
        int n[TILES_PER_CTA];
        unsigned bad_bits = 0;
#pragma unroll
        for (int k = 0; k < TILES_PER_CTA; ++k) {
            const int64_t base = (int64_t)(tile0 + k) * TILE;
            int32_t slot[TILE_TOK];
            bool bad = false;
            n[k] = base < T ? __popc(vtk_load_entries(a.tt_slots, a.keep, a.vec_in, base + threadIdx.x * TILE_TOK, first, T,
                                                      a.slots_per_layer, slot, bad))
                            : 0;
            if (bad) bad_bits |= 1u << k;
        }
#pragma unroll
        for (int k = 0; k < TILES_PER_CTA; ++k) {
#pragma unroll
            for (int d = 16; d > 0; d >>= 1) n[k] += __shfl_down_sync(0xffffffffu, n[k], d);
            if (lane == 0) warp_n[k][warp] = n[k];
        }
        __syncthreads();                                  // (bad_tiles is zero by now)
        if (bad_bits) atomicOr(&bad_tiles, bad_bits);
        __syncthreads();
        if (threadIdx.x < TILES_PER_CTA && (int64_t)(tile0 + threadIdx.x) * TILE < T) {
            const int k = threadIdx.x;
            int s = 0;
#pragma unroll
            for (int w = 0; w < TILE_NT / 32; ++w) s += warp_n[k][w];
            // a slot outside the pool somewhere in the tile travels in the sign bit (the count is at most
            // 1024): the scan kernel turns it into VTOKEN_FLAG_BAD_SLOT, and nothing has to be zeroed
            // before this kernel
            a.tile_n[tile0 + k] = s | (((bad_tiles >> k) & 1u) ? (int)0x80000000 : 0);
        }
        return;
    }
    // the CTAs behind those, one per request boundary: the live entries between the start of the boundary's
    // tile and the boundary (entries the tile's own CTA counts as well; flags are raised there)
    const int r = (int)blockIdx.x - n_tile_ctas;
    if (r > R) return;
    const int64_t limit = clipped_offset(a, r);
    const int64_t base = limit / TILE * TILE;
    if (base == limit) return;                           // nothing in front of it: the scan does not read req_part[r]
    bool bad = false;
    int32_t slot[TILE_TOK];
    int n = __popc(vtk_load_entries(a.tt_slots, a.keep, a.vec_in, base + threadIdx.x * TILE_TOK, first, limit,
                                    a.slots_per_layer, slot, bad));
#pragma unroll
    for (int d = 16; d > 0; d >>= 1) n += __shfl_down_sync(0xffffffffu, n, d);
    if (lane == 0) warp_n[0][warp] = n;
    __syncthreads();
    if (threadIdx.x == 0) {
        int s = 0;
#pragma unroll
        for (int w = 0; w < TILE_NT / 32; ++w) s += warp_n[0][w];
        a.req_part[r] = s;
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

constexpr int SCAN_STAGED = 8192;                // running counts of that many tiles are kept in shared memory

// What the scan reads from global memory for one request, requested in one go.
struct ScanInputs {
    int tt0, tt1, bt0, bt1, part0, part1;
    unsigned char sel;
};
__device__ __forceinline__ ScanInputs load_scan_inputs(const PlanArgs &a, int r, int R)
{
    ScanInputs in{0, 0, 0, 0, 0, 0, 1};
    if (r < R) {
        in.tt0 = a.tt_offsets[r];
        in.tt1 = a.tt_offsets[r + 1];
        in.bt0 = a.bt_offsets[r];
        in.bt1 = a.bt_offsets[r + 1];
        in.part0 = a.req_part[r];          // (scratch of the tiles kernel: only used when the offset is inside a tile)
        in.part1 = a.req_part[r + 1];
        if (!a.select.null()) in.sel = a.select[r];
    }
    return in;
}

__global__ void __launch_bounds__(SCAN_NT) plan_scan_kernel(PlanArgs a)
{
    __shared__ long long warp_ll[32];
    __shared__ Acc warp_acc[32];
    __shared__ long long carry_need;
    __shared__ Acc carry;
    __shared__ int warp_i[32];
    __shared__ unsigned int all_flags;
    __shared__ int staged[SCAN_STAGED + 1];
    const int tid = threadIdx.x;
    vtk_release_successor();
    vtk_wait_for_predecessor();
    // R, T and num_free in one load; the inputs of the first 1024 requests and the tile counts are requested
    // right behind it, before anything is computed
    const int4 hdr = *reinterpret_cast<const int4 *>(a.header.at(0, 4));
    const int R = hdr.x;
    const int64_t T = hdr.y;
    int nf = hdr.z;
    uint32_t flags = 0;
    if (tid == 0) {
        const int raw = *a.num_requests;
        if (raw > a.max_requests || raw < 0) flags |= VTOKEN_FLAG_CAPACITY;
        if (nf > a.max_free_blocks) flags |= VTOKEN_FLAG_CAPACITY;
        carry_need = 0;
        all_flags = 0;
        carry = Acc{0, 0, 0, 0, 0, 0};
    }
    nf = nf < 0 ? 0 : (nf > a.cap_dst_blocks ? a.cap_dst_blocks : nf);
    ScanInputs in = load_scan_inputs(a, tid, R);

    auto shfl_ll = [](long long v, int d) { return __shfl_up_sync(0xffffffffu, v, d); };
    auto shfl_acc = [](const Acc &v, int d) { return shfl_up(v, d); };
    auto shfl_int = [](int v, int d) { return __shfl_up_sync(0xffffffffu, v, d); };

    // live tokens before every tile (in place: tile_n[i] becomes the sum of the tiles before i; one entry
    // past the last tile holds the total): every thread sums a run of consecutive tiles, one scan over the
    // runs, every thread writes the running counts of its run -- to global memory for the assign kernel
    // and, while they fit, to shared memory for the request pass below
    const int tiles = (int)((T + TILE - 1) / TILE);
    const bool fits = tiles <= SCAN_STAGED;
    {
        const int per = (tiles + 1 + SCAN_NT - 1) / SCAN_NT;
        const int j0 = min(tiles + 1, tid * per), j1 = min(tiles + 1, j0 + per);
        int sum = 0, any = 0;
        if (per <= 4) {
            int v[4];
#pragma unroll
            for (int k = 0; k < 4; ++k) v[k] = (j0 + k < j1 && j0 + k < tiles) ? a.tile_n[j0 + k] : 0;
#pragma unroll
            for (int k = 0; k < 4; ++k) { sum += v[k] & 0x7fffffff; any |= v[k]; }
            __syncthreads();                                       // (carry_need, carry, all_flags are set)
            int run = vtk_block_incl_scan<int>(sum, warp_i, 0, shfl_int) - sum;
#pragma unroll
            for (int k = 0; k < 4; ++k) {
                if (j0 + k < j1) {
                    a.tile_n[j0 + k] = run;
                    if (fits) staged[j0 + k] = run;
                }
                run += v[k] & 0x7fffffff;
            }
        } else {
            for (int j = j0; j < j1; ++j) { const int v = j < tiles ? a.tile_n[j] : 0; sum += v & 0x7fffffff; any |= v; }
            __syncthreads();
            int run = vtk_block_incl_scan<int>(sum, warp_i, 0, shfl_int) - sum;
            for (int j = j0; j < j1; ++j) {
                const int v = j < tiles ? (a.tile_n[j] & 0x7fffffff) : 0;
                a.tile_n[j] = run;
                if (fits) staged[j] = run;
                run += v;
            }
        }
        if (any < 0) flags |= VTOKEN_FLAG_BAD_SLOT;
    }
    __syncthreads();
    const int32_t *before_tile = fits ? staged : a.tile_n.at(0, (int64_t)tiles + 1);
    auto clip = [](int64_t o, int64_t cap) { return o < 0 ? (int64_t)0 : (o > cap ? cap : o); };
    // live tokens before table entry o = live tokens before its tile + those between the tile's start and o
    auto live_before = [&](int64_t o, int part) { return before_tile[o / TILE] + (o % TILE != 0 ? part : 0); };

    for (int base = 0; base < R; base += SCAN_NT) {
        const int r = base + tid;
        const bool valid = r < R;
        if (base > 0) in = load_scan_inputs(a, r, R);
        int n = 0, nb = 0;
        if (valid) {
            // table ranges clipped to the create-time capacities (a range that runs backwards is empty)
            const int64_t t0 = clip(in.tt0, a.max_tokens), t1 = clip(in.tt1, a.max_tokens);
            const int64_t lo = clip(in.bt0, a.max_table_blocks), b1 = clip(in.bt1, a.max_table_blocks);
            const int64_t hi = b1 < lo ? lo : b1;
            if (lo != in.bt0 || hi != in.bt1 || t0 != in.tt0 || (t1 < t0 ? t0 : t1) != in.tt1) flags |= VTOKEN_FLAG_CAPACITY;
            const int before = live_before(t0, in.part0);
            n = live_before(t1, in.part1) - before;
            if (n < 0) n = 0;                                // offsets that run backwards
            a.req_before[r] = before;
            a.req_n[r] = n;
            nb = (int)(hi - lo);
        }
        const int need = (int)(((int64_t)n + a.S - 1) / a.S);       // ceil(T_live / S)
        bool sel = valid && in.sel != 0;
        if (sel && a.thr_den != 0)
            sel = (unsigned long long)n * a.thr_den <
                  (unsigned long long)a.thr_num * (unsigned long long)nb * (unsigned long long)a.S;
        const bool cand = sel && need < nb;                          // strictly fewer blocks afterwards
        // admission: cumulative demand of candidates so far (this one included) fits the free list
        const long long cum = vtk_block_incl_scan<long long>(cand ? need : 0, warp_ll, 0LL, shfl_ll) + carry_need;
        const bool adm = cand && cum <= (long long)nf;
        const int status = !sel ? VTOKEN_NOT_SELECTED
                                : (!cand ? VTOKEN_NO_GAIN : (adm ? VTOKEN_REPACKED : VTOKEN_DEFERRED_NO_FREE));
        Acc mine{adm ? need : 0, adm ? nb : 0, valid ? (adm ? need : nb) : 0, adm ? n : 0, adm ? 1 : 0,
                 (cand && !adm) ? 1 : 0};
        const Acc incl = vtk_block_incl_scan<Acc>(mine, warp_acc, Acc{0, 0, 0, 0, 0, 0}, shfl_acc) + carry;
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
    if (flags) atomicOr(&all_flags, flags);
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
        c.error_flags = all_flags;                       // whatever an earlier plan or copy left is overwritten
        c.num_released = 0;
        *a.counts = c;
        *a.out_counts = c;                               // later flags are OR-ed into both copies
    }
}

// ---- assign ----------------------------------------------------------------------------
__global__ void __launch_bounds__(TILE_NT, 8) plan_assign_kernel(PlanArgs a)
{
    __shared__ int warp_sums[TILE_NT / 32];
    __shared__ int tile_req[2];
    vtk_release_successor();
    vtk_wait_for_predecessor();
    const int4 hdr = *reinterpret_cast<const int4 *>(a.header.at(0, 4));      // R, T, num_free, first entry
    const int R = hdr.x;
    const int tid = threadIdx.x, lane = vtk_lane(), warp = tid >> 5;
    const int S = a.S;
    uint32_t flags = 0;

    if ((int)blockIdx.x >= a.num_tiles) {
        // block table and reclaimed list of one request
        const int r = (int)blockIdx.x - a.num_tiles;
        if (r >= R) return;
        int64_t b0, b1;
        vtk_range(a.bt_offsets, r, a.max_table_blocks, b0, b1);
        const int nb = (int)(b1 - b0);
        const int nbt0 = a.new_bt_offsets[r];
        if (a.req_status[r] == VTOKEN_REPACKED) {
            const int n = a.req_n[r];
            const int need = (int)(((int64_t)n + S - 1) / S);
            const int dst_base = a.req_dst_base[r];
            for (int j = tid; j < need; j += TILE_NT) {
                int blk = a.free_blocks[dst_base + j];
                if ((int64_t)nbt0 + j < a.max_table_blocks) a.new_bt_blocks[nbt0 + j] = blk;
                if (blk < 0 || blk >= a.num_blocks) { flags |= VTOKEN_FLAG_BAD_FREE; blk = -1; }
                a.dst_blocks[dst_base + j] = blk;
            }
            const int f0 = a.req_freed_base[r];
            for (int j = tid; j < nb && (int64_t)f0 + j < a.max_table_blocks; j += TILE_NT) {
                const int blk = a.bt_blocks[b0 + j];
                if (blk < 0 || blk >= a.num_blocks) flags |= VTOKEN_FLAG_BAD_BLOCK;
                a.freed_blocks[f0 + j] = blk;
            }
            // unused tail of the last destination block
            for (int i = n + tid; i < need * S; i += TILE_NT) a.dst_src[(int64_t)dst_base * S + i] = -1;
        } else {
            for (int j = tid; j < nb && (int64_t)nbt0 + j < a.max_table_blocks; j += TILE_NT)
                a.new_bt_blocks[nbt0 + j] = a.bt_blocks[b0 + j];
        }
        if (flags) raise_flags(a, flags);
        return;
    }

    // token table: rank of each live token in logical order -> destination slot
    const int64_t T = hdr.y, first = hdr.w;
    const int64_t base = (int64_t)blockIdx.x * TILE;
    if (base >= T) return;
    const int64_t t = base + tid * TILE_TOK;
    int32_t slot[TILE_TOK];
    bool bad = false;
    const unsigned bits = vtk_load_entries(a.tt_slots, a.keep, a.vec_in, t, first, T, a.slots_per_layer, slot, bad);
    // live tokens of the whole table before this thread's first entry
    const int cnt = __popc(bits);
    const int incl = vtk_warp_incl_scan(cnt);
    if (lane == 31) warp_sums[warp] = incl;
    vtk_tile_owners(a.tt_offsets, R, a.max_tokens, base, T, tile_req);
    __syncthreads();
    int before = a.tile_n[blockIdx.x] + incl - cnt;
    for (int w = 0; w < warp; ++w) before += warp_sums[w];
    if (t >= T) return;

    int r = vtk_entry_owner(a.tt_offsets, a.max_tokens, tile_req, t);      // -1: in front of the first request
    int64_t next = r + 1 <= R ? clipped_offset(a, r + 1) : T;
    int req_before = 0, n = 0, dst_base = 0;
    bool adm = false;
    auto load_request = [&]() {
        req_before = a.req_before[r];
        n = a.req_n[r];
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
        if (t + k >= next) {                                  // a request boundary inside the thread's entries
            while (r + 1 < R && clipped_offset(a, r + 1) <= t + k) ++r;
            next = clipped_offset(a, r + 1);
            if (r >= 0) load_request();
        }
        if (r < 0) { owned = false; continue; }
        if (!((bits >> k) & 1u)) continue;                    // dead or unmapped: -1
        if (!adm) { out[k] = slot[k]; continue; }            // the request keeps its layout
        const int i = before + __popc(bits & ((1u << k) - 1u)) - req_before;   // rank inside the request
        if (i < 0 || i >= n) continue;                        // only with inconsistent offsets
        const int j = i / S, off = i - j * S;
        const int blk = a.free_blocks[dst_base + j];
        out[k] = blk * S + off;                               // slot = block_id * S + offset
        a.dst_src[(int64_t)(dst_base + j) * S + off] = slot[k];
    }
    if (owned && a.vec_out) {
        *reinterpret_cast<int4 *>(a.new_tt_slots.at(t, TILE_TOK)) = make_int4(out[0], out[1], out[2], out[3]);
    } else {
        // the ragged end of the table, or entries in front of the first request (left untouched)
#pragma unroll
        for (int k = 0; k < TILE_TOK; ++k)
            if (t + k < T && t + k >= first) a.new_tt_slots[t + k] = out[k];
    }
}

}  // namespace

int vtk_launch_plan(vtoken_ctx *ctx, const vtoken_plan_in *in, const vtoken_plan_out *out, cudaStream_t st)
{
    // the two-kernel form (plan_small.cu; vtk_configure_plan chose at create time)
    if (ctx->plan_form == 2) return vtk_launch_plan_small(ctx, in, out, st);
    PlanArgs a{};
    const vtoken_config &c = ctx->cfg;
    const int64_t tiles_cap = (c.max_tokens + TILE - 1) / TILE;
    a.num_requests = VTK_ARR(ctx, in->num_requests, 1);
    a.bt_offsets = VTK_ARR(ctx, in->bt_offsets, (int64_t)c.max_requests + 1);
    a.bt_blocks = VTK_ARR(ctx, in->bt_blocks, c.max_table_blocks);
    a.tt_offsets = VTK_ARR(ctx, in->tt_offsets, (int64_t)c.max_requests + 1);
    a.tt_slots = VTK_ARR(ctx, in->tt_slots, c.max_tokens);
    a.keep = VTK_ARR(ctx, in->keep, c.max_tokens);
    a.select = VTK_ARR(ctx, in->select, c.max_requests);
    a.thr_num = in->thr_num;
    a.thr_den = in->thr_den;
    a.free_blocks = VTK_ARR(ctx, in->free_blocks, c.max_free_blocks);
    a.num_free = VTK_ARR(ctx, in->num_free, 1);
    a.new_bt_offsets = VTK_ARR(ctx, out->new_bt_offsets, (int64_t)c.max_requests + 1);
    a.new_bt_blocks = VTK_ARR(ctx, out->new_bt_blocks, c.max_table_blocks);
    a.new_tt_slots = VTK_ARR(ctx, out->new_tt_slots, c.max_tokens);
    a.freed_blocks = VTK_ARR(ctx, out->freed_blocks, c.max_table_blocks);
    a.out_status = VTK_ARR(ctx, out->req_status, c.max_requests);
    a.out_counts = VTK_ARR(ctx, out->counts, 1);
    a.req_n = VTK_ARR(ctx, ctx->req_n, c.max_requests);
    a.req_dst_base = VTK_ARR(ctx, ctx->req_dst_base, c.max_requests);
    a.req_freed_base = VTK_ARR(ctx, ctx->req_freed_base, c.max_requests);
    a.req_status = VTK_ARR(ctx, ctx->req_status, c.max_requests);
    a.dst_src = VTK_ARR(ctx, ctx->dst_src, (int64_t)ctx->cap_dst_blocks * c.block_size);
    a.dst_blocks = VTK_ARR(ctx, ctx->dst_blocks, ctx->cap_dst_blocks);
    a.tile_n = VTK_ARR(ctx, ctx->tile_n, tiles_cap + 1);
    a.req_part = VTK_ARR(ctx, ctx->req_part, (int64_t)c.max_requests + 1);
    a.req_before = VTK_ARR(ctx, ctx->req_before, (int64_t)c.max_requests + 1);
    a.header = VTK_ARR(ctx, ctx->plan_header, 4);
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
    // four entries per thread go through 16-byte (slots) and 4-byte (keep) accesses when the caller's
    // arrays allow it; tiles start at multiples of 1024 entries, so the base addresses decide
    a.vec_in = ((uintptr_t)in->tt_slots % 16 == 0 && (uintptr_t)in->keep % 4 == 0) ? 1 : 0;
    a.vec_out = ((uintptr_t)out->new_tt_slots % 16 == 0) ? 1 : 0;
#ifdef VTOKEN_CHECKED
    a.vec_in = a.vec_out = 0;      // one checked access per entry instead of one per four
#endif

    const int R = ctx->cfg.max_requests;
    VTK_CUDA(ctx, vtk_launch_dependent(ctx, plan_tiles_kernel, dim3(tile_ctas(a.num_tiles) + R + 1), dim3(TILE_NT), 0, st, a));
    VTK_CUDA(ctx, vtk_launch_dependent(ctx, plan_scan_kernel, dim3(1), dim3(SCAN_NT), 0, st, a));
    VTK_CUDA(ctx, vtk_launch_dependent(ctx, plan_assign_kernel, dim3(a.num_tiles + R), dim3(TILE_NT), 0, st, a));
    VTK_CUDA(ctx, cudaGetLastError());
    return VTOKEN_OK;
}
