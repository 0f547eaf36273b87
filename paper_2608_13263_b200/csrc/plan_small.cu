// Relocation planner for small tables (Sec. 3.3.3 of the paper): the same plan as the three kernels
// of plan.cu in two, for tables whose whole grid is resident at once (a few hundred CTAs).  A short
// plan is a chain of dependent steps -- each kernel boundary costs about 2 us, each dependent global
// load most of a microsecond -- so here the scan kernel is gone:
//   count  : live tokens per tile of 1024 consecutive table entries, and for every request the live
//            tokens between the start of the tile that holds its first entry and that entry
//   assign : every CTA first rebuilds, in shared memory, what the scan kernel would have handed to it:
//            the running live count at every tile start (the tile counts, one coalesced read), from
//            it the live tokens of every request as a difference of two running counts, then the
//            scan over the requests -- destinations needed -> candidates -> admission against the
//            free list -> bases.  Then the tile CTAs rank every live token inside its request ->
//            destination slot, new token table, inverse move plan; extra CTAs, one per request,
//            write the new block tables and the reclaimed list, one more the totals.
// No CTA waits for another.  Everything a CTA reads from global memory is requested in three rounds
// (header; entries, tile counts and request inputs; free-list entries).  The redundant scan costs
// every CTA about 2 us of issue slots, which a grid of one wave hides and a grid of five does not:
// measured on B200, 8.2 us instead of 11.5 on a 4-request table, even at 160 and 330 tiles, 49 us
// instead of 27 at 2 196 tiles -- hence the size limit (vtk_configure_plan decides).  A grid of one wave
// that redoes the scan once per CTA, keeps its results in shared memory and walks over the tiles in steps
// of the grid size was measured too: 30.9 us on the same table (four to five dependent rounds of loads
// per CTA in a row at half the occupancy of the three-kernel assign pass), so large tables keep three kernels.
#include "common.cuh"

namespace {

constexpr int TILE_NT = VTK_TILE_NT;             // threads per CTA
constexpr int TILE_TOK = VTK_TILE_TOK;           // table entries per thread
constexpr int TILE = VTK_TILE;                   // entries per tile
constexpr int RQ_PER_THREAD = 2;                 // requests per thread and round of the request scan
constexpr int RQ_ROUND = TILE_NT * RQ_PER_THREAD;
constexpr int NO_CUT = 0x7fffffff;
constexpr int MIN_CTAS = 4;                      // resident CTAs per SM the assign kernel is compiled for (64 registers, no spills)

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
    vtk_arr<int32_t> dst_src, dst_blocks;
    vtk_arr<int32_t> req_n;     // [max_requests] live tokens per request as the plan saw them (read by the commit of a wave)
    vtk_arr<int32_t> tile_n;    // [num_tiles] live tokens per tile (sign bit: a slot outside the pool)
    vtk_arr<int32_t> req_part;  // [max_requests + 1] live tokens between the start of the tile that holds the
                                // request's first entry and that entry
    vtk_arr<int32_t> header;    // [4] R, T, num_free, first entry as the count kernel read them: one load instead
                                // of a chain of three
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

// ---- count -----------------------------------------------------------------------------
__global__ void __launch_bounds__(TILE_NT) plan_small_count_kernel(PlanArgs a)
{
    __shared__ int warp_n[TILE_NT / 32];
    vtk_release_successor();
    vtk_wait_for_predecessor();
    const int R = clamp_requests(a);
    const int64_t T = clipped_offset(a, R);
    const int lane = vtk_lane(), warp = threadIdx.x >> 5;
    if (blockIdx.x == 0 && threadIdx.x == 0) {
        // flags of this plan are OR-ed in by the assign kernel: whatever an earlier plan or copy left goes here
        a.counts->error_flags = 0;
        a.out_counts->error_flags = 0;
        a.header[0] = R;
        a.header[1] = (int32_t)T;
        a.header[2] = *a.num_free;
        a.header[3] = (int32_t)clipped_offset(a, 0);
    }
    // A CTA counts the live entries of [base, limit): a whole tile, or -- the CTAs behind the tiles, one
    // per request boundary -- the entries between the start of the boundary's tile and the boundary
    // (entries the tile's own CTA counts as well).  Either way one pass.
    const bool is_tile = (int)blockIdx.x < a.num_tiles;
    const int rb = (int)blockIdx.x - a.num_tiles;
    int64_t base, limit;
    if (is_tile) {
        base = (int64_t)blockIdx.x * TILE;
        limit = T;
        if (base >= T) return;
    } else {
        if (rb > R) return;
        limit = clipped_offset(a, rb);
        base = limit / TILE * TILE;
        if (base == limit) return;                       // nothing in front of it: req_part[rb] is not read
    }
    bool bad = false;
    int32_t slot[TILE_TOK];
    int n = __popc(vtk_load_entries(a.tt_slots, a.keep, a.vec_in, base + threadIdx.x * TILE_TOK, clipped_offset(a, 0),
                                    limit, a.slots_per_layer, slot, bad));
#pragma unroll
    for (int d = 16; d > 0; d >>= 1) n += __shfl_down_sync(0xffffffffu, n, d);
    if (lane == 0) warp_n[warp] = n;
    const int any_bad = __syncthreads_or(bad);
    if (threadIdx.x == 0) {
        int s = 0;
#pragma unroll
        for (int w = 0; w < TILE_NT / 32; ++w) s += warp_n[w];
        // a slot outside the pool somewhere in the tile travels in the sign bit (the count is at most
        // 1024): the assign kernel turns it into VTOKEN_FLAG_BAD_SLOT
        if (is_tile) a.tile_n[blockIdx.x] = s | (any_bad ? (int)0x80000000 : 0);
        else a.req_part[rb] = s;
    }
}

// ---- the scan over the requests, redone by every CTA of the assign kernel ----------------
struct Sums {                   // running sums over the requests: over candidates (c_*) and over all
    int c_need, c_nb, c_n, c_cnt, nb_all;
};
__device__ __forceinline__ Sums operator+(const Sums &x, const Sums &y)
{
    return Sums{x.c_need + y.c_need, x.c_nb + y.c_nb, x.c_n + y.c_n, x.c_cnt + y.c_cnt, x.nb_all + y.nb_all};
}
__device__ __forceinline__ Sums operator-(const Sums &x, const Sums &y)
{
    return Sums{x.c_need - y.c_need, x.c_nb - y.c_nb, x.c_n - y.c_n, x.c_cnt - y.c_cnt, x.nb_all - y.nb_all};
}
__device__ __forceinline__ Sums shfl_up(const Sums &v, int d)
{
    return Sums{__shfl_up_sync(0xffffffffu, v.c_need, d), __shfl_up_sync(0xffffffffu, v.c_nb, d),
                __shfl_up_sync(0xffffffffu, v.c_n, d), __shfl_up_sync(0xffffffffu, v.c_cnt, d),
                __shfl_up_sync(0xffffffffu, v.nb_all, d)};
}

// What the scan knows about one request once the requests before it have been summed.
struct Request {
    int n, nb, need, status;
    int before;         // live entries of the table in front of its first entry
    int dst_base;       // first entry of its destinations in the free list (admitted requests)
    int freed_base;     // first entry of its old blocks in the reclaimed list (admitted requests)
    int newbt;          // first entry of its new block table
};

// Shared state of the scan.  The admitted requests are a prefix of the candidates (the cumulative
// demand only grows), so a sum over the admitted requests in front of a request equals the sum over
// the candidates in front of it -- until the first candidate that does not fit, where it freezes (`cut`).
struct ScanState {
    Sums carry;         // sums over the requests of the rounds before this one
    Sums cut;           // sums over the requests in front of the first deferred candidate
    int cut_r;          // request index of the first deferred candidate, NO_CUT while there is none
    Sums warp_tot[TILE_NT / 32];
    unsigned flags;
};

// Everything a thread reads from global memory for its requests of one round of the scan, loaded
// in one go so that the loads overlap (a dependent global load costs most of a microsecond).
struct RoundInputs {
    int tt[RQ_PER_THREAD + 1], bt[RQ_PER_THREAD + 1], part[RQ_PER_THREAD + 1];
    unsigned char sel[RQ_PER_THREAD];
};
__device__ __forceinline__ void load_round(const PlanArgs &a, int R, int r0, RoundInputs &in)
{
    const int r_mine = r0 + (int)threadIdx.x * RQ_PER_THREAD;
#pragma unroll
    for (int k = 0; k <= RQ_PER_THREAD; ++k) {
        const bool ok = r_mine + k <= R && r_mine < R;
        in.tt[k] = ok ? a.tt_offsets[r_mine + k] : 0;
        in.bt[k] = ok ? a.bt_offsets[r_mine + k] : 0;
        in.part[k] = ok ? a.req_part[r_mine + k] : 0;        // (scratch of the count kernel: only read when the offset is inside a tile)
    }
#pragma unroll
    for (int k = 0; k < RQ_PER_THREAD; ++k)
        in.sel[k] = (!a.select.null() && r_mine + k < R) ? a.select[r_mine + k] : (unsigned char)1;
}

__device__ __forceinline__ int64_t clip_to(int64_t o, int64_t cap) { return o < 0 ? 0 : (o > cap ? cap : o); }

// Running live count in front of table entry o, the first entry of a request (or one past the last
// entry of the request before it): the count at the start of o's tile plus what the count kernel
// found between that start and o (`part`).  `before` holds the counts at the tile starts.
__device__ __forceinline__ int live_before(const int *before, int tiles, int64_t o, int part)
{
    const int64_t j = o / TILE;                  // beyond the table only with offsets that are out of order
    return before[j < tiles ? j : tiles] + (o % TILE != 0 ? part : 0);
}

// One round of the scan: requests [r0, r0 + RQ_ROUND), RQ_PER_THREAD consecutive ones per thread.
// Returns this thread's requests in req[] (valid[] false beyond R) and the table range of each.
// All threads of the CTA call it.
__device__ __forceinline__ void scan_round(const PlanArgs &a, ScanState &st, const int *before_tile, int tiles, int R,
                                           int nf, int r0, const RoundInputs &in,
                                           Request (&req)[RQ_PER_THREAD], bool (&valid)[RQ_PER_THREAD],
                                           int64_t (&o0)[RQ_PER_THREAD], int64_t (&o1)[RQ_PER_THREAD])
{
    const int lane = vtk_lane(), warp = threadIdx.x >> 5;
    const int r_mine = r0 + (int)threadIdx.x * RQ_PER_THREAD;
    Sums mine[RQ_PER_THREAD];
    bool cand[RQ_PER_THREAD];
    uint32_t flags = 0;
    Sums run{0, 0, 0, 0, 0};
#pragma unroll
    for (int k = 0; k < RQ_PER_THREAD; ++k) {
        const int r = r_mine + k;
        valid[k] = r < R;
        int n = 0, nb = 0, lb = 0;
        bool sel = false;
        o0[k] = o1[k] = 0;
        if (valid[k]) {
            // table ranges clipped to the create-time capacities (a range that runs backwards is empty)
            const int64_t lo = clip_to(in.bt[k], a.max_table_blocks), b1 = clip_to(in.bt[k + 1], a.max_table_blocks);
            const int64_t hi = b1 < lo ? lo : b1;
            const int64_t t0 = clip_to(in.tt[k], a.max_tokens), t1 = clip_to(in.tt[k + 1], a.max_tokens);
            o0[k] = t0;
            o1[k] = t1 < t0 ? t0 : t1;
            if (lo != in.bt[k] || hi != in.bt[k + 1] || t0 != in.tt[k] || o1[k] != in.tt[k + 1]) flags |= VTOKEN_FLAG_CAPACITY;
            nb = (int)(hi - lo);
            // live tokens = difference of the running counts at its two ends
            lb = live_before(before_tile, tiles, t0, in.part[k]);
            n = live_before(before_tile, tiles, t1, in.part[k + 1]) - lb;
            if (n < 0) n = 0;                                // offsets that run backwards
            sel = in.sel[k] != 0;
            if (sel && a.thr_den != 0)
                sel = (unsigned long long)n * a.thr_den <
                      (unsigned long long)a.thr_num * (unsigned long long)nb * (unsigned long long)a.S;
        }
        const int need = (int)(((int64_t)n + a.S - 1) / a.S);       // ceil(T_live / S)
        cand[k] = sel && need < nb;                                  // strictly fewer blocks afterwards
        req[k].n = n;
        req[k].nb = nb;
        req[k].need = need;
        req[k].before = lb;
        req[k].status = !sel ? VTOKEN_NOT_SELECTED : (!cand[k] ? VTOKEN_NO_GAIN : VTOKEN_REPACKED);   // admission below
        mine[k] = Sums{cand[k] ? need : 0, cand[k] ? nb : 0, cand[k] ? n : 0, cand[k] ? 1 : 0, valid[k] ? nb : 0};
        run = run + mine[k];
    }
    // sums over the requests in front of this thread's
    Sums incl = run;
#pragma unroll
    for (int d = 1; d < 32; d <<= 1) {
        const Sums o = shfl_up(incl, d);
        if (lane >= d) incl = o + incl;
    }
    if (lane == 31) st.warp_tot[warp] = incl;
    __syncthreads();
    Sums before = st.carry + (incl - run);
    for (int w = 0; w < warp; ++w) before = before + st.warp_tot[w];
    // admission: the cumulative demand of the candidates so far (this one included) fits the free list
    const int cut_before = st.cut_r;
    Sums ex[RQ_PER_THREAD];
    int my_cut = NO_CUT;
#pragma unroll
    for (int k = 0; k < RQ_PER_THREAD; ++k) {
        ex[k] = before;
        before = before + mine[k];
        if (cand[k] && before.c_need > nf) {
            req[k].status = VTOKEN_DEFERRED_NO_FREE;
            if (my_cut == NO_CUT) my_cut = r_mine + k;
        }
    }
    if (cut_before == NO_CUT) {
        // the first deferred request of this round, if any
        int first = my_cut;
#pragma unroll
        for (int d = 16; d > 0; d >>= 1) first = min(first, __shfl_xor_sync(0xffffffffu, first, d));
        if (lane == 0 && first != NO_CUT) atomicMin(&st.cut_r, first);
    }
    if (flags) atomicOr(&st.flags, flags);
    __syncthreads();
    const int cut_r = st.cut_r;
    if (cut_before == NO_CUT && my_cut == cut_r && cut_r != NO_CUT) {       // its thread freezes the sums
#pragma unroll
        for (int k = 0; k < RQ_PER_THREAD; ++k)
            if (r_mine + k == cut_r) st.cut = ex[k];
    }
    if (threadIdx.x == TILE_NT - 1) st.carry = before;       // the last thread holds the totals so far
    __syncthreads();
    const Sums cut = st.cut;
#pragma unroll
    for (int k = 0; k < RQ_PER_THREAD; ++k) {
        const bool after_cut = r_mine + k > cut_r;            // a candidate was deferred in front of this request
        const Sums &adm = after_cut ? cut : ex[k];            // sums over the admitted requests in front of it
        req[k].dst_base = adm.c_need;
        req[k].freed_base = adm.c_nb;
        req[k].newbt = ex[k].nb_all - (adm.c_nb - adm.c_need);
    }
}

// ---- assign ----------------------------------------------------------------------------
// What a tile CTA keeps of a request that owns entries of its tile, at index max(0, first entry of
// the request - first entry of the tile): every such request but the first starts inside the tile,
// at an entry of its own.
struct TileRequest {
    int dst_base;       // -1: the request keeps its layout
    int n;
    int before;         // live entries of the table in front of the request's first entry
};

__global__ void __launch_bounds__(TILE_NT, MIN_CTAS) plan_small_assign_kernel(PlanArgs a)
{
    extern __shared__ int staged[];          // [tiles + 1] tile counts, then live entries in front of every tile
    __shared__ ScanState st;
    __shared__ TileRequest tile_rq[TILE];
    __shared__ unsigned start_bits[TILE / 32];   // one bit per entry of the tile at which a request starts
    __shared__ int warp_sums[TILE_NT / 32];
    __shared__ Request own;                  // request CTAs: their request
    vtk_release_successor();
    vtk_wait_for_predecessor();
    const int tid = threadIdx.x, lane = vtk_lane(), warp = tid >> 5;
    const int S = a.S;
    const int4 hdr = *reinterpret_cast<const int4 *>(a.header.at(0, 4));
    const int R = hdr.x;
    const int64_t T = hdr.y, first_entry = hdr.w;
    int nf = hdr.z;
    const bool nf_over = nf > a.max_free_blocks;
    nf = nf < 0 ? 0 : (nf > a.cap_dst_blocks ? a.cap_dst_blocks : nf);
    const int tiles = (int)((T + TILE - 1) / TILE);

    // role of this CTA
    const int q = (int)blockIdx.x - a.num_tiles;              // request CTAs: 0 .. R - 1; totals CTA: R
    const int64_t base = (int64_t)blockIdx.x * TILE;
    const bool is_tile = q < 0;
    if (is_tile ? base >= T : q > R) return;
    uint32_t flags = 0;
    // Everything this CTA needs from global memory before it can do anything, requested back to back:
    // its entries of the token table, the inputs of the first round of the request scan, the tile counts
    const int64_t t = base + tid * TILE_TOK;
    int32_t slot[TILE_TOK] = {-1, -1, -1, -1};
    uint8_t kp[TILE_TOK] = {0, 0, 0, 0};
    if (is_tile) {
        if (a.vec_in && t + TILE_TOK <= T) {
            const int4 s4 = *reinterpret_cast<const int4 *>(a.tt_slots.at(t, TILE_TOK));
            const uchar4 k4 = *reinterpret_cast<const uchar4 *>(a.keep.at(t, TILE_TOK));
            slot[0] = s4.x; slot[1] = s4.y; slot[2] = s4.z; slot[3] = s4.w;
            kp[0] = k4.x; kp[1] = k4.y; kp[2] = k4.z; kp[3] = k4.w;
        } else {
#pragma unroll
            for (int k = 0; k < TILE_TOK; ++k)
                if (t + k < T) { slot[k] = a.tt_slots[t + k]; kp[k] = a.keep[t + k]; }
        }
    }
    RoundInputs rin;
    load_round(a, R, 0, rin);
#pragma unroll 4
    for (int j = tid; j < tiles; j += TILE_NT) staged[j] = a.tile_n[j];
    unsigned bits = 0;
    if (is_tile) {
        // live: owns a slot inside the pool, kept by the policy, not in front of the first request
#pragma unroll
        for (int k = 0; k < TILE_TOK; ++k)
            if (slot[k] >= 0 && (int64_t)slot[k] < a.slots_per_layer && kp[k] != 0 && t + k >= first_entry) bits |= 1u << k;
#pragma unroll
        for (int k = 0; k < TILE_TOK; ++k) tile_rq[tid + k * TILE_NT] = TileRequest{-1, 0, 0};
        if (tid < TILE / 32) start_bits[tid] = 0u;
    }
    if (tid == 0) {
        st.carry = Sums{0, 0, 0, 0, 0};
        st.cut = Sums{0, 0, 0, 0, 0};
        st.cut_r = NO_CUT;
        st.flags = 0;
    }

    // running live count at every tile start, from the tile counts in shared memory (above): every thread
    // sums a run of consecutive tiles, the runs are scanned over the CTA, every thread writes the running
    // counts of its run
    __syncthreads();
    {
        const int per = (tiles + TILE_NT - 1) / TILE_NT;
        const int j0 = tid * per, j1 = min(tiles, j0 + per);
        int sum = 0, any_bad = 0;
        for (int j = j0; j < j1; ++j) { const int v = staged[j]; sum += v & 0x7fffffff; any_bad |= v; }
        if (any_bad < 0) atomicOr(&st.flags, VTOKEN_FLAG_BAD_SLOT);     // a slot outside the pool in one of the tiles
        const int incl = vtk_warp_incl_scan(sum);
        if (lane == 31) warp_sums[warp] = incl;
        __syncthreads();
        int run = incl - sum;
        for (int w = 0; w < warp; ++w) run += warp_sums[w];
        for (int j = j0; j < j1; ++j) { const int v = staged[j] & 0x7fffffff; staged[j] = run; run += v; }
        if (j1 == tiles && j0 <= tiles) staged[tiles] = run;      // (several threads may write it: the same total)
    }
    const int *before_tile = staged;
    __syncthreads();

    // tile CTAs: running count in front of each thread's entries
    int before = 0;
    if (is_tile) {
        const int cnt = __popc(bits);
        const int incl = vtk_warp_incl_scan(cnt);
        if (lane == 31) warp_sums[warp] = incl;
        __syncthreads();
        before = before_tile[blockIdx.x] + incl - cnt;
        for (int w = 0; w < warp; ++w) before += warp_sums[w];
    }

    // the scan over the requests, as far as this CTA needs it: a tile CTA up to the last request that
    // starts in front of the end of its tile, a request CTA up to its request, the totals CTA to the end
    const int64_t tile_end = base + TILE < T ? base + TILE : T;
    for (int r0 = 0; r0 < R; r0 += RQ_ROUND) {
        if (r0 > 0) {
            if (is_tile ? clipped_offset(a, r0) >= tile_end : r0 > (q < R ? q : R - 1)) break;
            load_round(a, R, r0, rin);
        }
        Request req[RQ_PER_THREAD];
        bool valid[RQ_PER_THREAD];
        int64_t o0[RQ_PER_THREAD], o1[RQ_PER_THREAD];
        scan_round(a, st, before_tile, tiles, R, nf, r0, rin, req, valid, o0, o1);
#pragma unroll
        for (int k = 0; k < RQ_PER_THREAD; ++k) {
            if (!valid[k]) continue;
            if (is_tile) {
                // requests that own entries of this tile
                if (o1[k] > o0[k] && o1[k] > base && o0[k] < tile_end) {
                    const int idx = o0[k] > base ? (int)(o0[k] - base) : 0;
                    tile_rq[idx] = TileRequest{req[k].status == VTOKEN_REPACKED ? req[k].dst_base : -1, req[k].n,
                                               req[k].before};
                    atomicOr(&start_bits[idx >> 5], 1u << (idx & 31));
                }
            } else if (r0 + tid * RQ_PER_THREAD + k == q) {
                own = req[k];
            }
        }
    }
    __syncthreads();

    if (!is_tile && q == R) {
        // totals: counts, the end of the new block tables, flags found on the way
        if (tid == 0) {
            const Sums tot = st.carry;
            const Sums adm = st.cut_r != NO_CUT ? st.cut : tot;
            flags |= st.flags;
            if (*a.num_requests > a.max_requests || *a.num_requests < 0 || nf_over) flags |= VTOKEN_FLAG_CAPACITY;
            a.new_bt_offsets[R] = tot.nb_all - (adm.c_nb - adm.c_need);
            // field by field: the flags of this plan are OR-ed in by whichever CTA finds them
            a.counts->num_moves = a.out_counts->num_moves = adm.c_n;
            a.counts->num_dst_blocks = a.out_counts->num_dst_blocks = adm.c_need;
            a.counts->num_freed = a.out_counts->num_freed = adm.c_nb;
            a.counts->num_free_consumed = a.out_counts->num_free_consumed = adm.c_need;
            a.counts->num_admitted = a.out_counts->num_admitted = adm.c_cnt;
            a.counts->num_deferred = a.out_counts->num_deferred = tot.c_cnt - adm.c_cnt;
            a.counts->num_released = a.out_counts->num_released = 0;
        }
    } else if (!is_tile) {
        // block table and reclaimed list of request q
        const Request me = own;
        const int n = me.n, nb = me.nb, need = me.need, dst_base = me.dst_base, f0 = me.freed_base, nbt0 = me.newbt;
        int64_t b0, b1;
        vtk_range(a.bt_offsets, q, a.max_table_blocks, b0, b1);
        if (tid == 0) {
            a.out_status[q] = me.status;
            a.new_bt_offsets[q] = nbt0;
            a.req_n[q] = n;
        }
        if (me.status == VTOKEN_REPACKED) {
            for (int j = tid; j < need; j += TILE_NT) {
                int blk = a.free_blocks[dst_base + j];
                if ((int64_t)nbt0 + j < a.max_table_blocks) a.new_bt_blocks[nbt0 + j] = blk;
                if (blk < 0 || blk >= a.num_blocks) { flags |= VTOKEN_FLAG_BAD_FREE; blk = -1; }
                a.dst_blocks[dst_base + j] = blk;
            }
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
    } else if (t < T) {
        // token table: rank of each live token in logical order -> destination slot
        // the request of an entry: the nearest request start at or in front of it inside the tile (the
        // first owner of the tile sits at index 0 wherever it started)
        auto owner_index = [&](int p) {
            int w = p >> 5;
            unsigned m = start_bits[w] & (0xffffffffu >> (31 - (p & 31)));
            while (m == 0u && w > 0) m = start_bits[--w];
            return m != 0u ? (w << 5) + 31 - __clz((int)m) : -1;
        };
        const int p0 = tid * TILE_TOK;
        int idx = owner_index(p0);
        TileRequest rq = idx >= 0 ? tile_rq[idx] : TileRequest{-1, 0, 0};
        int32_t out[TILE_TOK];
        int64_t dst[TILE_TOK];                                    // entry of the inverse plan, -1: none
        int off_in_block[TILE_TOK];
        bool owned = true;
#pragma unroll
        for (int k = 0; k < TILE_TOK; ++k) {
            out[k] = -1;
            dst[k] = -1;
            off_in_block[k] = 0;
            if (t + k >= T) { owned = false; continue; }
            if (k > 0 && (start_bits[(p0 + k) >> 5] >> ((p0 + k) & 31)) & 1u) {     // a request starts at this entry
                idx = p0 + k;
                rq = tile_rq[idx];
            }
            if (idx < 0) { owned = false; continue; }             // in front of the first request: left untouched
            if (!((bits >> k) & 1u)) continue;                    // dead or unmapped: -1
            if (rq.dst_base < 0) { out[k] = slot[k]; continue; } // the request keeps its layout
            const int i = before + __popc(bits & ((1u << k) - 1u)) - rq.before;    // rank inside the request
            if (i < 0 || i >= rq.n) continue;                     // only with inconsistent offsets
            const int j = i / S;
            off_in_block[k] = i - j * S;
            dst[k] = rq.dst_base + j;
        }
        // the destination blocks (up to four loads in flight), then the stores
        int blk[TILE_TOK];
#pragma unroll
        for (int k = 0; k < TILE_TOK; ++k) blk[k] = dst[k] >= 0 ? __ldg(a.free_blocks.at(dst[k])) : 0;
#pragma unroll
        for (int k = 0; k < TILE_TOK; ++k) {
            if (dst[k] < 0) continue;
            out[k] = blk[k] * S + off_in_block[k];                // slot = block_id * S + offset
            a.dst_src[dst[k] * S + off_in_block[k]] = slot[k];
        }
        if (owned && a.vec_out) {
            *reinterpret_cast<int4 *>(a.new_tt_slots.at(t, TILE_TOK)) = make_int4(out[0], out[1], out[2], out[3]);
        } else {
            // the ragged end of the table, or entries in front of the first request (left untouched)
#pragma unroll
            for (int k = 0; k < TILE_TOK; ++k)
                if (t + k < T && t + k >= first_entry) a.new_tt_slots[t + k] = out[k];
        }
    }
    if (flags) raise_flags(a, flags);
}

}  // namespace

// Which form of the whole-request planner this context uses (ctx->plan_form: 1 three kernels, 2 two kernels).
// Two kernels instead of three -- one kernel boundary less, at the price of a scan over the requests that
// every CTA redoes -- pay while the whole grid (tiles + requests + 1 CTAs) is resident at once, so that the
// scan is paid once per resident CTA; everything else takes the three kernels.  vtoken_config.plan_variant
// forces a form where it fits.  The checked build defaults to the three kernels.
int vtk_configure_plan(vtoken_ctx *ctx)
{
    const int64_t roles = (ctx->cfg.max_tokens + TILE - 1) / TILE + ctx->cfg.max_requests + 1;
    const bool resident_ok = roles <= (int64_t)ctx->num_sms * MIN_CTAS;
    int form = ctx->cfg.plan_variant;
#ifdef VTOKEN_CHECKED
    if (form == 0) form = 1;
#endif
    if (form == 0) form = resident_ok ? 2 : 1;
    if (form == 2 && !resident_ok) form = 1;
    ctx->plan_form = form;
    return VTOKEN_OK;
}

// The caller (vtk_launch_plan) has checked that the grid is small enough for this planner.
int vtk_launch_plan_small(vtoken_ctx *ctx, const vtoken_plan_in *in, const vtoken_plan_out *out, cudaStream_t st)
{
    PlanArgs a{};
    const vtoken_config &c = ctx->cfg;
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
    a.dst_src = VTK_ARR(ctx, ctx->dst_src, (int64_t)ctx->cap_dst_blocks * c.block_size);
    a.dst_blocks = VTK_ARR(ctx, ctx->dst_blocks, ctx->cap_dst_blocks);
    a.req_n = VTK_ARR(ctx, ctx->req_n, c.max_requests);
    a.tile_n = VTK_ARR(ctx, ctx->tile_n, (c.max_tokens + TILE - 1) / TILE + 1);
    a.req_part = VTK_ARR(ctx, ctx->req_part, (int64_t)c.max_requests + 1);
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

    const int R = ctx->cfg.max_requests;
    const dim3 grid(a.num_tiles + R + 1);
    VTK_CUDA(ctx, vtk_launch_dependent(ctx, plan_small_count_kernel, grid, dim3(TILE_NT), 0, st, a));
    const size_t smem = sizeof(int) * (size_t)(a.num_tiles + 1);
    VTK_CUDA(ctx, vtk_launch_dependent(ctx, plan_small_assign_kernel, grid, dim3(TILE_NT), smem, st, a));
    VTK_CUDA(ctx, cudaGetLastError());
    return VTOKEN_OK;
}
