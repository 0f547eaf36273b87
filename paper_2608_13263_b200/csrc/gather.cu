// Logical view of the cache (invariant I1; the before/after relocation check of Sec. 5):
// K and V rows of the active tokens of the selected requests, request order then token-id
// order, written densely.  Same structure as the planner: count -> scan -> assign, then a
// row-copy kernel that reads through the token table (the slot-translation read pattern of
// Sec. 3.4).  Two versions of the index kernels: a flat tiling of the token table like the planner's
// (contexts made by vtoken_create), and one that walks the table request by request, every request cut
// into 1 .. VTK_PLAN_PARTS equal token ranges with one CTA each (the context-free entry point, which
// has no capacity for the table's length).
#include "common.cuh"

namespace {

constexpr int G_NT = 512;
constexpr int G_PARTS = VTK_PLAN_PARTS;

struct GatherArgs {
    vtk_arr<const int32_t> num_requests, tt_offsets, tt_slots;
    vtk_arr<const uint8_t> keep, select;
    vtk_arr<int32_t> req_n, part_n, out_offsets, g_src, g_total;
    vtk_arr<int32_t> g_ids, g_req;      // logical id / request of each output row, or NULL
    vtk_arr<unsigned long long> digest;  // per-request digest (digest kernel only)
    vtk_arr<vtoken_counts> counts;
    const uint8_t *k_pool, *v_pool;
    uint8_t *out_k, *out_v;
    int64_t layer_stride, row_bytes, slots_per_layer, out_capacity, max_tokens;
    int32_t layer_begin, layer_end, max_requests;
    int32_t parts;               // token ranges (CTAs) per request, <= G_PARTS (the stride of part_n)
    // flat tiling (contexts made by vtoken_create; see plan.cu): live tokens per tile, then before every tile;
    // live tokens between the start of a request boundary's tile and the boundary; live tokens before a request
    vtk_arr<int32_t> tile_n, req_part, req_before;
    int32_t num_tiles, vec_in;
    int64_t table_cap;           // capacity of the token table: offsets are clipped to it
};

__device__ __forceinline__ int g_requests(const GatherArgs &a)
{
    int R = *a.num_requests;
    return R < 0 ? 0 : (R > a.max_requests ? a.max_requests : R);
}

// token range [p0, p1) of part c of a request spanning [t0, t1): equal parts, multiples of 128
__device__ __forceinline__ void g_part_range(int64_t t0, int64_t t1, int c, int parts, int64_t &p0, int64_t &p1)
{
    int64_t per = (t1 - t0 + parts - 1) / parts;
    per = (per + 127) & ~(int64_t)127;
    p0 = t0 + (int64_t)c * per;
    p1 = p0 + per;
    if (p0 > t1) p0 = t1;
    if (p1 > t1) p1 = t1;
}

__global__ void __launch_bounds__(G_NT) gather_count_kernel(GatherArgs a)
{
    vtk_release_successor();
    vtk_wait_for_predecessor();
    const int r = blockIdx.x / a.parts, c = blockIdx.x % a.parts;
    if (r >= g_requests(a)) return;
    int n = 0;
    bool bad = false;
    if (a.select.null() || a.select[r] != 0) {
        int64_t p0, p1;
        g_part_range(a.tt_offsets[r], a.tt_offsets[r + 1], c, a.parts, p0, p1);
        for (int64_t t = p0 + threadIdx.x; t < p1; t += G_NT)
            n += vtk_live(a.tt_slots[t], a.keep, t, a.slots_per_layer, bad) ? 1 : 0;
    }
    __shared__ int warp_n[G_NT / 32];
#pragma unroll
    for (int d = 16; d > 0; d >>= 1) n += __shfl_down_sync(0xffffffffu, n, d);
    if (vtk_lane() == 0) warp_n[threadIdx.x >> 5] = n;
    if (bad) atomicOr(&a.counts->error_flags, VTOKEN_FLAG_BAD_SLOT);
    __syncthreads();
    if (threadIdx.x == 0) {
        int s = 0;
        for (int w = 0; w < G_NT / 32; ++w) s += warp_n[w];
        a.part_n[r * G_PARTS + c] = s;
    }
}

// exclusive scan of the per-request counts -> out_offsets[R+1]; one CTA
__global__ void __launch_bounds__(1024) gather_scan_kernel(GatherArgs a)
{
    vtk_release_successor();
    vtk_wait_for_predecessor();
    __shared__ int warp_tot[33];
    __shared__ int carry;
    const int R = g_requests(a);
    const int tid = threadIdx.x, lane = vtk_lane(), warp = tid >> 5;
    if (tid == 0) carry = 0;
    __syncthreads();
    for (int base = 0; base < R; base += 1024) {
        const int r = base + tid;
        int v = 0;
        if (r < R) {
#pragma unroll
            for (int c = 0; c < a.parts; ++c) v += a.part_n[r * G_PARTS + c];
        }
        int incl = vtk_warp_incl_scan(v);
        if (lane == 31) warp_tot[warp] = incl;
        __syncthreads();
        if (warp == 0) {
            const int w = warp_tot[lane];
            const int wi = vtk_warp_incl_scan(w);
            warp_tot[lane] = wi - w;
            if (lane == 31) warp_tot[32] = wi;
        }
        __syncthreads();
        const int excl = carry + warp_tot[warp] + incl - v;
        if (r < R) a.out_offsets[r] = excl;
        __syncthreads();
        if (tid == 0) carry += warp_tot[32];
        __syncthreads();
    }
    if (tid == 0) {
        a.out_offsets[R] = carry;
        int64_t cap = a.out_capacity < a.max_tokens ? a.out_capacity : a.max_tokens;
        if ((int64_t)carry > cap) {
            atomicOr(&a.counts->error_flags, VTOKEN_FLAG_GATHER_OVERFLOW);
            *a.g_total = (int32_t)cap;
        } else {
            *a.g_total = carry;
        }
    }
}

__global__ void __launch_bounds__(G_NT) gather_assign_kernel(GatherArgs a)
{
    vtk_release_successor();
    vtk_wait_for_predecessor();
    __shared__ int warp_sums[G_NT / 32 + 1];
    const int r = blockIdx.x / a.parts, c = blockIdx.x % a.parts;
    if (r >= g_requests(a)) return;
    if (!a.select.null() && a.select[r] == 0) return;
    const int64_t t0 = a.tt_offsets[r];
    int64_t p0, p1;
    g_part_range(t0, a.tt_offsets[r + 1], c, a.parts, p0, p1);
    const int64_t cap = *a.g_total;
    int carry = a.out_offsets[r];
    for (int cc = 0; cc < c; ++cc) carry += a.part_n[r * G_PARTS + cc];
    for (int64_t tb = p0; tb < p1; tb += G_NT) {
        const int64_t t = tb + threadIdx.x;
        int32_t slot = -1;
        bool live = false, bad = false;
        if (t < p1) {
            slot = a.tt_slots[t];
            live = vtk_live(slot, a.keep, t, a.slots_per_layer, bad);
        }
        int total;
        const int i = carry + vtk_block_rank<G_NT>(live, warp_sums, total);
        carry += total;
        if (live && i < cap) {
            a.g_src[i] = slot;
            if (!a.g_ids.null()) a.g_ids[i] = (int32_t)(t - t0);
            if (!a.g_req.null()) a.g_req[i] = r;
        }
    }
}

// ---- the same index over a flat tiling of the token table ------------------------------------------
// Tiles of 1024 consecutive table entries whatever request they belong to; per-request numbers are
// differences of running live counts (see plan.cu).  Used when the context has the tile scratch, which
// needs a capacity for the table's length; the context-free entry point keeps the kernels above.
__device__ __forceinline__ int64_t g_offset(const GatherArgs &a, int r)
{
    return vtk_clipped_offset(a.tt_offsets, r, a.table_cap);
}

__global__ void __launch_bounds__(VTK_TILE_NT) gather_tiles_kernel(GatherArgs a)
{
    __shared__ int warp_n[VTK_TILE_NT / 32];
    vtk_release_successor();
    vtk_wait_for_predecessor();
    const int R = g_requests(a);
    const int64_t T = g_offset(a, R);
    // a whole tile, or (CTAs behind the tiles, one per request boundary) the entries between the start of
    // the boundary's tile and the boundary
    const bool is_tile = (int)blockIdx.x < a.num_tiles;
    const int rb = (int)blockIdx.x - a.num_tiles;
    int64_t base, limit;
    if (is_tile) {
        base = (int64_t)blockIdx.x * VTK_TILE;
        limit = T;
        if (base >= T) return;
    } else {
        if (rb > R) return;
        limit = g_offset(a, rb);
        base = limit / VTK_TILE * VTK_TILE;
        if (base == limit) return;
    }
    bool bad = false;
    int32_t slot[VTK_TILE_TOK];
    int n = __popc(vtk_load_entries(a.tt_slots, a.keep, a.vec_in, base + threadIdx.x * VTK_TILE_TOK, g_offset(a, 0),
                                    limit, a.slots_per_layer, slot, bad));
#pragma unroll
    for (int d = 16; d > 0; d >>= 1) n += __shfl_down_sync(0xffffffffu, n, d);
    if (vtk_lane() == 0) warp_n[threadIdx.x >> 5] = n;
    __syncthreads();
    if (threadIdx.x == 0) {
        int s = 0;
#pragma unroll
        for (int w = 0; w < VTK_TILE_NT / 32; ++w) s += warp_n[w];
        (is_tile ? a.tile_n[blockIdx.x] : a.req_part[rb]) = s;
    }
}

__global__ void __launch_bounds__(1024) gather_scan_flat_kernel(GatherArgs a)
{
    vtk_release_successor();
    vtk_wait_for_predecessor();
    __shared__ int warp_tot[32];
    __shared__ int carry;
    const int R = g_requests(a);
    const int tid = threadIdx.x;
    if (tid == 0) carry = 0;
    __syncthreads();
    auto shfl_int = [](int v, int d) { return __shfl_up_sync(0xffffffffu, v, d); };
    // live tokens before every tile, in place; one entry past the last tile holds the total
    const int64_t T = g_offset(a, R);
    const int tiles = (int)((T + VTK_TILE - 1) / VTK_TILE);
    for (int base = 0; base <= tiles; base += 1024) {
        const int i = base + tid;
        const int v = i < tiles ? a.tile_n[i] : 0;
        const int incl = vtk_block_incl_scan<int>(v, warp_tot, 0, shfl_int) + carry;
        if (i <= tiles) a.tile_n[i] = incl - v;
        __syncthreads();
        if (tid == 1023) carry = incl;
        __syncthreads();
    }
    auto live_before = [&](int r) {
        const int64_t o = g_offset(a, r);
        return a.tile_n[o / VTK_TILE] + (o % VTK_TILE != 0 ? a.req_part[r] : 0);
    };
    // live tokens of the selected requests -> first output row of every request
    if (tid == 0) carry = 0;
    __syncthreads();
    for (int base = 0; base < R; base += 1024) {
        const int r = base + tid;
        int v = 0;
        if (r < R) {
            const int before = live_before(r);
            a.req_before[r] = before;
            if (a.select.null() || a.select[r] != 0) v = live_before(r + 1) - before;
            if (v < 0) v = 0;                                // offsets that run backwards
        }
        const int incl = vtk_block_incl_scan<int>(v, warp_tot, 0, shfl_int) + carry;
        if (r < R) a.out_offsets[r] = incl - v;
        __syncthreads();
        if (tid == 1023) carry = incl;
        __syncthreads();
    }
    if (tid == 0) {
        a.out_offsets[R] = carry;
        int64_t cap = a.out_capacity < a.max_tokens ? a.out_capacity : a.max_tokens;
        if ((int64_t)carry > cap) {
            atomicOr(&a.counts->error_flags, VTOKEN_FLAG_GATHER_OVERFLOW);
            *a.g_total = (int32_t)cap;
        } else {
            *a.g_total = carry;
        }
    }
}

__global__ void __launch_bounds__(VTK_TILE_NT) gather_assign_flat_kernel(GatherArgs a)
{
    __shared__ int warp_sums[VTK_TILE_NT / 32];
    __shared__ int tile_req[2];
    vtk_release_successor();
    vtk_wait_for_predecessor();
    const int R = g_requests(a);
    const int64_t T = g_offset(a, R);
    const int64_t base = (int64_t)blockIdx.x * VTK_TILE;
    if (base >= T) return;
    const int tid = threadIdx.x, lane = vtk_lane(), warp = tid >> 5;
    const int64_t t = base + tid * VTK_TILE_TOK;
    int32_t slot[VTK_TILE_TOK];
    bool bad_any = false;
    const unsigned bits = vtk_load_entries(a.tt_slots, a.keep, a.vec_in, t, g_offset(a, 0), T, a.slots_per_layer, slot,
                                           bad_any);
    const int cnt = __popc(bits);
    const int incl = vtk_warp_incl_scan(cnt);
    if (lane == 31) warp_sums[warp] = incl;
    vtk_tile_owners(a.tt_offsets, R, a.table_cap, base, T, tile_req);
    __syncthreads();
    int before = a.tile_n[blockIdx.x] + incl - cnt;          // live tokens of the table before entry t
    for (int w = 0; w < warp; ++w) before += warp_sums[w];
    if (t >= T) return;
    int r = vtk_entry_owner(a.tt_offsets, a.table_cap, tile_req, t);
    int64_t next = g_offset(a, r + 1), t0 = r >= 0 ? g_offset(a, r) : 0;
    int first_row = 0;
    bool sel = false;
    auto load_request = [&]() {
        sel = a.select.null() || a.select[r] != 0;
        first_row = a.out_offsets[r] - a.req_before[r];      // output row of a token = this + its running count
        t0 = g_offset(a, r);
    };
    if (r >= 0) load_request();
    const int64_t cap = *a.g_total;
    bool bad = false;
#pragma unroll
    for (int k = 0; k < VTK_TILE_TOK; ++k) {
        if (t + k >= T) break;
        if (t + k >= next && r + 1 < R) {                     // a request boundary inside the thread's entries
            while (r + 1 < R && g_offset(a, r + 1) <= t + k) ++r;
            next = g_offset(a, r + 1);
            load_request();
        }
        if (r < 0 || !sel) continue;
        if (slot[k] >= 0 && (int64_t)slot[k] >= a.slots_per_layer) bad = true;     // reported for selected requests only
        if (!((bits >> k) & 1u)) continue;
        const int64_t i = (int64_t)first_row + before + __popc(bits & ((1u << k) - 1u));
        if (i < 0 || i >= cap) continue;
        a.g_src[i] = slot[k];
        if (!a.g_ids.null()) a.g_ids[i] = (int32_t)(t + k - t0);
        if (!a.g_req.null()) a.g_req[i] = r;
    }
    if (bad) atomicOr(&a.counts->error_flags, VTOKEN_FLAG_BAD_SLOT);
}

// count -> scan -> assign: flat tiles when the context has their scratch, else the per-request kernels
int launch_index(vtoken_ctx *ctx, GatherArgs &a, cudaStream_t st)
{
    if (ctx->g_tile_n != nullptr) {
        a.tile_n = VTK_ARR(ctx, ctx->g_tile_n, (ctx->cfg.max_tokens + VTK_TILE - 1) / VTK_TILE + 1);
        a.req_part = VTK_ARR(ctx, ctx->g_req_part, (int64_t)ctx->cfg.max_requests + 1);
        a.req_before = VTK_ARR(ctx, ctx->g_req_before, (int64_t)ctx->cfg.max_requests + 1);
        a.num_tiles = (int32_t)((ctx->cfg.max_tokens + VTK_TILE - 1) / VTK_TILE);
        a.vec_in = ((uintptr_t)a.tt_slots.p % 16 == 0 && (a.keep.null() || (uintptr_t)a.keep.p % 4 == 0)) ? 1 : 0;
#ifdef VTOKEN_CHECKED
        a.vec_in = 0;              // one checked access per entry instead of one per four
#endif
        a.table_cap = ctx->cfg.max_tokens;
        VTK_CUDA(ctx, vtk_launch_dependent(ctx, gather_tiles_kernel, dim3(a.num_tiles + ctx->cfg.max_requests + 1),
                                           dim3(VTK_TILE_NT), 0, st, a));
        VTK_CUDA(ctx, vtk_launch_dependent(ctx, gather_scan_flat_kernel, dim3(1), dim3(1024), 0, st, a));
        VTK_CUDA(ctx, vtk_launch_dependent(ctx, gather_assign_flat_kernel, dim3(a.num_tiles), dim3(VTK_TILE_NT), 0, st, a));
        return VTOKEN_OK;
    }
    VTK_CUDA(ctx, vtk_launch_dependent(ctx, gather_count_kernel, dim3(ctx->cfg.max_requests * a.parts), dim3(G_NT), 0, st, a));
    VTK_CUDA(ctx, vtk_launch_dependent(ctx, gather_scan_kernel, dim3(1), dim3(1024), 0, st, a));
    VTK_CUDA(ctx, vtk_launch_dependent(ctx, gather_assign_kernel, dim3(ctx->cfg.max_requests * a.parts), dim3(G_NT), 0, st, a));
    return VTOKEN_OK;
}

__device__ __forceinline__ uint4 ld_stream(const uint4 *p)
{
    uint4 v;
    asm volatile("ld.global.cs.v4.u32 {%0,%1,%2,%3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "l"(p));
    return v;
}
__device__ __forceinline__ void st_stream(uint4 *p, const uint4 &v)
{
    asm volatile("st.global.cs.v4.u32 [%0], {%1,%2,%3,%4};" ::"l"(p), "r"(v.x), "r"(v.y), "r"(v.z), "r"(v.w) : "memory");
}

constexpr int GC_NT = 256;

// one warp per (pool, layer, output row)
__global__ void __launch_bounds__(GC_NT) gather_copy_kernel(GatherArgs a)
{
    vtk_release_successor();
    vtk_wait_for_predecessor();
    const int64_t n = *a.g_total;
    const int nl = a.layer_end - a.layer_begin;
    const int64_t total = n * nl * 2;
    const int lane = vtk_lane();
    const int64_t nwarps = (int64_t)gridDim.x * (GC_NT / 32);
    const int row_vecs = (int)(a.row_bytes >> 4);
    for (int64_t u = (int64_t)blockIdx.x * (GC_NT / 32) + (threadIdx.x >> 5); u < total; u += nwarps) {
        const int slab = (int)(u / n);                 // [0, nl): K layers, [nl, 2nl): V layers
        const int64_t idx = u - (int64_t)slab * n;
        const int li = slab < nl ? slab : slab - nl;
        const uint8_t *pool = slab < nl ? a.k_pool : a.v_pool;
        uint8_t *out = slab < nl ? a.out_k : a.out_v;
        const int32_t src = a.g_src[idx];
        const uint4 *sp = reinterpret_cast<const uint4 *>(pool + (int64_t)(a.layer_begin + li) * a.layer_stride +
                                                          (int64_t)src * a.row_bytes);
        uint4 *dp = reinterpret_cast<uint4 *>(out + ((int64_t)li * a.out_capacity + idx) * a.row_bytes);
        for (int c = lane; c < row_vecs; c += 128) {
            uint4 v[4];
#pragma unroll
            for (int k = 0; k < 4; ++k)
                if (c + 32 * k < row_vecs) v[k] = ld_stream(sp + c + 32 * k);
#pragma unroll
            for (int k = 0; k < 4; ++k)
                if (c + 32 * k < row_vecs) st_stream(dp + c + 32 * k, v[k]);
        }
    }
}

__device__ __forceinline__ unsigned long long g_mix64(unsigned long long x)   // splitmix64 finaliser
{
    x ^= x >> 30;
    x *= 0xBF58476D1CE4E5B9ull;
    x ^= x >> 27;
    x *= 0x94D049BB133111EBull;
    x ^= x >> 31;
    return x;
}

// Relocation digest (Sec. 5 of the paper hashes ordered retained ids with their K/V contents):
//   key(i, s) = mix(((i*A + t_i)*B + s)*C);  per 32-byte group g of the row (8-byte words w_4g .. w_4g+3,
//   x_j = w_j ^ (key + j*D)):  a = x_4g + x_4g+2, b = x_4g+1 + x_4g+3;  digest[r] = sum of low64(a*b) ^ high64(a*b)
// a sum of position-bound terms, so any evaluation order gives the same 64-bit value.
// A warp walks a contiguous run of (slab, output row) units; lanes take 32-byte groups of the row.
// One (slab, row) unit of the digest: where it is and what it hashes.
struct DigestRow {
    const uint4 *ptr;            // first byte of the K or V row
    int32_t r, tok, slab, idx;
};

__global__ void __launch_bounds__(GC_NT, 3) gather_digest_kernel(GatherArgs a)
{
    vtk_release_successor();
    vtk_wait_for_predecessor();
    const unsigned long long A = 0x9E3779B97F4A7C15ull, B = 0xD1B54A32D192ED03ull, C = 0x8CB92BA72F3D8DD7ull,
                             D = 0xA0761D6478BD642Full;
    const int64_t n = *a.g_total;
    const int nl = a.layer_end - a.layer_begin;
    const int64_t total = n * nl * 2;
    const int lane = vtk_lane();
    const int row_vecs = (int)(a.row_bytes >> 4);
    // A row is hashed by a group of G lanes, each taking two 32-byte groups of the row (four 16-byte
    // loads): the whole warp for rows of 2 KiB and more, half a warp for 1 KiB rows, ... so that
    // every lane's loads carry bytes.
    const int row_groups = (row_vecs + 1) >> 1;                // 32-byte groups, the last one may be half
    int G = 32;
    while (G > 1 && 2 * G > row_groups) G >>= 1;
    const int gl = lane & (G - 1), per_warp = 32 / G;
    const unsigned gmask = G == 32 ? 0xffffffffu : (((1u << G) - 1u) << (lane & ~(G - 1)));
    const int64_t ngroups = (int64_t)gridDim.x * (GC_NT / 32) * per_warp;
    // Each group takes a contiguous run of (slab, row) pairs, so that consecutive rows mostly belong
    // to one request: the per-lane partial sums are folded into the request's digest only when the
    // request changes (one 64-bit atomic per run instead of one per row -- with one atomic per row
    // the kernel was bound by atomic throughput on a few addresses).
    const int64_t chunk = (total + ngroups - 1) / ngroups;
    const int64_t w = ((int64_t)blockIdx.x * (GC_NT / 32) + (threadIdx.x >> 5)) * per_warp + lane / G;
    const int64_t u0 = w * chunk, u1 = min(total, u0 + chunk);
    if (u0 >= u1) return;                                      // whole groups leave; shuffles below name gmask
    unsigned long long sum = 0;
    int cur_r = -1;
    auto flush = [&]() {
#pragma unroll
        for (int d = 16; d > 0; d >>= 1)
            if (d < G) sum += __shfl_down_sync(gmask, sum, d, G);
        if (gl == 0 && cur_r >= 0 && sum != 0) atomicAdd(&a.digest[cur_r], sum);
        sum = 0;
    };
    const uint8_t *slab_base = nullptr;                        // pool + layer offset of the slab being fetched
    auto set_slab = [&](int slab) {
        const int li = slab < nl ? slab : slab - nl;
        slab_base = (slab < nl ? a.k_pool : a.v_pool) + (int64_t)(a.layer_begin + li) * a.layer_stride;
    };
    const uint32_t row_bytes32 = (uint32_t)a.row_bytes;        // rows are far below 4 GiB
    auto fetch_meta = [&](DigestRow &m, int slab, int32_t idx) {
        m.slab = slab;
        m.idx = idx;
        m.ptr = reinterpret_cast<const uint4 *>(slab_base + (uint64_t)(uint32_t)a.g_src[idx] * row_bytes32);
        m.r = a.g_req[idx];
        m.tok = a.g_ids[idx];
    };
    // v[2m], v[2m+1] = the two 16-byte halves of 32-byte group p0 + G*m, m = 0, 1
    auto load4 = [&](uint4 (&v)[4], const uint4 *sp, int p0) {
#pragma unroll
        for (int k = 0; k < 4; ++k) {
            const int vec = 2 * (p0 + G * (k >> 1)) + (k & 1);
            v[k] = vec < row_vecs ? ld_stream(sp + vec) : make_uint4(0, 0, 0, 0);
        }
    };
    // word offsets without multiplies in the row loop: the words of group p = p0 + G*m carry the
    // offsets (4p + j)*D = 4*p0*D + m*(4*G*D) + j*D, j = 0..3
    const unsigned long long lane_off = 4ull * gl * D, k_step = 4ull * G * D;
    auto hash4 = [&](const uint4 (&v)[4], unsigned long long key_p0, int p0) {   // key_p0 = key + 4*p0*D
#pragma unroll
        for (int m = 0; m < 2; ++m) {
            const int p = p0 + G * m;
            if (2 * p < row_vecs) {
                const unsigned long long ko = key_p0 + (unsigned long long)m * k_step;
                const unsigned long long w0 = ((unsigned long long)v[2 * m].y << 32) | v[2 * m].x;
                const unsigned long long w1 = ((unsigned long long)v[2 * m].w << 32) | v[2 * m].z;
                unsigned long long x = w0 ^ ko, y = w1 ^ (ko + D);
                if (2 * p + 1 < row_vecs) {                        // the second half of the group exists
                    const unsigned long long w2 = ((unsigned long long)v[2 * m + 1].y << 32) | v[2 * m + 1].x;
                    const unsigned long long w3 = ((unsigned long long)v[2 * m + 1].w << 32) | v[2 * m + 1].z;
                    x += w2 ^ (ko + 2ull * D);
                    y += w3 ^ (ko + 3ull * D);
                }
                sum += (x * y) ^ __umul64hi(x, y);                 // low64 ^ high64 of the 128-bit product
            }
        }
    };
    // Software pipeline over rows: the table entries of a row (source slot, request, logical id)
    // are fetched two rows ahead and the first 64 bytes per lane of its K/V row one row ahead, so
    // that a group always has a row in flight while it hashes the previous one.
    int slab = (int)(u0 / n);
    int32_t idx = (int32_t)(u0 - (int64_t)slab * n);             // n < 2^31: it counts token-table entries
    const int32_t n32 = (int32_t)n;
    auto advance = [&]() { if (++idx == n32) { idx = 0; set_slab(++slab); } };
    set_slab(slab);
    DigestRow cur, nxt;
    fetch_meta(cur, slab, idx);
    advance();
    if (u0 + 1 < u1) { fetch_meta(nxt, slab, idx); advance(); }
    uint4 vc[4], vn[4];
    load4(vc, cur.ptr, gl);
    for (int64_t left = u1 - u0; left > 0; --left) {
        const bool has_next = left > 1;
        if (has_next) load4(vn, nxt.ptr, gl);
        DigestRow nn = nxt;
        if (left > 2) { fetch_meta(nn, slab, idx); advance(); }
        if (cur.r != cur_r) {
            flush();
            cur_r = cur.r;
        }
        const unsigned long long i = (unsigned long long)(cur.idx - a.out_offsets[cur.r]);
        const unsigned long long key =
            g_mix64(((i * A + (unsigned long long)cur.tok) * B + (unsigned long long)cur.slab) * C);
        unsigned long long key_p0 = key + lane_off;
        hash4(vc, key_p0, gl);
        if (row_groups > 2 * G) {                              // rows above 64 bytes per lane: the rest, unpipelined
            for (int p0 = gl + 2 * G; p0 < row_groups; p0 += 2 * G) {
                uint4 v[4];
                key_p0 += 2ull * k_step;
                load4(v, cur.ptr, p0);
                hash4(v, key_p0, p0);
            }
        }
#pragma unroll
        for (int k = 0; k < 4; ++k) vc[k] = vn[k];
        cur = nxt;
        nxt = nn;
    }
    flush();
}

// the table inputs and the scratch every call of the gather family uses
void bind_inputs(vtoken_ctx *ctx, GatherArgs &a, const int32_t *num_requests, const int32_t *tt_offsets,
                 const int32_t *tt_slots, const uint8_t *keep, const uint8_t *select)
{
    const vtoken_config &c = ctx->cfg;
    a.num_requests = VTK_ARR(ctx, num_requests, 1);
    a.tt_offsets = VTK_ARR(ctx, tt_offsets, (int64_t)c.max_requests + 1);
    a.tt_slots = VTK_ARR(ctx, tt_slots, c.max_tokens);
    a.keep = VTK_ARR(ctx, keep, c.max_tokens);
    a.select = VTK_ARR(ctx, select, c.max_requests);
    a.req_n = VTK_ARR(ctx, ctx->req_n, c.max_requests);
    a.part_n = VTK_ARR(ctx, ctx->part_n, (int64_t)c.max_requests * G_PARTS);
    a.g_total = VTK_ARR(ctx, ctx->g_total, 1);
    a.counts = VTK_ARR(ctx, ctx->rt_counts, 1);
    a.g_ids = vtk_arr<int32_t>();
    a.g_req = vtk_arr<int32_t>();
    a.digest = vtk_arr<unsigned long long>();
    a.tile_n = a.req_part = a.req_before = vtk_arr<int32_t>();
}

}  // namespace

extern "C" int vtoken_digest_logical(vtoken_ctx *ctx, const int32_t *num_requests, const int32_t *tt_offsets,
                                     const int32_t *tt_slots, const uint8_t *keep, const uint8_t *select,
                                     int32_t layer_begin, int32_t layer_end, uint64_t *out_digest,
                                     int32_t *out_offsets, void *cuda_stream)
{
    if (!ctx || !num_requests || !tt_offsets || !tt_slots || !out_digest) return VTOKEN_EINVAL;
    if (layer_begin < 0 || layer_end > ctx->cfg.num_layers || layer_begin >= layer_end) return VTOKEN_EINVAL;
    cudaStream_t st = (cudaStream_t)cuda_stream;
    GatherArgs a;
    bind_inputs(ctx, a, num_requests, tt_offsets, tt_slots, keep, select);
    a.out_offsets = VTK_ARR(ctx, out_offsets ? out_offsets : ctx->g_offsets, (int64_t)ctx->cfg.max_requests + 1);
    a.g_src = VTK_ARR(ctx, ctx->g_src, ctx->cfg.max_tokens);
    a.g_ids = VTK_ARR(ctx, ctx->g_ids, ctx->cfg.max_tokens);
    a.g_req = VTK_ARR(ctx, ctx->g_req, ctx->cfg.max_tokens);
    a.digest = VTK_ARR(ctx, (unsigned long long *)out_digest, ctx->cfg.max_requests);
    a.k_pool = (const uint8_t *)ctx->cfg.k_pool;
    a.v_pool = (const uint8_t *)ctx->cfg.v_pool;
    a.out_k = a.out_v = nullptr;
    a.layer_stride = ctx->layer_stride;
    a.row_bytes = ctx->row_bytes;
    a.slots_per_layer = ctx->slots_per_layer;
    a.out_capacity = ctx->cfg.max_tokens;
    a.max_tokens = ctx->cfg.max_tokens;
    a.layer_begin = layer_begin;
    a.layer_end = layer_end;
    a.max_requests = ctx->cfg.max_requests;
    a.parts = G_PARTS;
    VTK_CUDA(ctx, cudaMemsetAsync(out_digest, 0, sizeof(uint64_t) * (size_t)ctx->cfg.max_requests, st));
    { const int rc = launch_index(ctx, a, st); if (rc != VTOKEN_OK) return rc; }
    VTK_CUDA(ctx, vtk_launch_dependent(ctx, gather_digest_kernel, dim3(ctx->num_sms * 8), dim3(GC_NT), 0, st, a));
    VTK_CUDA(ctx, cudaGetLastError());
    return VTOKEN_OK;
}

int vtk_launch_gather(vtoken_ctx *ctx, const int32_t *num_requests, const int32_t *tt_offsets,
                      const int32_t *tt_slots, const uint8_t *keep, const uint8_t *select,
                      int32_t layer_begin, int32_t layer_end, void *out_k, void *out_v,
                      int64_t out_capacity_tokens, int32_t *out_offsets, cudaStream_t st)
{
    GatherArgs a;
    bind_inputs(ctx, a, num_requests, tt_offsets, tt_slots, keep, select);
    a.out_offsets = VTK_ARR(ctx, out_offsets, (int64_t)ctx->cfg.max_requests + 1);
    a.g_src = VTK_ARR(ctx, ctx->g_src, ctx->cfg.max_tokens);
    a.k_pool = (const uint8_t *)ctx->cfg.k_pool;
    a.v_pool = (const uint8_t *)ctx->cfg.v_pool;
    a.out_k = (uint8_t *)out_k;
    a.out_v = (uint8_t *)out_v;
    a.layer_stride = ctx->layer_stride;
    a.row_bytes = ctx->row_bytes;
    a.slots_per_layer = ctx->slots_per_layer;
    a.out_capacity = out_capacity_tokens;
    a.max_tokens = ctx->cfg.max_tokens;
    a.layer_begin = layer_begin;
    a.layer_end = layer_end;
    a.max_requests = ctx->cfg.max_requests;
    a.parts = G_PARTS;
    { const int rc = launch_index(ctx, a, st); if (rc != VTOKEN_OK) return rc; }
    // the rows go through the bulk-copy rings when the context has them (vtoken_create does; the
    // context-free entry point does not), else through the register kernel
    const bool aligned = (((uintptr_t)out_k | (uintptr_t)out_v) & 15) == 0;
    const int bulk = aligned ? vtk_launch_gather_bulk(ctx, ctx->g_src, ctx->g_total, layer_begin, layer_end, out_k, out_v,
                                                      out_capacity_tokens, st) : 0;
    if (bulk < 0) return bulk;
    if (bulk == 0)
        VTK_CUDA(ctx, vtk_launch_dependent(ctx, gather_copy_kernel, dim3(ctx->num_sms * 8), dim3(GC_NT), 0, st, a));
    VTK_CUDA(ctx, cudaGetLastError());
    return VTOKEN_OK;
}

// Slot mapping (Sec. 3.4): the same count / scan / assign, with the slot list written straight
// into the caller's buffer and no row copy.
extern "C" int vtoken_build_slot_mapping(vtoken_ctx *ctx, const int32_t *num_requests, const int32_t *tt_offsets,
                                         const int32_t *tt_slots, const uint8_t *keep, const uint8_t *select,
                                         int32_t *out_slots, int32_t *out_token_ids, int64_t out_capacity,
                                         int32_t *out_offsets, void *cuda_stream)
{
    if (!ctx || !num_requests || !tt_offsets || !tt_slots || !out_slots || !out_offsets) return VTOKEN_EINVAL;
    if (out_capacity < 0) return VTOKEN_EINVAL;
    cudaStream_t st = (cudaStream_t)cuda_stream;
    GatherArgs a;
    bind_inputs(ctx, a, num_requests, tt_offsets, tt_slots, keep, select);
    a.out_offsets = VTK_ARR(ctx, out_offsets, (int64_t)ctx->cfg.max_requests + 1);
    a.g_src = VTK_ARR(ctx, out_slots, out_capacity);
    a.g_ids = VTK_ARR(ctx, out_token_ids, out_capacity);
    a.k_pool = a.v_pool = nullptr;
    a.out_k = a.out_v = nullptr;
    a.layer_stride = 0;
    a.row_bytes = 0;
    a.slots_per_layer = ctx->slots_per_layer;
    a.out_capacity = out_capacity;
    a.max_tokens = out_capacity;
    a.layer_begin = a.layer_end = 0;
    a.max_requests = ctx->cfg.max_requests;
    a.parts = G_PARTS;
    { const int rc = launch_index(ctx, a, st); if (rc != VTOKEN_OK) return rc; }
    VTK_CUDA(ctx, cudaGetLastError());
    return VTOKEN_OK;
}
