/*
 * vtoken.h -- C ABI of the B200 (sm_100a) repack library for token-evicted paged KV caches.
 *
 * The library implements the reclamation backend's relocation step of vToken: the live
 * tokens of fragmented requests are compacted into dense destination blocks and the
 * indirection tables are rewritten so that the logical token view of every request stays
 * the same while whole blocks become free.
 *
 * Vocabulary (paper notation): S = block size, a slot = block_id * S + offset (Sec. 3.4,
 * slot-mapping equation); block table = logical block -> physical block (Sec. 2.1);
 * token table = logical token id -> slot, plus a liveness bit (Sec. 3.2) -- here an int32
 * slot with -1 for "no physical copy" and a separate uint8 keep mask written by the
 * eviction policy (evict_token marks, Sec. 3.2).
 *
 * Memory: every pointer below says DEVICE or HOST.  The caller owns all of them; the
 * library owns only scratch it allocates in vtoken_create.  K and V pools are laid out
 * [num_layers][num_blocks][block_size][num_kv_heads][head_dim] with elem_bytes-wide
 * elements that are treated as opaque bytes (any bit pattern survives).
 *
 * Streams and graphs: vtoken_plan, vtoken_repack and vtoken_gather_logical only enqueue
 * kernels on the given stream.  They allocate nothing, never synchronise and never read
 * device data on the host; every grid is fixed by the capacities given at create time and
 * every data-dependent count stays in device memory.  They can therefore be captured in a
 * CUDA graph and replayed after the caller rewrites the CONTENTS of the input buffers.
 *
 * Ordering contract (Sec. 3.3.4, invariant I3): call vtoken_plan then vtoken_repack on the
 * same stream (or ordered by events).  Inputs must stay unmodified until the repack has
 * completed.  The outputs are the PROPOSED new state: record an event behind vtoken_repack;
 * make every consumer of the new tables wait on it; only after it may the caller adopt the
 * new tables, return freed_blocks[0 .. num_freed) to its allocator and drop
 * free_blocks[0 .. num_free_consumed).  One plan may be in flight per context (I4).
 *
 * Errors: every function returns 0 (VTOKEN_OK) or a negative code, never aborts or throws.
 * Argument and capacity problems visible on the host return an error and enqueue nothing.
 * Data-dependent problems found on the device (slot or block id out of range, request or
 * token count above the capacities, output overflow) set a bit in counts.error_flags; the
 * offending row or request is skipped and the kernels complete.  A short free list is not an
 * error: the request gets status VTOKEN_DEFERRED_NO_FREE (Sec. 3.3.2).
 *
 * Bounded waits: the only waits inside the kernels are on shared-memory barriers that the
 * kernel's own bulk copies complete.  Each is bounded (default 2 s, vtoken_config.wait_limit_ms
 * changes it): when it runs out the warp sets VTOKEN_FLAG_TIMEOUT, gives its copies in flight a
 * bounded time to land and returns, so the kernel always ends and the context stays usable.  Rows
 * may then be missing: those of the item the warp was waiting for, of the items already in its
 * ring, of the rest of its ticket and of the ticket it had requested ahead.
 *
 * Threads: a context is not thread-safe.  Calls on one context must come from one thread at a
 * time; different contexts (different pools) are independent.
 *
 * No environment variable is read: every knob is a field of vtoken_config.
 *
 * Preconditions assumed (not checked) on the fast path: each live slot is referenced by one
 * token only (I2) and lies in a block of its own request; block ids are unique across block
 * tables (shared-prefix blocks are excluded from plans, I4); the free list has no duplicates
 * and is disjoint from all block tables.
 */
#ifndef VTOKEN_H
#define VTOKEN_H
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct vtoken_ctx vtoken_ctx;

/* return codes */
enum {
    VTOKEN_OK = 0,
    VTOKEN_EINVAL = -1,      /* malformed argument (NULL, shape, alignment) */
    VTOKEN_ECAPACITY = -2,   /* a size exceeds a capacity given at create time */
    VTOKEN_ECUDA = -3,       /* a CUDA call failed; see vtoken_last_cuda_error */
    VTOKEN_ENOMEM = -4,      /* scratch allocation failed in vtoken_create */
    VTOKEN_ESTATE = -5       /* vtoken_repack without a plan */
};

/* per-request status written by vtoken_plan */
enum {
    VTOKEN_NOT_SELECTED = 0,     /* not chosen by select[] / at or above the live-fraction threshold */
    VTOKEN_REPACKED = 1,         /* admitted: its live tokens move, all its old blocks are reclaimed */
    VTOKEN_NO_GAIN = 2,          /* ceil(n/S) is not below its block count (I4: must strictly decrease) */
    VTOKEN_DEFERRED_NO_FREE = 3  /* candidate, but the free list cannot supply its destinations */
};

/* bits of vtoken_counts.error_flags */
enum {
    VTOKEN_FLAG_BAD_SLOT = 1u,        /* a token-table slot >= num_blocks * block_size: token treated as not live */
    VTOKEN_FLAG_BAD_BLOCK = 2u,       /* a block-table id outside [0, num_blocks) */
    VTOKEN_FLAG_BAD_FREE = 4u,        /* a free-list id outside [0, num_blocks): that destination block is skipped */
    VTOKEN_FLAG_CAPACITY = 8u,        /* R, num_free, or a table range beyond the create-time capacities: R and
                                         num_free are clamped; table entries at or beyond max_tokens /
                                         max_table_blocks (and ranges that run backwards) do not exist for the
                                         planners, so no output buffer is written behind its capacity */
    VTOKEN_FLAG_TIMEOUT = 16u,        /* a bounded wait inside a kernel ran out; rows may be missing */
    VTOKEN_FLAG_GATHER_OVERFLOW = 32u,/* gather_logical / build_slot_mapping: more live tokens than the output holds */
    VTOKEN_FLAG_BAD_VICTIM = 64u,     /* vtoken_evict_tokens: a victim outside its request's registered tokens: skipped */
    VTOKEN_FLAG_APPEND_STOPPED = 128u,/* vtoken_sync_new_tokens: table capacity or block list exhausted: request grew less */
    VTOKEN_FLAG_CHECK_FAILED = 256u   /* checked build only: an index into scratch, a table or a pool fell outside its
                                         range; the access was skipped */
};

/* Launch shape of the bulk-copy kernel (tuning and tests; the defaults are the measured best).
 * With enabled == 0 every field is ignored.  With enabled != 0: warps per CTA (0 => 8, at most 16),
 * ring stages per warp (0 => 4, 2 .. 12), rows per work item (0 => 4 KiB worth; rounded down to a
 * power of two that divides the block size, at most 32), work items loading ahead of the one being
 * stored (0 .. stages - 2), plan entries fetched ahead (1 or 2), fixed_shares != 0: every warp gets a
 * fixed share of the work items instead of taking them from a ticket counter, chunk = items per
 * ticket (0 => one ticket per >= 16 KiB, at least 4 items), ctas = grid size (0 => auto). */
typedef struct {
    int32_t enabled;
    int32_t warps, stages, rows, depth, ahead;
    int32_t fixed_shares, chunk, ctas;
} vtoken_copy_tuning;

typedef struct {
    int32_t num_layers, num_blocks, block_size, num_kv_heads, head_dim;
    int32_t elem_bytes;            /* bytes per element (2 for bf16/fp16); rows are opaque bytes */
    void *k_pool, *v_pool;         /* DEVICE, 16-byte aligned, must outlive the context */
    int64_t layer_stride_bytes;    /* bytes between layers of a pool; 0 => num_blocks*block_size*row_bytes */
    int32_t max_requests;          /* capacities: they fix every grid and scratch size */
    int64_t max_tokens;            /* upper bound of the token-table length (sum of request lengths) */
    int64_t max_table_blocks;      /* upper bound of the block-table length (sum over requests) */
    int32_t max_free_blocks;       /* upper bound of num_free */
    int32_t max_ctas;              /* copy-kernel grid cap, 0 => one CTA per SM.  The default launch shape (128 KiB of
                                      shared-memory rings per SM) is also the one with which a repack beside a
                                      bandwidth-bound decode kernel costs that kernel least (the overlapped operation
                                      Sec. 5 measures as a stress test); a smaller grid gives the other kernel a larger
                                      share of HBM still, at the price of a slower repack */
    int32_t copy_variant;          /* 0 auto (bulk-copy path when row_bytes <= 32768, else register path);
                                      1 register path; 2 bulk-copy (TMA) path */
    int32_t wait_limit_ms;         /* bound of every wait inside a kernel, 1 .. 60000; 0 => 2000 */
    int32_t plain_launches;        /* 0: every kernel of the library is launched with programmatic stream
                                      serialization, i.e. it may become resident while the previous kernel in the
                                      stream is finishing and waits (griddepcontrol.wait, first thing it does) until
                                      that kernel has completed and its writes are visible; a chain of short
                                      kernels loses about 1 us per boundary, results are identical, and a caller's
                                      own kernel that follows in the stream is ordered as usual.  1: plain
                                      stream-ordered launches */
    int32_t plan_variant;          /* whole-request planner: 0 auto; 1 three kernels (count, scan, assign); 2 two
                                      kernels, every CTA redoing the scan over the requests (tables whose grid of
                                      tiles + requests is resident at once; larger capacities fall back to 1).
                                      Same results either way; other values are VTOKEN_EINVAL */
    vtoken_copy_tuning tuning;     /* see above; all zero => defaults */
    int64_t debug_stall_item;      /* must be 0 for the production library (VTOKEN_EINVAL otherwise).  The checked
                                      build (libvtoken_checked.so) arms the barrier of work item
                                      debug_stall_item - 1 of the copy kernel with bytes that never arrive, so that
                                      its wait runs out: the time-out path is exercised without faulting anything */
} vtoken_config;

/* row_bytes = num_kv_heads * head_dim * elem_bytes must be a multiple of 16, pools and
 * layer stride 16-byte aligned (VTOKEN_EINVAL otherwise).  Allocates all scratch once. */
int vtoken_create(const vtoken_config *cfg, vtoken_ctx **out_ctx);
void vtoken_destroy(vtoken_ctx *ctx);

typedef struct {                   /* all DEVICE pointers, read-only to the library */
    const int32_t *num_requests;   /* device scalar R <= max_requests */
    const int32_t *bt_offsets;     /* [R+1] CSR offsets into bt_blocks */
    const int32_t *bt_blocks;      /* [bt_offsets[R]] physical block ids, logical block order */
    const int32_t *tt_offsets;     /* [R+1] CSR offsets into tt_slots / keep, non-decreasing; entries in front of
                                      tt_offsets[0] belong to no request: neither read as tokens nor written */
    const int32_t *tt_slots;       /* [tt_offsets[R]] slot = block*S+offset, or -1 */
    const uint8_t *keep;           /* [tt_offsets[R]] 0 = evicted, non-zero = keep */
    const uint8_t *select;         /* [R] or NULL (= every request) */
    uint32_t thr_num, thr_den;     /* candidate iff n_r*thr_den < thr_num*nb_r*S (64-bit); thr_den==0 => no threshold */
    const int32_t *free_blocks;    /* caller's free list, consumed from index 0 in list order */
    const int32_t *num_free;       /* device scalar <= max_free_blocks */
} vtoken_plan_in;

typedef struct {
    int32_t num_moves;             /* live tokens of admitted requests (rows moved per layer per pool) */
    int32_t num_dst_blocks;        /* destination blocks written */
    int32_t num_freed;             /* entries of freed_blocks */
    int32_t num_free_consumed;     /* entries taken from the front of free_blocks (== num_dst_blocks) */
    int32_t num_admitted;          /* requests with status VTOKEN_REPACKED */
    int32_t num_deferred;          /* requests with status VTOKEN_DEFERRED_NO_FREE */
    uint32_t error_flags;          /* VTOKEN_FLAG_* */
    int32_t num_released;          /* entries of released_blocks (copy-on-write detach of vtoken_plan_partial) */
} vtoken_counts;

typedef struct {                   /* all DEVICE pointers, written by vtoken_plan */
    int32_t *new_bt_offsets;       /* [R+1] */
    int32_t *new_bt_blocks;        /* capacity max_table_blocks */
    int32_t *new_tt_slots;         /* [T], same CSR offsets as the input token table */
    int32_t *freed_blocks;         /* capacity max_table_blocks */
    int32_t *req_status;           /* [R] VTOKEN_NOT_SELECTED .. VTOKEN_DEFERRED_NO_FREE */
    vtoken_counts *counts;         /* one struct */
    int32_t *released_blocks;      /* capacity max_table_blocks; only vtoken_plan_partial with a detach threshold
                                      writes it (may be NULL otherwise) */
} vtoken_plan_out;

/* Relocation planning and table rewrite (Sec. 3.3.3; apply_moves of Sec. 3.2; I1, I2, I4).
 * For every request in ascending index: n = live tokens (slot >= 0 and keep != 0),
 * need = ceil(n / S).  A selected request below the threshold with need < its block count is
 * a candidate; candidates are admitted in order while the cumulative need fits num_free, all
 * later candidates are deferred.  An admitted request receives the next `need` entries of
 * free_blocks; its i-th live token (logical order) gets slot dst[i / S] * S + i % S; its new
 * block table is dst[0 .. need); its old blocks are appended to freed_blocks in table order.
 * Every other request keeps its block table and the slots of its live tokens.  Entries of
 * evicted tokens become -1 in every request.  The move plan is kept inside the context for
 * vtoken_repack.  The structs are read on the host during the call (HOST pointers to
 * structs holding DEVICE pointers). */
int vtoken_plan(vtoken_ctx *ctx, const vtoken_plan_in *in, const vtoken_plan_out *out, void *cuda_stream);

/* Stage-aware asynchronous copy (Sec. 3.3.4): executes the plan held in the context.  For
 * every move, every layer, K and V: row[dst_slot] = row[src_slot], row_bytes each, in place
 * in the pools.  Destinations are free blocks, sources are allocated blocks, so the two sets
 * are disjoint and no other byte of the pools changes.  One launch covers all layers and both
 * pools; the amount of work is read from device memory. */
int vtoken_repack(vtoken_ctx *ctx, void *cuda_stream);

/* Logical view (invariant I1; the before/after relocation check of Sec. 5): K and V rows of
 * the active tokens (slot >= 0, and keep != 0 when keep is given) of the selected requests in
 * request order then token-id order, for layers [layer_begin, layer_end), written densely:
 *   out_k / out_v : DEVICE, [layer_end-layer_begin][out_capacity_tokens][row_bytes] bytes
 *                   (the layer stride is out_capacity_tokens rows whatever the live count)
 *   out_offsets   : DEVICE int32 [R+1], first output row of each request (unselected: empty)
 * Tokens beyond out_capacity_tokens are dropped and VTOKEN_FLAG_GATHER_OVERFLOW is set in the
 * context's flags (see vtoken_read_counts).  The gather family -- this call, vtoken_digest_logical
 * and vtoken_build_slot_mapping -- has scratch of its own: such a call may overlap a plan / repack
 * in flight on another stream (the slot mapping is built every decode step on the compute stream
 * while relocation runs beside it, Sec. 3.3.4), but two calls of the family must not overlap each
 * other. */
int vtoken_gather_logical(vtoken_ctx *ctx, const int32_t *num_requests, const int32_t *tt_offsets,
                          const int32_t *tt_slots, const uint8_t *keep, const uint8_t *select,
                          int32_t layer_begin, int32_t layer_end, void *out_k, void *out_v,
                          int64_t out_capacity_tokens, int32_t *out_offsets, void *cuda_stream);

/* Online relocation check (Sec. 5, "Relocation Correctness": the ordered retained token ids are
 * hashed together with their K/V contents before and after a relocation).  The paper does not
 * name the hash; this library fixes one that any evaluation order reproduces bit for bit: for a
 * request whose active tokens have rank i = 0, 1, ... and logical ids t_i, over the slabs
 * s = 0 .. 2*(layer_end-layer_begin)-1 (K layers first, then V layers) and the 32-byte groups g of a
 * token's row, each four 8-byte little-endian words w_4g .. w_4g+3 (a row of 16 mod 32 bytes ends
 * with a group of two words),
 *     key(i, s) = mix(((i * A + t_i) * B + s) * C),      x_j = w_j ^ (key(i, s) + j * D),
 *     a = x_4g + x_4g+2,   b = x_4g+1 + x_4g+3           (mod 2^64; absent words add nothing),
 *     digest    = sum of  low64(a * b) ^ high64(a * b)  mod 2^64        (a * b: the 128-bit product),
 * mix = splitmix64 finaliser, A = 0x9E3779B97F4A7C15, B = 0xD1B54A32D192ED03, C = 0x8CB92BA72F3D8DD7,
 * D = 0xA0761D6478BD642F.
 * Equal digests before (old table + keep) and after (new table) a repack show token conservation
 * (I1) without materialising the rows.  out_digest: DEVICE uint64 [max_requests] (zeroed by the
 * call); out_offsets: DEVICE int32 [R+1] or NULL, first active-token index of each request (the
 * differences are the active counts).  Same selection arguments and scratch sharing as
 * vtoken_gather_logical. */
int vtoken_digest_logical(vtoken_ctx *ctx, const int32_t *num_requests, const int32_t *tt_offsets,
                          const int32_t *tt_slots, const uint8_t *keep, const uint8_t *select,
                          int32_t layer_begin, int32_t layer_end, uint64_t *out_digest, int32_t *out_offsets,
                          void *cuda_stream);

/* Copies the context's counts of the last plan (with the flags its repack raised) to HOST memory.
 * Flags raised since the previous vtoken_read_counts by the calls outside plan / repack (logical
 * gather, digest, slot mapping, token-table runtime, slot cache) are OR-ed in and reported once.
 * Synchronises the stream: the only call that does. */
int vtoken_read_counts(vtoken_ctx *ctx, vtoken_counts *host_out, void *cuda_stream);

/* ---- Eligibility metadata and partial plans (Sec. 3.3.1 - 3.3.3) --------------------------------
 * The paper's reclamation backend keeps per-block liveness n_b (live tokens stored in block b),
 * derives the intra-block waste ratio F = 1 - sum(n_b) / (N * S) over the N allocated blocks
 * (Sec. 2.3.1), attempts reclamation only when F exceeds a threshold theta_F (default 0.25,
 * Sec. 3.3.2), and plans per request over its under-utilised, unprotected blocks, at most B of
 * them, admitting a plan only when those sources release more blocks than the ceil(T_live / S)
 * destinations they need (Sec. 3.3.3).  Shared-prefix blocks are excluded from plans (I4). */

/* Per-block liveness: n_b[num_blocks] (DEVICE int32) = live tokens per physical block;
 * hist[block_size + 1] (DEVICE uint64, may be NULL) = number of block-table entries whose block
 * holds k live tokens; summary[2] (DEVICE int64, may be NULL) = {live tokens, allocated blocks},
 * i.e. F = 1 - summary[0] / (summary[1] * S).  Uses the context's planner scratch. */
int vtoken_block_liveness(vtoken_ctx *ctx, const int32_t *num_requests, const int32_t *bt_offsets,
                          const int32_t *bt_blocks, const int32_t *tt_offsets, const int32_t *tt_slots,
                          const uint8_t *keep, int32_t *n_b, uint64_t *hist, int64_t *summary, void *cuda_stream);

typedef struct {
    const uint8_t *protect;        /* DEVICE [num_blocks] or NULL: non-zero = the block never moves (shared prefix) */
    uint32_t util_num, util_den;   /* a block is a source iff n_b * util_den < util_num * S (64-bit);
                                      util_den == 0: every unprotected block (whole-request compaction);
                                      1/1: every block that is not fully live */
    int32_t max_source_blocks;     /* B: per request at most this many sources, the first eligible ones in
                                      block-table order; 0 = no bound */
    uint32_t theta_num, theta_den; /* global trigger: plan only when F > theta_num / theta_den (64-bit integers);
                                      theta_den == 0: always */
    uint32_t detach_num, detach_den; /* copy-on-write detach: a request leaves ALL its protected blocks when its own
                                      live tokens in them fill less than detach_num / detach_den of those blocks
                                      (n_shared * den < num * ns_shared * S); detach_den == 0: never */
    uint32_t detach_rule;          /* what the threshold is applied to.  0: the request's protected blocks as a whole
                                      (above).  1: every protected block by itself, on the request's own live tokens
                                      in it: it leaves b when n_rb * detach_den < detach_num * S and stays in the
                                      others.  2: every protected block by itself, on the live tokens of ALL its
                                      holders: every holder leaves b when n_b * detach_den < detach_num * S.
                                      Other values: VTOKEN_EINVAL */
} vtoken_partial_opts;

/* vtoken_plan restricted to source blocks.  Differences from vtoken_plan: only live tokens stored
 * in a request's source blocks move (logical order, destinations filled completely), need =
 * ceil(live tokens in sources / S), candidate iff need < number of sources; live tokens in the
 * other blocks keep their slots; new block table = the non-source blocks in old order followed by
 * the destinations; freed_blocks receives the source blocks in old order; when the trigger does
 * not hold every request is VTOKEN_NOT_SELECTED.  With all options zero / NULL the result equals
 * vtoken_plan's.  vtoken_repack executes the plan.
 *
 * Copy-on-write detach (the paper's outlook for shared-prefix blocks, Sec. 5 and Sec. 6: copying a
 * request's tokens out of shared blocks once the blocks it gets back outweigh the copy).  With a protect mask and
 * detach_den != 0, a request whose own live tokens occupy less than detach_num / detach_den of its
 * protected blocks treats all of them as sources too: its live tokens there are COPIED to its
 * destinations with the rest (the shared blocks keep their bytes for the other holders), the blocks
 * leave its table and are listed in out->released_blocks (a reference dropped; the caller's
 * reference counts decide when such a block is free) instead of freed_blocks; counts.num_released
 * says how many.  max_source_blocks bounds the unprotected sources only.  The gain gate is unchanged
 * (destinations < sources, in the request's own table), so whether the POOL gains depends on the
 * other holders: enabling detach is the caller's policy decision.  vtoken_repack_waves and
 * vtoken_repack_host_partial take the threshold too; each has a released list of its own in its
 * output struct.
 * With detach_rule 1 the threshold is applied block by block instead: the request leaves exactly
 * those protected blocks of its table in which its own live tokens (not the other holders') fill
 * less than the fraction of the S slots, and keeps the others in place, in old order with its other
 * kept blocks.  The planner then takes a census of every request's live tokens per protected table
 * entry (one more kernel and a memset of 16 B per block-table entry in front of the plan; a lookup
 * per live token in a protected block).  A token stored in a protected block that its request's
 * table does not list stays where it is.
 * With detach_rule 2 a protected block is judged by everything stored in it, n_b = the live tokens
 * of all its holders (one count per referencing token-table entry): every holder reaches the same
 * verdict, so the block is left by all the holders this plan repacks or by none.  The copies made
 * on leaving it (n_b tokens in all) take less room than the block they give back exactly when
 * n_b < S -- threshold 1/1 -- which makes this the rule under which the POOL gains whenever all
 * holders are repacked; it costs nothing beyond the plain partial plan (no census, no owners). */
int vtoken_plan_partial(vtoken_ctx *ctx, const vtoken_plan_in *in, const vtoken_partial_opts *opts,
                        const vtoken_plan_out *out, void *cuda_stream);

/* ---- Repack in waves: blocks reclaimed by one wave are destinations of the next ----------------
 * The paper returns source blocks to the free pool once the packed layout is committed (Sec. 3.3.4)
 * and defers plans that the evacuation headroom cannot serve (Sec. 3.3.2).  Chained on the device,
 * the two rules give a repack whose headroom is the largest single demand instead of the sum of
 * all demands: wave k plans against the pool P_k (vtoken_plan, or vtoken_plan_partial when opts is
 * given), its rows are copied, its tables are committed, and
 *     P_{k+1} = P_k without the consumed prefix, followed by the blocks wave k reclaimed
 * (reclaim order); wave k+1 plans on the committed tables of wave k with the same keep mask.
 * Exactly num_waves waves are enqueued (plan + copy + commit each, all on the given stream, so a
 * wave's copies finish before the next wave writes into the blocks they read); a wave that admits
 * nothing moves nothing.  Capturable like vtoken_plan / vtoken_repack.
 *
 * Ordering contract: unlike vtoken_plan + vtoken_repack, waves after the first overwrite blocks
 * that the INPUT tables still reference.  No reader of the old tables may run concurrently: order
 * the call after the last consumer of the old layout (the paper launches relocation after the
 * step's forward has returned, Sec. 3.3.4), and make consumers of the new tables wait on an event
 * recorded behind it. */
typedef struct {                   /* all DEVICE pointers, written by vtoken_repack_waves */
    int32_t *new_bt_offsets;       /* [R+1] block tables after the last wave */
    int32_t *new_bt_blocks;        /* capacity max_table_blocks */
    int32_t *new_tt_slots;         /* [T] token table after the last wave */
    int32_t *req_status;           /* [R] VTOKEN_REPACKED when some wave admitted the request, else its
                                      status in the last wave */
    int32_t *req_wave;             /* [R] last wave that admitted the request, -1 = none */
    int32_t *req_append_pos;       /* [R] or NULL: position in the request's final block list behind the tokens
                                      that wave moved ((blocks - ceil(moved / S)) * S + moved with that wave's
                                      figures), -1 = none; pass it to vtoken_apply_moves */
    int32_t *free_out;             /* [free_capacity] the pool after the last wave */
    int32_t *num_free_out;         /* device scalar */
    vtoken_counts *wave_counts;    /* [num_waves] counts of every wave (flags of its copy included) */
    int32_t free_capacity;         /* entries of free_out; num_free + total block-table entries always
                                      suffices; must not exceed the context's max_free_blocks
                                      (VTOKEN_ECAPACITY); a pool that outgrows it is truncated and
                                      VTOKEN_FLAG_CAPACITY is raised */
    void *workspace;               /* DEVICE scratch, 16-byte aligned, owned by the caller */
    int64_t workspace_bytes;       /* >= vtoken_waves_workspace_bytes (VTOKEN_ECAPACITY otherwise) */
    int32_t *released_blocks;      /* capacity max_table_blocks: references to shared blocks dropped by the waves'
                                      copy-on-write detaches, wave after wave (wave_counts[k].num_released each);
                                      needed when opts has a detach threshold, may be NULL otherwise */
    int32_t *num_released;         /* device scalar or NULL: entries of released_blocks after the last wave */
} vtoken_waves_out;

/* Bytes of workspace vtoken_repack_waves needs for this context and free_capacity. */
int64_t vtoken_waves_workspace_bytes(const vtoken_ctx *ctx, int32_t free_capacity);

/* in: as for vtoken_plan (read-only); opts: NULL = whole-request planner; num_waves >= 1. */
int vtoken_repack_waves(vtoken_ctx *ctx, const vtoken_plan_in *in, const vtoken_partial_opts *opts,
                        int32_t num_waves, const vtoken_waves_out *out, void *cuda_stream);

/* ---- Token-table runtime on the device (Sec. 3.2 interfaces, Sec. 3.4 slot mapping) ----------
 * For callers that keep the token tables resident on the GPU between decode steps.  Layout: the
 * table of request r occupies tt_slots / keep [tt_offsets[r] .. tt_offsets[r+1]) -- that range is
 * its CAPACITY; tt_len[r] entries are registered and the rest hold slot -1 / keep 0, which
 * vtoken_plan, vtoken_gather_logical and vtoken_build_slot_mapping treat as not live, so the same
 * buffers feed them unchanged.  phys_len[r] = slots already used in the request's block list
 * (where the next token is written).  All pointers DEVICE; every call only enqueues kernels on
 * the stream (capturable); problems found on the device raise VTOKEN_FLAG_* bits in the context's
 * counts (vtoken_read_counts). */

/* evict_token (Sec. 3.2) for a batch: keep[tt_offsets[req] + tok] = 0 for the first *num_victims
 * (device scalar, <= max_victims) pairs.  Metadata only: no KV byte moves, the slot stays until
 * a repack.  A victim outside [0, R) x [0, tt_len[req]) is skipped (VTOKEN_FLAG_BAD_VICTIM). */
int vtoken_evict_tokens(vtoken_ctx *ctx, const int32_t *num_victims, int32_t max_victims,
                        const int32_t *victim_req, const int32_t *victim_tok, const int32_t *num_requests,
                        const int32_t *tt_offsets, const int32_t *tt_len, uint8_t *keep, void *cuda_stream);

/* sync_new_tokens (Sec. 3.2) for a batch: request r grows from tt_len[r] to new_len[r] registered
 * tokens (unchanged when new_len[r] <= tt_len[r]).  New tokens get sequential logical ids; the
 * i-th new one sits at position p = phys_len[r] + i of the block list bt_blocks[bt_offsets[r] ..):
 * slot = block[p / S] * S + p % S, keep = 1.  Growth stops at the table capacity or at the end of
 * the block list (VTOKEN_FLAG_APPEND_STOPPED).  A token whose block id lies outside [0, num_blocks)
 * is registered without a physical copy (slot -1, keep 0; VTOKEN_FLAG_BAD_BLOCK).  Updates tt_len
 * and phys_len. */
int vtoken_sync_new_tokens(vtoken_ctx *ctx, const int32_t *num_requests, const int32_t *tt_offsets,
                           int32_t *tt_slots, uint8_t *keep, int32_t *tt_len, int32_t *phys_len,
                           const int32_t *bt_offsets, const int32_t *bt_blocks, const int32_t *new_len,
                           void *cuda_stream);

/* The same two interfaces with the per-block liveness metadata kept current (Sec. 3.3.1: per-block
 * liveness lets the planner find under-utilised blocks without scanning the table).  n_b: DEVICE
 * int32 [num_blocks] as vtoken_block_liveness computes it; live_total: DEVICE int64 scalar = sum of
 * n_b, or NULL (F = 1 - live_total / (allocated blocks * S)).  An eviction takes one live token
 * from the block of its slot, but only if this call is what deactivates the token: a token named
 * twice in the batch, or already evicted, counts once (the keep byte is cleared with an atomic on
 * the aligned 32-bit word that holds it, so keep must be 4-byte aligned and allocated in multiples
 * of four bytes).  Every newly registered token adds one to the block that holds it.  After a
 * repack recount with vtoken_block_liveness: relocation is a structural change. */
int vtoken_evict_tokens_counted(vtoken_ctx *ctx, const int32_t *num_victims, int32_t max_victims,
                                const int32_t *victim_req, const int32_t *victim_tok, const int32_t *num_requests,
                                const int32_t *tt_offsets, const int32_t *tt_len, const int32_t *tt_slots,
                                uint8_t *keep, int32_t *n_b, int64_t *live_total, void *cuda_stream);
int vtoken_sync_new_tokens_counted(vtoken_ctx *ctx, const int32_t *num_requests, const int32_t *tt_offsets,
                                   int32_t *tt_slots, uint8_t *keep, int32_t *tt_len, int32_t *phys_len,
                                   const int32_t *bt_offsets, const int32_t *bt_blocks, const int32_t *new_len,
                                   int32_t *n_b, int64_t *live_total, void *cuda_stream);

/* Slot mapping (Sec. 3.4: slot = token_table[token].block_id * S + offset, looked up once per token
 * at input preparation): the slots of the active tokens (slot >= 0, and keep != 0 when keep is
 * given) of the selected requests, request order then token-id order, written densely to
 * out_slots[out_capacity]; out_token_ids (may be NULL) receives their logical ids; out_offsets[R+1]
 * the first entry of each request.  Entries beyond out_capacity are dropped
 * (VTOKEN_FLAG_GATHER_OVERFLOW).  The buffers are stable, only their contents change between
 * calls -- the property the paper relies on for CUDA-Graph replay.  Shares the scratch of the gather
 * family (see vtoken_gather_logical): it may overlap a plan / repack on another stream. */
int vtoken_build_slot_mapping(vtoken_ctx *ctx, const int32_t *num_requests, const int32_t *tt_offsets,
                              const int32_t *tt_slots, const uint8_t *keep, const uint8_t *select,
                              int32_t *out_slots, int32_t *out_token_ids, int64_t out_capacity,
                              int32_t *out_offsets, void *cuda_stream);

/* apply_moves (Sec. 3.2; invariant I2): commit of a plan after its repack event.  Every entry takes
 * its slot from new_tt_slots (the source entry is cleared by the same write) and keep becomes
 * (slot >= 0).  For requests with status VTOKEN_REPACKED the append position moves behind the
 * tokens the repack moved: the request's block list is now the blocks that stayed followed by the
 * destination blocks, so  phys_len[r] = (blocks - ceil(moved / S)) * S + moved  with blocks from
 * new_bt_offsets and moved = entries whose slot changed.  new_bt_offsets may be NULL: phys_len[r]
 * is then the number of entries that own a slot -- the same value after vtoken_plan (nothing
 * stays), wrong after a partial plan.  append_pos (may be NULL; req_append_pos of
 * vtoken_repack_waves) overrides both: phys_len[r] = append_pos[r] -- after several waves a partly
 * filled destination block of an early wave may sit in the middle of the list, and only the
 * wave-by-wave bookkeeping knows where the list ends.  phys_len may be NULL.  The block tables are
 * the caller's: it adopts new_bt_* and returns freed blocks itself. */
int vtoken_apply_moves(vtoken_ctx *ctx, const int32_t *num_requests, const int32_t *tt_offsets,
                       int32_t *tt_slots, uint8_t *keep, int32_t *phys_len, const int32_t *new_tt_slots,
                       const int32_t *req_status, const int32_t *new_bt_offsets, const int32_t *append_pos,
                       void *cuda_stream);

/* Cached slot-translation arrays (Sec. 3.2, last paragraph; Sec. 4): per request the slots (and
 * ids) of its active tokens in token-id order, kept on the device between decode steps and
 * refreshed only after structural changes -- appended to when the sequence merely grew, rebuilt
 * after an eviction or a relocation.  Layout: the cache of request r occupies cache_slots /
 * cache_ids [tt_offsets[r] ..) (the capacity of its token table); cache_len[r] entries are valid
 * and cover the first cache_seen[r] registered tokens; dirty[r] != 0 asks for a rebuild.  A fresh
 * cache is cache_len = cache_seen = 0 (dirty anything).  All pointers DEVICE.
 *
 * vtoken_slot_cache_mark: dirty[r] = 1 for the request of each of the first *num_victims
 * (<= max_victims) entries of victim_req (requests outside [0, R) are skipped) and for every request
 * whose req_status is VTOKEN_REPACKED.  victim_req / num_victims may be NULL (max_victims 0), and
 * so may req_status: call it with the victims after vtoken_evict_tokens and with the plan's
 * statuses after vtoken_apply_moves.
 *
 * vtoken_slot_cache_update, per request: dirty -> rebuild from the first tt_len[r] entries, clear
 * the mark; else tt_len[r] > cache_seen[r] -> append the active ones among the new entries; else
 * nothing is read or written.  cache_ids may be NULL.  stats: DEVICE int32[2] or NULL, receives
 * {requests rebuilt, requests appended to}. */
int vtoken_slot_cache_mark(vtoken_ctx *ctx, uint8_t *dirty, const int32_t *num_victims, int32_t max_victims,
                           const int32_t *victim_req, const int32_t *req_status, const int32_t *num_requests,
                           void *cuda_stream);
int vtoken_slot_cache_update(vtoken_ctx *ctx, const int32_t *num_requests, const int32_t *tt_offsets,
                             const int32_t *tt_slots, const uint8_t *keep, const int32_t *tt_len, uint8_t *dirty,
                             int32_t *cache_slots, int32_t *cache_ids, int32_t *cache_len, int32_t *cache_seen,
                             int32_t *stats, void *cuda_stream);

/* Host-table front end.  The paper keeps the canonical token table on the CPU (Sec. 3.2);
 * this entry point serves such a caller: all tables are HOST memory (pinned for speed), the
 * pools stay on the device.  Copies the inputs to device staging owned by the context, runs
 * vtoken_plan and vtoken_repack, copies every output back and synchronises the stream. */
typedef struct {                   /* all HOST pointers */
    int32_t num_requests;
    const int32_t *bt_offsets, *bt_blocks, *tt_offsets, *tt_slots;
    const uint8_t *keep, *select;  /* select may be NULL */
    uint32_t thr_num, thr_den;
    const int32_t *free_blocks;
    int32_t num_free;
    int32_t *new_bt_offsets;       /* [R+1] */
    int32_t *new_bt_blocks;        /* [bt_offsets[R]] */
    int32_t *new_tt_slots;         /* [tt_offsets[R]] */
    int32_t *freed_blocks;         /* [bt_offsets[R]] */
    int32_t *req_status;           /* [R] */
    vtoken_counts *counts;
    int32_t *released_blocks;      /* [bt_offsets[R]] or NULL: references dropped by a copy-on-write detach
                                      (vtoken_repack_host_partial with a detach threshold; counts->num_released) */
} vtoken_host_tables;
int vtoken_repack_host(vtoken_ctx *ctx, const vtoken_host_tables *tables, void *cuda_stream);

/* The same front end with the partial planner (vtoken_plan_partial): opts as there, except that
 * opts->protect, when given, is a HOST array of num_blocks bytes (copied to the device with the
 * tables).  opts must not be NULL.  With a detach threshold tables->released_blocks must be given
 * (VTOKEN_EINVAL otherwise). */
int vtoken_repack_host_partial(vtoken_ctx *ctx, const vtoken_host_tables *tables, const vtoken_partial_opts *opts,
                               void *cuda_stream);

/* Logical gather for callers that cannot allocate device memory.  (The paper has no
 * counterpart: this is a packaging variant of vtoken_gather_logical, same result.)
 *
 * Who needs it: a serving engine that has handed nearly all of HBM to its KV pool (the paper
 * runs at gpu_mem_util = 0.90) has nothing left for vtoken_create's scratch and may see
 * cudaMalloc fail; code on a latency-critical step cannot afford cudaMalloc either, because
 * it synchronises the whole device; and some embedders simply forbid allocator calls outside
 * their own pool.  This entry point takes no context and calls no cudaMalloc, cudaFree or
 * other allocating routine.  Its scratch is a fixed array inside the library's device image
 * (about 1 MiB per GPU that loads the library, held until the process exits), which bounds
 * the problem size:
 *     max_requests        <= 4096
 *     out_capacity_tokens <= 262144
 * Larger values return VTOKEN_ECAPACITY and enqueue nothing.
 *
 * Arguments: the pool geometry that vtoken_create would take (pools DEVICE, 16-byte aligned,
 * row_bytes a multiple of 16, layer_stride_bytes 0 => num_blocks*block_size*row_bytes), then
 * exactly the arguments of vtoken_gather_logical; max_requests bounds *num_requests and fixes
 * the grid.  error_flags: DEVICE uint32 or NULL, receives the VTOKEN_FLAG_* bits of this call
 * (bad slot, gather overflow), written on the stream.  The caller owns inputs and outputs.
 *
 * The first call on each device looks up the device address of the scratch array (that
 * device must be current); make that first call before starting any stream capture.
 * All calls on a device share the one scratch array: the call clears what it needs cleared,
 * but two calls whose kernels overlap on the GPU (different streams without an event between
 * them) race on it and corrupt each other's output.  Order them on one stream or by events. */
int vtoken_gather_logical_noalloc(const void *k_pool, const void *v_pool, int32_t num_layers,
                                  int32_t num_blocks, int32_t block_size, int64_t row_bytes,
                                  int64_t layer_stride_bytes, const int32_t *num_requests,
                                  int32_t max_requests, const int32_t *tt_offsets, const int32_t *tt_slots,
                                  const uint8_t *keep, const uint8_t *select, int32_t layer_begin,
                                  int32_t layer_end, void *out_k, void *out_v, int64_t out_capacity_tokens,
                                  int32_t *out_offsets, uint32_t *error_flags, void *cuda_stream);

/* Input-precondition checker (a debugging aid: the fast path assumes these and does not check
 * them; invariant I2 -- unique mapping -- is bit 128).  Writes to out_bits (DEVICE uint32) the
 * set of violated preconditions of the planner inputs in `in` (keep, select and the threshold
 * are not consulted: an evicted token still owns its slot until a repack):
 *   1   CSR offsets not monotone (only this bit is reported then)
 *   2   a block-table id outside [0, num_blocks)
 *   4   a block id held by more than one block-table entry
 *   8   a free-list id outside [0, num_blocks)
 *   16  a free-list id listed twice, or also held by a block table
 *   32  a slot >= num_blocks * block_size
 *   64  a slot whose block is held by no block table, or by exactly one request that is not the
 *       slot's request (blocks held by several requests are outside this check)
 *   128 a slot referenced by more than one token-table entry
 * protect (DEVICE [num_blocks] or NULL): blocks marked there may sit in several tables and their
 * slots may be mapped by every sharer (shared prefix): bits 4 and 128 are not raised for them.
 * Uses the context's planner scratch (do not overlap with a plan in flight).  Capturable. */
int vtoken_check_tables(vtoken_ctx *ctx, const vtoken_plan_in *in, const uint8_t *protect, uint32_t *out_bits,
                        void *cuda_stream);

/* Diagnostics. */
const char *vtoken_strerror(int code);
int vtoken_last_cuda_error(const vtoken_ctx *ctx);       /* cudaError_t of the last VTOKEN_ECUDA */
int vtoken_copy_grid(const vtoken_ctx *ctx, int32_t *ctas, int32_t *threads, int32_t *smem_bytes,
                     int32_t *variant);                   /* launch shape of the copy kernel */
int64_t vtoken_scratch_bytes(const vtoken_ctx *ctx);      /* device scratch held by the context */
int vtoken_plan_form(const vtoken_ctx *ctx);              /* planner form vtoken_plan uses for this context's
                                                             capacities: 1 or 2 as vtoken_config.plan_variant */
int vtoken_checked_build(void);                           /* 1: this library was compiled with VTOKEN_CHECKED */
/* Self-test of the checked build: one thread reads element `index` of a context scratch array of
 * max_requests int32 through the same checked accessor every kernel of that build uses, and stores what
 * it read to *out_value (DEVICE).  Inside the array: the element.  Outside: nothing is read there,
 * VTOKEN_FLAG_CHECK_FAILED is raised (vtoken_read_counts), nothing faults.  The production library
 * returns VTOKEN_EINVAL. */
int vtoken_debug_probe(vtoken_ctx *ctx, int64_t index, int32_t *out_value, void *cuda_stream);

#ifdef __cplusplus
}
#endif
#endif
