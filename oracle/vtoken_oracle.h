/*
 * CPU oracle for the vToken repack path.  TEST INFRASTRUCTURE ONLY.
 *
 * A plain, slow, single-pass restatement of what the repack computes, written from the
 * paper's description so that it can be checked against the paper by eye.  It shares no
 * code with the CUDA library and must never be called from the product path: only the
 * tests, the smoke check and the benchmark's CPU-baseline leg use it.
 *
 * What it states (paper passages):
 *   - live footprint, ceil(T_live / S) destinations, positive-gain gate  (Sec. 3.3.3, invariant I4)
 *   - destinations taken from the free pool, plan deferred when short    (Sec. 3.3.2, 3.3.3)
 *   - move list in logical order, each destination filled completely     (Sec. 3.3.3)
 *   - slot = block_id * S + offset                                        (Sec. 3.4, slot-mapping equation)
 *   - token-table update clears the source and writes the destination    (Sec. 3.2 apply_moves, invariant I2)
 *   - sources freed after the packed layout is committed                 (Sec. 3.3.4)
 *   - logical view = K/V rows of active tokens in token-id order         (invariant I1, Sec. 5 relocation check)
 *   - intra-block waste ratio F                                           (Sec. 2.3.1)
 *
 * Readings fixed where the paper is silent (same readings bind the CUDA library):
 *   whole-request compaction; requests planned in ascending index; admission is the longest
 *   prefix of candidates whose cumulative demand fits the free list, every later candidate
 *   deferred; destinations are consecutive entries from the front of the caller's free list;
 *   the reclaimed list is admitted requests ascending, each old block table in order; dead
 *   tokens map to -1 in every request; the canonical orders are conventions ("parity
 *   unpinned" by the paper itself -- the semantic checker vto_check_semantics accepts any
 *   valid permutation and guards against a convention hiding a real defect).
 *
 * All pointers are HOST memory owned by the caller.  Functions return 0 on success, a
 * negative VTO_E* code on a malformed argument, and never abort.
 */
#ifndef VTOKEN_ORACLE_H
#define VTOKEN_ORACLE_H
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

enum { VTO_OK = 0, VTO_EINVAL = -1, VTO_EPRECOND = -2 };
enum { VTO_NOT_SELECTED = 0, VTO_REPACKED = 1, VTO_NO_GAIN = 2, VTO_DEFERRED_NO_FREE = 3 };

typedef struct {
    int32_t num_moves, num_dst_blocks, num_freed, num_free_consumed, num_admitted, num_deferred;
    int32_t num_released;   /* references to shared blocks dropped by a copy-on-write detach (vto_plan_partial) */
} vto_counts;

/* Relocation planning + table rewrite for R requests.
 * Inputs: CSR block tables (bt_offsets[R+1], bt_blocks), CSR token tables (tt_offsets[R+1],
 * tt_slots: slot or -1), keep mask (0 = evicted), optional select[R] (NULL = all), live-fraction
 * threshold thr_num/thr_den (thr_den == 0: none; candidate iff n*thr_den < thr_num*nb*S),
 * free list free_blocks[num_free].
 * Outputs (caller-sized): new_bt_offsets[R+1], new_bt_blocks[<= total old blocks],
 * new_tt_slots[T], freed_blocks[<= total old blocks], req_status[R],
 * move_src/move_dst[<= T] (slot pairs, plan order), counts. */
int vto_plan(int32_t R, int32_t S,
             const int32_t *bt_offsets, const int32_t *bt_blocks,
             const int32_t *tt_offsets, const int32_t *tt_slots, const uint8_t *keep,
             const uint8_t *select, uint32_t thr_num, uint32_t thr_den,
             const int32_t *free_blocks, int32_t num_free,
             int32_t *new_bt_offsets, int32_t *new_bt_blocks, int32_t *new_tt_slots,
             int32_t *freed_blocks, int32_t *req_status,
             int32_t *move_src, int32_t *move_dst, vto_counts *counts);

/* Apply a move list to ONE (K|V, layer) slab of num_slots rows of row_bytes bytes, in place:
 * row[dst] = row[src] for every move, nothing else changes. */
int vto_apply_moves_slab(uint8_t *slab, int64_t num_slots, int64_t row_bytes,
                         const int32_t *move_src, const int32_t *move_dst, int32_t num_moves);

/* Apply a move list to whole K and V pools laid out [L][num_slots][row_bytes] with the given
 * layer stride, every layer, K then V.  threads > 1 spreads the 2L independent slabs over
 * that many OpenMP threads (when built with OpenMP; otherwise runs on one). */
int vto_apply_moves_pools(uint8_t *k_pool, uint8_t *v_pool, int32_t L, int64_t layer_stride_bytes,
                          int64_t num_slots, int64_t row_bytes,
                          const int32_t *move_src, const int32_t *move_dst, int32_t num_moves,
                          int32_t threads);

/* Logical view of one request in one slab: rows of tokens t with tt_slots[t] >= 0 and
 * (keep == NULL or keep[t] != 0), ascending t, concatenated into out.  Returns the row count
 * (>= 0) or a negative error. */
int64_t vto_gather_logical(const uint8_t *slab, int64_t num_slots, int64_t row_bytes,
                           const int32_t *tt_slots, const uint8_t *keep, int32_t len,
                           uint8_t *out, int64_t out_capacity_rows);

/* Input preconditions: every live slot in [0, NB*S) and inside a block of the request's own
 * block table; no slot referenced by two tokens (I2); block ids unique across block tables
 * and in range; free list in range, duplicate-free and disjoint from the block tables.
 * Returns VTO_OK or VTO_EPRECOND; *first_bad (optional) gets a small code naming the check. */
int vto_validate(int32_t R, int32_t S, int32_t NB,
                 const int32_t *bt_offsets, const int32_t *bt_blocks,
                 const int32_t *tt_offsets, const int32_t *tt_slots, const uint8_t *keep,
                 const int32_t *free_blocks, int32_t num_free, int32_t *first_bad);

/* The same preconditions, every violated one reported as a bit (evaluation order does not
 * matter: each bit is defined by counting, so a parallel checker gives the same answer):
 *   1   CSR offsets not monotone (block tables or token tables)
 *   2   a block-table id outside [0, NB)
 *   4   a block id held by more than one block-table entry
 *   8   a free-list id outside [0, NB)
 *   16  a free-list id listed twice, or also held by a block table
 *   32  a slot >= NB*S
 *   64  a slot (>= 0, in range) whose block is held by no block table, or by exactly one request
 *       that is not the slot's request (blocks held by several requests are outside this check)
 *   128 a slot (>= 0, in range) referenced by more than one token-table entry (I2)
 * Entries with slot < 0 are ignored; keep is not consulted (an evicted token still owns its slot
 * until a repack).  protect (may be NULL): blocks marked there may sit in several tables
 * (shared prefix) and their slots are mapped by every sharer, so bits 4 and 128 are not raised
 * for them. */
int vto_check_tables(int32_t R, int32_t S, int32_t NB,
                     const int32_t *bt_offsets, const int32_t *bt_blocks,
                     const int32_t *tt_offsets, const int32_t *tt_slots,
                     const int32_t *free_blocks, int32_t num_free, const uint8_t *protect, uint32_t *bits);

/* Order-free check of a plan result against the inputs: statuses follow the admission rule,
 * admitted requests got ceil(n/S) distinct blocks of the consumed free prefix and their live
 * tokens fill those blocks completely in logical order, the reclaimed set equals the admitted
 * requests' old blocks, other requests are unchanged, dead tokens are -1.  Returns VTO_OK,
 * VTO_EPRECOND (*first_bad names the check) or VTO_EINVAL. */
int vto_check_semantics(int32_t R, int32_t S,
                        const int32_t *bt_offsets, const int32_t *bt_blocks,
                        const int32_t *tt_offsets, const int32_t *tt_slots, const uint8_t *keep,
                        const uint8_t *select, uint32_t thr_num, uint32_t thr_den,
                        const int32_t *free_blocks, int32_t num_free,
                        const int32_t *new_bt_offsets, const int32_t *new_bt_blocks,
                        const int32_t *new_tt_slots, const int32_t *freed_blocks,
                        int32_t num_freed, int32_t num_free_consumed,
                        const int32_t *req_status, int32_t *first_bad);

/* Intra-block waste ratio F = 1 - sum(n_b) / (N * S) over the N allocated blocks, with n_b
 * the live tokens per block (Sec. 2.3.1).  live = slot >= 0 and keep != 0 (keep NULL: slot >= 0). */
double vto_waste_ratio(int32_t S, int64_t num_allocated_blocks,
                       const int32_t *tt_slots, const uint8_t *keep, int64_t T);

/* ---- token-table runtime (Sec. 3.2 interfaces, Sec. 3.4 slot mapping) -------------------------
 * The token table of request r occupies tt_slots[tt_offsets[r] .. tt_offsets[r+1]) -- that range
 * is its CAPACITY; tt_len[r] entries are registered, the rest hold -1 / keep 0.  phys_len[r] is the
 * number of slots already used in the request's block list (the append position). */

/* evict_token for a batch: keep[tt_offsets[req] + tok] = 0.  A victim with req outside [0, R) or
 * tok outside [0, tt_len[req]) is skipped and counted in *num_bad. */
int vto_evict_tokens(int32_t R, const int32_t *tt_offsets, const int32_t *tt_len, uint8_t *keep,
                     const int32_t *victim_req, const int32_t *victim_tok, int32_t num_victims,
                     int32_t *num_bad);

/* sync_new_tokens for a batch: request r grows from tt_len[r] to new_len[r] registered tokens (no
 * change when new_len[r] <= tt_len[r]).  New tokens get sequential logical ids; the i-th new token
 * sits at position p = phys_len[r] + i of the request's block list:
 * slot = bt_blocks[bt_offsets[r] + p / S] * S + p % S, keep = 1.  A token beyond the table capacity
 * or beyond the block list is not registered: the request stops growing there and is counted in
 * *num_bad.  Updates tt_len and phys_len. */
int vto_sync_new_tokens(int32_t R, int32_t S, const int32_t *tt_offsets, int32_t *tt_slots, uint8_t *keep,
                        int32_t *tt_len, int32_t *phys_len, const int32_t *bt_offsets,
                        const int32_t *bt_blocks, const int32_t *new_len, int32_t *num_bad);

/* The same two interfaces with the per-block liveness metadata kept current (Sec. 3.3.1: per-block
 * liveness n_b lets the planner find under-utilised blocks without scanning the table): n_b[NB] as
 * vto_block_liveness computes it, *live_total (optional) = sum of n_b.  An eviction takes one live
 * token from the block of its slot, but only if this call is what deactivates the token (a token
 * named twice, or already evicted, counts once); every newly registered token adds one to the
 * block that holds it.  After a repack the counters are recomputed (vto_block_liveness). */
int vto_evict_tokens_counted(int32_t R, int32_t S, int32_t NB, const int32_t *tt_offsets, const int32_t *tt_len,
                             const int32_t *tt_slots, uint8_t *keep, const int32_t *victim_req,
                             const int32_t *victim_tok, int32_t num_victims, int32_t *n_b, int64_t *live_total,
                             int32_t *num_bad);
int vto_sync_new_tokens_counted(int32_t R, int32_t S, int32_t NB, const int32_t *tt_offsets, int32_t *tt_slots,
                                uint8_t *keep, int32_t *tt_len, int32_t *phys_len, const int32_t *bt_offsets,
                                const int32_t *bt_blocks, const int32_t *new_len, int32_t *n_b, int64_t *live_total,
                                int32_t *num_bad);

/* Slot mapping of the active tokens (slot = token_table[token].block * S + offset, Sec. 3.4): for each
 * selected request, in request order, the slots (and logical ids) of its tokens with slot >= 0 and
 * keep != 0 (keep NULL: slot >= 0) in ascending token id.  out_offsets[R+1] = first entry of each
 * request.  Returns the entry count or VTO_EINVAL when it exceeds capacity. */
int64_t vto_build_slot_mapping(int32_t R, const int32_t *tt_offsets, const int32_t *tt_slots,
                               const uint8_t *keep, const uint8_t *select, int32_t *out_slots,
                               int32_t *out_token_ids, int32_t *out_offsets, int64_t capacity);

/* apply_moves / commit of a repack: every entry takes its new slot, liveness follows it (an entry
 * without a slot is dead), and a repacked request appends behind the tokens the repack moved: its
 * block list is now the blocks that stayed followed by the destination blocks, so for requests
 * with status VTO_REPACKED  phys_len[r] = (blocks - ceil(moved / S)) * S + moved, with blocks from
 * new_bt_offsets and moved = entries whose slot changed.  new_bt_offsets == NULL: phys_len[r] =
 * number of entries with a slot (the same value after a whole-request plan, where nothing stays).
 * append_pos != NULL (the per-request positions a repack in waves reports): phys_len[r] =
 * append_pos[r] -- after several waves a partly filled destination block of an early wave may sit
 * in the middle of the list, and only the wave-by-wave bookkeeping knows where the list ends. */
int vto_apply_moves(int32_t R, int32_t S, const int32_t *tt_offsets, int32_t *tt_slots, uint8_t *keep,
                    int32_t *phys_len, const int32_t *new_tt_slots, const int32_t *req_status,
                    const int32_t *new_bt_offsets, const int32_t *append_pos);

/* ---- cached slot-translation arrays (Sec. 3.2, last paragraph; Sec. 4) -------------------------
 * The worker keeps, per request, the slots of its active tokens in token-id order -- the array a
 * decode step translates through -- and refreshes it only after structural changes: growth of a
 * sequence at its end is taken in by appending the new entries, and only an eviction or a
 * relocation of the request makes the array be rebuilt.
 * Layout: the cache of request r lives in cache_slots / cache_ids [tt_offsets[r] ..) (same capacity
 * as its token table); cache_len[r] entries are valid and cover the first cache_seen[r] registered
 * tokens.
 * vto_slot_cache_mark: dirty[r] = 1 for the request of every victim (requests outside [0, R) are
 * skipped) and for every request with status VTO_REPACKED; either list may be NULL.
 * vto_slot_cache_update, per request: dirty -> rebuild from the first tt_len[r] entries and clear
 * the mark; else tt_len[r] > cache_seen[r] -> append the active ones among the new entries; else
 * leave everything as it is.  *num_rebuilt / *num_appended (optional) count the requests. */
int vto_slot_cache_mark(int32_t R, uint8_t *dirty, const int32_t *victim_req, int32_t num_victims,
                        const int32_t *req_status);
int vto_slot_cache_update(int32_t R, const int32_t *tt_offsets, const int32_t *tt_slots, const uint8_t *keep,
                          const int32_t *tt_len, uint8_t *dirty, int32_t *cache_slots, int32_t *cache_ids,
                          int32_t *cache_len, int32_t *cache_seen, int32_t *num_rebuilt, int32_t *num_appended);

/* ---- eligibility metadata and partial plans (Sec. 3.3.1 - 3.3.3) ------------------------------
 * Per-block liveness n_b = live tokens stored in physical block b (over all requests), the
 * histogram hist[k] = number of ALLOCATED blocks (entries of the block tables) with n_b == k for
 * k = 0..S, the total live count and the allocated-block count N, from which
 * F = 1 - live_total / (N * S) (Sec. 2.3.1).  n_b has NB entries, hist has S + 1. */
int vto_block_liveness(int32_t R, int32_t S, int32_t NB, const int32_t *bt_offsets, const int32_t *bt_blocks,
                       const int32_t *tt_offsets, const int32_t *tt_slots, const uint8_t *keep,
                       int32_t *n_b, int64_t *hist, int64_t *live_total, int64_t *num_allocated);

typedef struct {
    const uint8_t *protect;       /* [NB] or NULL: non-zero = the block must stay (shared prefix, I4) */
    uint32_t util_num, util_den;  /* a block is a source iff n_b * util_den < util_num * S; util_den == 0: every
                                     unprotected block (whole-request compaction) */
    int32_t max_source_blocks;    /* B: at most this many sources per request, first in table order; 0 = no bound */
    uint32_t theta_num, theta_den;/* plan only when F > theta_num / theta_den; theta_den == 0: always */
    uint32_t detach_num, detach_den; /* copy-on-write detach: a request leaves ALL its protected blocks when its own
                                     live tokens in them fill less than detach_num / detach_den of those blocks;
                                     detach_den == 0: never (protected blocks always stay) */
    uint32_t detach_rule;         /* what the detach threshold is applied to.  0: the request's protected blocks as a
                                     whole (above).  1: every protected block by itself, counting the request's own
                                     live tokens in it: it leaves b when n_rb * detach_den < detach_num * S and stays
                                     in the others.  2: every protected block by itself, counting the live tokens of
                                     ALL holders (n_b): every holder leaves b when n_b * detach_den < detach_num * S */
} vto_partial_opts;

/* Relocation planning that evacuates only low-utilisation source blocks (Sec. 3.3.3): the planner
 * picks the eligible, poorly filled blocks of a request as sources, counts the live tokens T_live
 * stored in them, needs ceil(T_live / S) destinations and admits the plan only when the sources
 * release more blocks than that.  Everything else as vto_plan, except:
 *   - only live tokens stored in source blocks move (logical order, destinations filled completely);
 *     live tokens in the other blocks keep their slots; dead tokens become -1;
 *   - new block table of a repacked request = its non-source blocks in old order, then its
 *     destination blocks; the reclaimed list receives its source blocks in old order;
 *   - when the global trigger F > theta does not hold, every request is VTO_NOT_SELECTED.
 * With util_den == 0, protect == NULL, B == 0 and theta_den == 0 the result equals vto_plan's.
 * NB = number of physical blocks (size of protect and of the internal n_b).
 *
 * Copy-on-write detach (the paper's outlook for shared-prefix blocks, Sec. 5 on prefix caching and
 * Sec. 6: copy a request's tokens out of shared blocks once the blocks that brings back outweigh
 * the copy): with detach_den != 0, a request whose own live tokens occupy less than
 * detach_num / detach_den of its protected blocks (n_shared * den < num * ns_shared * S) treats all
 * of them as sources too: its live tokens there are COPIED to its destinations with the rest (the
 * shared blocks keep their bytes for the other holders), the blocks leave its table, and they are
 * listed in released_blocks (references dropped; the caller's reference counts decide when such a
 * block is free) instead of freed_blocks.  B bounds the unprotected sources only.  The gain gate
 * is unchanged: destinations < sources, counted in the request's own table.
 * With detach_rule 1 the same threshold is applied block by block: the request leaves exactly
 * those protected blocks of its table in which its own live tokens fill less than the fraction
 * (n_rb * den < num * S; the other holders' tokens do not count), and keeps the others in place,
 * at the head of its new table with its other kept blocks.
 * With detach_rule 2 the block is judged by everything stored in it: n_b, the live tokens of all
 * its holders (one count per referencing token-table entry).  Every holder reaches the same verdict
 * on the same number, so a block is left by all the planned holders or by none: the copies its
 * holders make (n_b tokens in all) cost less than the block they give back exactly when n_b < S,
 * which is the threshold 1/1 -- the paper's condition for copy-on-write (the reclaimed capacity
 * must outweigh the extra copy) as a test the planner can make without knowing who else holds
 * the block. */
int vto_plan_partial(int32_t R, int32_t S, int32_t NB,
                     const int32_t *bt_offsets, const int32_t *bt_blocks,
                     const int32_t *tt_offsets, const int32_t *tt_slots, const uint8_t *keep,
                     const uint8_t *select, uint32_t thr_num, uint32_t thr_den,
                     const int32_t *free_blocks, int32_t num_free, const vto_partial_opts *opts,
                     int32_t *new_bt_offsets, int32_t *new_bt_blocks, int32_t *new_tt_slots,
                     int32_t *freed_blocks, int32_t *req_status,
                     int32_t *move_src, int32_t *move_dst, vto_counts *counts, int32_t *released_blocks);

/* ---- online relocation check (Sec. 5, "Relocation Correctness") ---------------------------------
 * The paper hashes the ordered retained token ids together with their K/V contents before and
 * after a relocation.  It does not name the hash; this build fixes one that can be evaluated in
 * any order (a sum of per-word terms, each bound to its position): for a request whose active
 * tokens are t_0 < t_1 < ... (rank i, logical id t_i), over slabs s = 0 .. 2*(layer_end-layer_begin)-1
 * (K layers first, then V layers) and the 32-byte groups g of the token's row, each four 8-byte
 * little-endian words w_4g .. w_4g+3 (a row of 16 mod 32 bytes ends with a group of two words),
 *     key(i, s) = mix(((i * A + t_i) * B + s) * C),      x_j = w_j ^ (key(i, s) + j * D)
 *     a = x_4g + x_4g+2,   b = x_4g+1 + x_4g+3           (mod 2^64; absent words add nothing)
 *     digest    = sum over (i, s, g) of  low64(a * b) ^ high64(a * b)        mod 2^64
 * with a * b the full 128-bit product, mix = the splitmix64 finaliser and A, B, C, D the odd
 * constants in the source (one multiply-fold per 32 bytes: the check reads K/V at memory speed).
 * Every word is bound to its place by its own key; a lost, duplicated, reordered or altered token
 * changes the digest.  row_bytes must be a multiple of 16.
 * Pools are [L][num_slots][row_bytes] with layer_stride_bytes between layers (0 = dense). */
int vto_digest_logical(const uint8_t *k_pool, const uint8_t *v_pool, int64_t layer_stride_bytes, int64_t num_slots,
                       int64_t row_bytes, int32_t layer_begin, int32_t layer_end, const int32_t *tt_slots,
                       const uint8_t *keep, int32_t len, uint64_t *digest, int32_t *num_active);

/* ---- repack in waves: blocks reclaimed by one wave are destinations of the next ----------------
 * The paper returns source blocks to the free pool once the packed layout is committed
 * (Sec. 3.3.4) and defers plans that the headroom cannot serve (Sec. 3.3.2).  Run as a loop, the
 * two statements give a repack that needs only a small headroom: wave k plans against the pool
 * P_k (vto_plan, or vto_plan_partial when opts != NULL), its copies run, its tables are committed,
 * and   P_{k+1} = P_k without the consumed prefix, followed by the blocks wave k reclaimed
 * (reclaim order).  Wave k+1 plans on the committed tables of wave k with the same keep mask
 * (evicted entries are -1 from wave 0 on).  Exactly num_waves waves run; a wave that admits
 * nothing changes nothing.
 * Outputs: the tables after the last wave; req_status[r] = VTO_REPACKED when some wave admitted r,
 * else its status in the last wave; req_wave[r] = last wave that admitted r, -1 when none;
 * req_append_pos[r] (may be NULL) = position in r's final block list behind the tokens that wave
 * moved, (blocks - ceil(moved / S)) * S + moved with that wave's figures, -1 when none;
 * free_out[<= num_free + total old blocks] / *num_free_out = the pool after the last wave;
 * wave_counts[num_waves] = counts of every wave; move_src / move_dst = the move lists of all
 * waves back to back, wave k in [wave_move_offsets[k], wave_move_offsets[k+1]) -- they must be
 * applied in this order, because a later wave overwrites blocks an earlier wave has read.
 * released_blocks (capacity: total old blocks; may be NULL without a detach threshold) = the references to
 * shared blocks the waves' copy-on-write detaches dropped, wave after wave (wave_counts[k].num_released each).
 * Returns VTO_EINVAL when move_capacity is too small. */
int vto_plan_waves(int32_t R, int32_t S, int32_t NB,
                   const int32_t *bt_offsets, const int32_t *bt_blocks,
                   const int32_t *tt_offsets, const int32_t *tt_slots, const uint8_t *keep,
                   const uint8_t *select, uint32_t thr_num, uint32_t thr_den,
                   const int32_t *free_blocks, int32_t num_free, const vto_partial_opts *opts,
                   int32_t num_waves,
                   int32_t *new_bt_offsets, int32_t *new_bt_blocks, int32_t *new_tt_slots,
                   int32_t *req_status, int32_t *req_wave, int32_t *req_append_pos, int32_t *free_out,
                   int32_t *num_free_out, int32_t *move_src, int32_t *move_dst, int64_t move_capacity,
                   int64_t *wave_move_offsets, vto_counts *wave_counts, int32_t *released_blocks);

int vto_openmp_threads(void);   /* max OpenMP threads of this build, 1 when built without */

#ifdef __cplusplus
}
#endif
#endif
