/*
 * CPU oracle for the vToken repack path.  TEST INFRASTRUCTURE ONLY -- see vtoken_oracle.h.
 *
 * Everything below is the definition written out: one request, one token, one layer, one
 * row at a time.  No blocking, no fusion, no reordering beyond what the paper states.
 */
#include "vtoken_oracle.h"

#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

static int is_live(const int32_t *tt_slots, const uint8_t *keep, int64_t t)
{
    /* an active token: it owns a physical copy and the policy has not evicted it
     * (token table: location plus liveness bit, Sec. 3.2) */
    return tt_slots[t] >= 0 && (keep == NULL || keep[t] != 0);
}

static int32_t ceil_div(int64_t a, int64_t b) { return (int32_t)((a + b - 1) / b); }

int vto_plan(int32_t R, int32_t S,
             const int32_t *bt_offsets, const int32_t *bt_blocks,
             const int32_t *tt_offsets, const int32_t *tt_slots, const uint8_t *keep,
             const uint8_t *select, uint32_t thr_num, uint32_t thr_den,
             const int32_t *free_blocks, int32_t num_free,
             int32_t *new_bt_offsets, int32_t *new_bt_blocks, int32_t *new_tt_slots,
             int32_t *freed_blocks, int32_t *req_status,
             int32_t *move_src, int32_t *move_dst, vto_counts *counts)
{
    if (R < 0 || S < 1 || num_free < 0 || !bt_offsets || !tt_offsets || !counts) return VTO_EINVAL;

    int32_t consumed = 0;     /* free-list entries handed out so far */
    int32_t num_freed = 0, num_moves = 0, num_admitted = 0, num_deferred = 0;
    int32_t new_bt_fill = 0;
    int stop = 0;             /* once a candidate does not fit, every later one is deferred */

    for (int32_t r = 0; r < R; ++r) {                       /* requests in ascending index */
        const int64_t t0 = tt_offsets[r], t1 = tt_offsets[r + 1];
        const int32_t b0 = bt_offsets[r], b1 = bt_offsets[r + 1];
        const int32_t nb = b1 - b0;                         /* blocks the request holds now */

        /* live-token footprint T_live of the request (Sec. 3.3.3) */
        int64_t n = 0;
        for (int64_t t = t0; t < t1; ++t) n += is_live(tt_slots, keep, t);

        /* destinations needed: ceil(T_live / S) (Sec. 3.3.3) */
        const int32_t need = ceil_div(n, S);

        /* eligibility: caller's selection and the live-fraction threshold, in integers */
        int sel = (select == NULL || select[r] != 0);
        if (sel && thr_den != 0) {
            const uint64_t lhs = (uint64_t)n * (uint64_t)thr_den;
            const uint64_t rhs = (uint64_t)thr_num * (uint64_t)nb * (uint64_t)S;
            sel = lhs < rhs;
        }

        int32_t status;
        if (!sel) status = VTO_NOT_SELECTED;
        else if (!(need < nb)) status = VTO_NO_GAIN;        /* block count must strictly drop (I4) */
        else if (stop || (int64_t)consumed + need > num_free) {
            status = VTO_DEFERRED_NO_FREE;                  /* destinations unavailable (Sec. 3.3.2) */
            stop = 1;
        } else status = VTO_REPACKED;
        req_status[r] = status;

        new_bt_offsets[r] = new_bt_fill;
        if (status == VTO_REPACKED) {
            const int32_t *dst = free_blocks + consumed;    /* next `need` entries, list order */
            int64_t i = 0;                                  /* rank among the live tokens */
            for (int64_t t = t0; t < t1; ++t) {             /* ascending logical id */
                if (is_live(tt_slots, keep, t)) {
                    /* fill each destination block completely before the next (Sec. 3.3.3);
                     * slot = block * S + offset (Sec. 3.4) */
                    const int32_t slot = dst[i / S] * S + (int32_t)(i % S);
                    new_tt_slots[t] = slot;
                    move_src[num_moves] = tt_slots[t];
                    move_dst[num_moves] = slot;
                    ++num_moves;
                    ++i;
                } else {
                    new_tt_slots[t] = -1;                   /* evicted: no slot any more */
                }
            }
            for (int32_t j = 0; j < need; ++j) new_bt_blocks[new_bt_fill++] = dst[j];
            for (int32_t j = b0; j < b1; ++j) freed_blocks[num_freed++] = bt_blocks[j];
            consumed += need;
            ++num_admitted;
        } else {
            if (status == VTO_DEFERRED_NO_FREE) ++num_deferred;
            for (int64_t t = t0; t < t1; ++t)
                new_tt_slots[t] = is_live(tt_slots, keep, t) ? tt_slots[t] : -1;
            for (int32_t j = b0; j < b1; ++j) new_bt_blocks[new_bt_fill++] = bt_blocks[j];
        }
    }
    new_bt_offsets[R] = new_bt_fill;

    counts->num_moves = num_moves;
    counts->num_dst_blocks = consumed;
    counts->num_freed = num_freed;
    counts->num_free_consumed = consumed;
    counts->num_admitted = num_admitted;
    counts->num_deferred = num_deferred;
    counts->num_released = 0;
    return VTO_OK;
}

int vto_apply_moves_slab(uint8_t *slab, int64_t num_slots, int64_t row_bytes,
                         const int32_t *move_src, const int32_t *move_dst, int32_t num_moves)
{
    if (!slab || row_bytes < 1 || num_moves < 0) return VTO_EINVAL;
    for (int32_t m = 0; m < num_moves; ++m) {
        const int64_t s = move_src[m], d = move_dst[m];
        if (s < 0 || d < 0 || s >= num_slots || d >= num_slots) return VTO_EINVAL;
        memcpy(slab + d * row_bytes, slab + s * row_bytes, (size_t)row_bytes);
    }
    return VTO_OK;
}

int vto_apply_moves_pools(uint8_t *k_pool, uint8_t *v_pool, int32_t L, int64_t layer_stride_bytes,
                          int64_t num_slots, int64_t row_bytes,
                          const int32_t *move_src, const int32_t *move_dst, int32_t num_moves,
                          int32_t threads)
{
    if (!k_pool || !v_pool || L < 1) return VTO_EINVAL;
    if (layer_stride_bytes == 0) layer_stride_bytes = num_slots * row_bytes;
    int rc = VTO_OK;
    (void)threads;
    /* the 2L (K|V, layer) slabs are independent of one another */
#ifdef _OPENMP
#pragma omp parallel for num_threads(threads > 0 ? threads : 1) schedule(dynamic, 1)
#endif
    for (int32_t i = 0; i < 2 * L; ++i) {
        uint8_t *pool = (i < L) ? k_pool : v_pool;
        const int32_t layer = (i < L) ? i : i - L;
        int e = vto_apply_moves_slab(pool + (int64_t)layer * layer_stride_bytes, num_slots, row_bytes,
                                     move_src, move_dst, num_moves);
        if (e != VTO_OK) {
#ifdef _OPENMP
#pragma omp critical
#endif
            rc = e;
        }
    }
    return rc;
}

int64_t vto_gather_logical(const uint8_t *slab, int64_t num_slots, int64_t row_bytes,
                           const int32_t *tt_slots, const uint8_t *keep, int32_t len,
                           uint8_t *out, int64_t out_capacity_rows)
{
    if (!slab || !tt_slots || row_bytes < 1 || len < 0) return VTO_EINVAL;
    int64_t n = 0;
    for (int32_t t = 0; t < len; ++t) {
        if (!is_live(tt_slots, keep, t)) continue;
        if (tt_slots[t] >= num_slots || n >= out_capacity_rows) return VTO_EINVAL;
        memcpy(out + n * row_bytes, slab + (int64_t)tt_slots[t] * row_bytes, (size_t)row_bytes);
        ++n;
    }
    return n;
}

int vto_validate(int32_t R, int32_t S, int32_t NB,
                 const int32_t *bt_offsets, const int32_t *bt_blocks,
                 const int32_t *tt_offsets, const int32_t *tt_slots, const uint8_t *keep,
                 const int32_t *free_blocks, int32_t num_free, int32_t *first_bad)
{
    int32_t bad = 0;
    if (R < 0 || S < 1 || NB < 0) return VTO_EINVAL;
    /* owner[b]: -1 unused, r >= 0 block of request r, -2 on the free list */
    int32_t *owner = (int32_t *)malloc(sizeof(int32_t) * (size_t)(NB > 0 ? NB : 1));
    uint8_t *taken = (uint8_t *)calloc((size_t)NB * (size_t)S + 1, 1);
    if (!owner || !taken) { free(owner); free(taken); return VTO_EINVAL; }
    for (int32_t b = 0; b < NB; ++b) owner[b] = -1;

    for (int32_t r = 0; r < R && !bad; ++r) {
        if (bt_offsets[r + 1] < bt_offsets[r] || tt_offsets[r + 1] < tt_offsets[r]) bad = 1;
        for (int32_t j = bt_offsets[r]; j < bt_offsets[r + 1] && !bad; ++j) {
            const int32_t b = bt_blocks[j];
            if (b < 0 || b >= NB) bad = 2;                 /* block id out of range */
            else if (owner[b] != -1) bad = 3;              /* block in two tables (or twice) */
            else owner[b] = r;
        }
    }
    for (int32_t j = 0; j < num_free && !bad; ++j) {
        const int32_t b = free_blocks[j];
        if (b < 0 || b >= NB) bad = 4;                     /* free id out of range */
        else if (owner[b] != -1) bad = 5;                  /* free block allocated or listed twice */
        else owner[b] = -2;
    }
    for (int32_t r = 0; r < R && !bad; ++r) {
        for (int64_t t = tt_offsets[r]; t < tt_offsets[r + 1] && !bad; ++t) {
            const int32_t s = tt_slots[t];
            if (s < 0) { if (keep && keep[t]) { /* kept but no physical copy: not live */ } continue; }
            if ((int64_t)s >= (int64_t)NB * S) bad = 6;    /* slot out of range */
            else if (owner[s / S] != r) bad = 7;           /* slot outside the request's blocks */
            else if (taken[s]) bad = 8;                    /* slot referenced twice (I2) */
            else taken[s] = 1;
        }
    }
    free(owner); free(taken);
    if (first_bad) *first_bad = bad;
    return bad ? VTO_EPRECOND : VTO_OK;
}

int vto_check_tables(int32_t R, int32_t S, int32_t NB,
                     const int32_t *bt_offsets, const int32_t *bt_blocks,
                     const int32_t *tt_offsets, const int32_t *tt_slots,
                     const int32_t *free_blocks, int32_t num_free, const uint8_t *protect, uint32_t *bits)
{
    if (R < 0 || S < 1 || NB < 0 || num_free < 0 || !bt_offsets || !tt_offsets || !bits) return VTO_EINVAL;
    uint32_t f = 0;
    const size_t nb = (size_t)(NB > 0 ? NB : 1);
    int32_t *in_tables = (int32_t *)calloc(nb, sizeof(int32_t));     /* block-table entries holding block b */
    int32_t *in_free = (int32_t *)calloc(nb, sizeof(int32_t));       /* free-list entries naming block b */
    int32_t *refs = (int32_t *)calloc((size_t)NB * (size_t)S + 1, sizeof(int32_t));   /* entries naming slot s */
    int32_t *holders = (int32_t *)calloc(nb, sizeof(int32_t));       /* distinct requests holding block b */
    int32_t *last_holder = (int32_t *)calloc(nb, sizeof(int32_t));   /* the last of them */
    if (!in_tables || !in_free || !refs || !holders || !last_holder) {
        free(in_tables); free(in_free); free(refs); free(holders); free(last_holder);
        return VTO_EINVAL;
    }

    for (int32_t r = 0; r < R; ++r)
        if (bt_offsets[r + 1] < bt_offsets[r] || tt_offsets[r + 1] < tt_offsets[r]) f |= 1u;
    if (f) goto done;                                      /* the ranges below would be meaningless */

    for (int32_t r = 0; r < R; ++r) {
        for (int32_t j = bt_offsets[r]; j < bt_offsets[r + 1]; ++j) {
            const int32_t b = bt_blocks[j];
            if (b < 0 || b >= NB) { f |= 2u; continue; }
            ++in_tables[b];
            /* number of distinct requests holding b (a request's entries are consecutive) */
            if (holders[b] == 0 || last_holder[b] != r) ++holders[b];
            last_holder[b] = r;
        }
    }
    for (int32_t b = 0; b < NB; ++b)
        if (in_tables[b] > 1 && !(protect && protect[b])) f |= 4u;
    for (int32_t j = 0; j < num_free; ++j) {
        const int32_t b = free_blocks[j];
        if (b < 0 || b >= NB) f |= 8u;
        else ++in_free[b];
    }
    for (int32_t b = 0; b < NB; ++b)
        if (in_free[b] > 1 || (in_free[b] == 1 && in_tables[b] > 0)) f |= 16u;
    for (int32_t r = 0; r < R; ++r) {
        for (int64_t t = tt_offsets[r]; t < tt_offsets[r + 1]; ++t) {
            const int32_t s = tt_slots[t];
            if (s < 0) continue;
            if ((int64_t)s >= (int64_t)NB * S) { f |= 32u; continue; }
            /* whose block is it?  a block held by several requests (shared prefix) is outside this check */
            const int32_t b = s / S;
            if (holders[b] == 0 || (holders[b] == 1 && last_holder[b] != r)) f |= 64u;
            ++refs[s];
        }
    }
    for (int64_t s = 0; s < (int64_t)NB * S; ++s)
        if (refs[s] > 1 && !(protect && protect[s / S])) f |= 128u;   /* sharers all map a shared block's slots */
done:
    free(in_tables); free(in_free); free(refs); free(holders); free(last_holder);
    *bits = f;
    return VTO_OK;
}

static int cmp_i32(const void *a, const void *b)
{
    const int32_t x = *(const int32_t *)a, y = *(const int32_t *)b;
    return (x > y) - (x < y);
}

int vto_check_semantics(int32_t R, int32_t S,
                        const int32_t *bt_offsets, const int32_t *bt_blocks,
                        const int32_t *tt_offsets, const int32_t *tt_slots, const uint8_t *keep,
                        const uint8_t *select, uint32_t thr_num, uint32_t thr_den,
                        const int32_t *free_blocks, int32_t num_free,
                        const int32_t *new_bt_offsets, const int32_t *new_bt_blocks,
                        const int32_t *new_tt_slots, const int32_t *freed_blocks,
                        int32_t num_freed, int32_t num_free_consumed,
                        const int32_t *req_status, int32_t *first_bad)
{
    int32_t bad = 0;
    if (R < 0 || S < 1) return VTO_EINVAL;
    const int32_t total_old = bt_offsets[R];
    int32_t *exp_freed = (int32_t *)malloc(sizeof(int32_t) * (size_t)(total_old + 1));
    int32_t *got_freed = (int32_t *)malloc(sizeof(int32_t) * (size_t)(num_freed + 1));
    int32_t *got_dst = (int32_t *)malloc(sizeof(int32_t) * (size_t)(num_free + 1));
    int32_t *exp_dst = (int32_t *)malloc(sizeof(int32_t) * (size_t)(num_free + 1));
    if (!exp_freed || !got_freed || !got_dst || !exp_dst) {
        free(exp_freed); free(got_freed); free(got_dst); free(exp_dst); return VTO_EINVAL;
    }
    int32_t n_exp_freed = 0, n_got_dst = 0;
    int64_t demand = 0;
    int stop = 0;
    if (new_bt_offsets[0] != 0) bad = 1;
    for (int32_t r = 0; r < R && !bad; ++r) {
        const int64_t t0 = tt_offsets[r], t1 = tt_offsets[r + 1];
        const int32_t nb = bt_offsets[r + 1] - bt_offsets[r];
        int64_t n = 0;
        for (int64_t t = t0; t < t1; ++t) n += is_live(tt_slots, keep, t);
        const int32_t need = ceil_div(n, S);
        int sel = (select == NULL || select[r] != 0);
        if (sel && thr_den != 0)
            sel = (uint64_t)n * thr_den < (uint64_t)thr_num * (uint64_t)nb * (uint64_t)S;
        int32_t want;
        if (!sel) want = VTO_NOT_SELECTED;
        else if (need >= nb) want = VTO_NO_GAIN;
        else if (stop || demand + need > num_free) { want = VTO_DEFERRED_NO_FREE; stop = 1; }
        else { want = VTO_REPACKED; demand += need; }
        if (req_status[r] != want) { bad = 2; break; }

        const int32_t nbt0 = new_bt_offsets[r], nbt1 = new_bt_offsets[r + 1];
        if (want == VTO_REPACKED) {
            if (nbt1 - nbt0 != need) { bad = 3; break; }
            int64_t i = 0;
            for (int64_t t = t0; t < t1; ++t) {
                if (is_live(tt_slots, keep, t)) {
                    /* i-th live token sits at offset i % S of the request's (i / S)-th new block */
                    if (new_tt_slots[t] != new_bt_blocks[nbt0 + i / S] * S + (int32_t)(i % S)) { bad = 4; break; }
                    ++i;
                } else if (new_tt_slots[t] != -1) { bad = 5; break; }
            }
            if (bad) break;
            for (int32_t j = nbt0; j < nbt1; ++j) got_dst[n_got_dst++] = new_bt_blocks[j];
            for (int32_t j = bt_offsets[r]; j < bt_offsets[r + 1]; ++j) exp_freed[n_exp_freed++] = bt_blocks[j];
        } else {
            if (nbt1 - nbt0 != nb) { bad = 6; break; }
            for (int32_t j = 0; j < nb; ++j)
                if (new_bt_blocks[nbt0 + j] != bt_blocks[bt_offsets[r] + j]) { bad = 7; break; }
            for (int64_t t = t0; t < t1 && !bad; ++t) {
                const int32_t want_slot = is_live(tt_slots, keep, t) ? tt_slots[t] : -1;
                if (new_tt_slots[t] != want_slot) bad = 8;
            }
        }
    }
    if (!bad) {
        /* the destination set is the consumed prefix of the free list; the reclaimed set is
         * the admitted requests' old blocks -- as sets, order not constrained here */
        if (n_got_dst != num_free_consumed || num_free_consumed != (int32_t)demand) bad = 9;
        else if (n_exp_freed != num_freed) bad = 10;
        else {
            memcpy(exp_dst, free_blocks, sizeof(int32_t) * (size_t)num_free_consumed);
            memcpy(got_freed, freed_blocks, sizeof(int32_t) * (size_t)num_freed);
            qsort(exp_dst, (size_t)num_free_consumed, sizeof(int32_t), cmp_i32);
            qsort(got_dst, (size_t)n_got_dst, sizeof(int32_t), cmp_i32);
            qsort(exp_freed, (size_t)n_exp_freed, sizeof(int32_t), cmp_i32);
            qsort(got_freed, (size_t)num_freed, sizeof(int32_t), cmp_i32);
            if (memcmp(exp_dst, got_dst, sizeof(int32_t) * (size_t)n_got_dst) != 0) bad = 11;
            else if (memcmp(exp_freed, got_freed, sizeof(int32_t) * (size_t)num_freed) != 0) bad = 12;
        }
    }
    free(exp_freed); free(got_freed); free(got_dst); free(exp_dst);
    if (first_bad) *first_bad = bad;
    return bad ? VTO_EPRECOND : VTO_OK;
}

double vto_waste_ratio(int32_t S, int64_t num_allocated_blocks,
                       const int32_t *tt_slots, const uint8_t *keep, int64_t T)
{
    if (num_allocated_blocks <= 0 || S < 1) return 0.0;
    int64_t live = 0;                                       /* sum over blocks of n_b */
    for (int64_t t = 0; t < T; ++t) live += is_live(tt_slots, keep, t);
    return 1.0 - (double)live / ((double)num_allocated_blocks * (double)S);
}

int vto_evict_tokens(int32_t R, const int32_t *tt_offsets, const int32_t *tt_len, uint8_t *keep,
                     const int32_t *victim_req, const int32_t *victim_tok, int32_t num_victims,
                     int32_t *num_bad)
{
    if (R < 0 || num_victims < 0 || !tt_offsets || !tt_len || !keep) return VTO_EINVAL;
    int32_t bad = 0;
    for (int32_t i = 0; i < num_victims; ++i) {
        const int32_t r = victim_req[i], t = victim_tok[i];
        if (r < 0 || r >= R || t < 0 || t >= tt_len[r]) { ++bad; continue; }
        keep[(int64_t)tt_offsets[r] + t] = 0;          /* logically inactive; the KV bytes stay (Sec. 3.2) */
    }
    if (num_bad) *num_bad = bad;
    return VTO_OK;
}

int vto_sync_new_tokens(int32_t R, int32_t S, const int32_t *tt_offsets, int32_t *tt_slots, uint8_t *keep,
                        int32_t *tt_len, int32_t *phys_len, const int32_t *bt_offsets,
                        const int32_t *bt_blocks, const int32_t *new_len, int32_t *num_bad)
{
    if (R < 0 || S < 1) return VTO_EINVAL;
    int32_t bad = 0;
    for (int32_t r = 0; r < R; ++r) {
        const int32_t cap = tt_offsets[r + 1] - tt_offsets[r];
        const int64_t room = (int64_t)(bt_offsets[r + 1] - bt_offsets[r]) * S;   /* slots in the block list */
        int stopped = 0;
        while (tt_len[r] < new_len[r]) {
            const int32_t t = tt_len[r];                /* next sequential logical id */
            const int64_t p = phys_len[r];              /* next position in the block list */
            if (t >= cap || p >= room) { stopped = 1; break; }
            const int32_t block = bt_blocks[bt_offsets[r] + p / S];
            tt_slots[(int64_t)tt_offsets[r] + t] = block * S + (int32_t)(p % S);
            keep[(int64_t)tt_offsets[r] + t] = 1;
            tt_len[r] = t + 1;
            phys_len[r] = (int32_t)(p + 1);
        }
        bad += stopped;
    }
    if (num_bad) *num_bad = bad;
    return VTO_OK;
}

int vto_evict_tokens_counted(int32_t R, int32_t S, int32_t NB, const int32_t *tt_offsets, const int32_t *tt_len,
                             const int32_t *tt_slots, uint8_t *keep, const int32_t *victim_req,
                             const int32_t *victim_tok, int32_t num_victims, int32_t *n_b, int64_t *live_total,
                             int32_t *num_bad)
{
    if (R < 0 || S < 1 || NB < 0 || num_victims < 0 || !tt_offsets || !tt_len || !tt_slots || !keep || !n_b)
        return VTO_EINVAL;
    int32_t bad = 0;
    for (int32_t i = 0; i < num_victims; ++i) {
        const int32_t r = victim_req[i], t = victim_tok[i];
        if (r < 0 || r >= R || t < 0 || t >= tt_len[r]) { ++bad; continue; }
        const int64_t e = (int64_t)tt_offsets[r] + t;
        const int32_t s = tt_slots[e];
        /* the block loses a live token only if this call is what deactivates it */
        if (keep[e] != 0 && s >= 0 && (int64_t)s < (int64_t)NB * S) {
            --n_b[s / S];
            if (live_total) --*live_total;
        }
        keep[e] = 0;
    }
    if (num_bad) *num_bad = bad;
    return VTO_OK;
}

int vto_sync_new_tokens_counted(int32_t R, int32_t S, int32_t NB, const int32_t *tt_offsets, int32_t *tt_slots,
                                uint8_t *keep, int32_t *tt_len, int32_t *phys_len, const int32_t *bt_offsets,
                                const int32_t *bt_blocks, const int32_t *new_len, int32_t *n_b, int64_t *live_total,
                                int32_t *num_bad)
{
    if (R < 0 || S < 1 || NB < 0 || !tt_offsets || !tt_len || !n_b) return VTO_EINVAL;
    int32_t *before = (int32_t *)malloc(sizeof(int32_t) * (size_t)(R > 0 ? R : 1));
    if (!before) return VTO_EINVAL;
    for (int32_t r = 0; r < R; ++r) before[r] = tt_len[r];
    /* register the tokens ... */
    const int rc = vto_sync_new_tokens(R, S, tt_offsets, tt_slots, keep, tt_len, phys_len, bt_offsets, bt_blocks,
                                       new_len, num_bad);
    /* ... and every new token is one more live token in the block that holds it */
    for (int32_t r = 0; r < R && rc == VTO_OK; ++r) {
        for (int32_t t = before[r]; t < tt_len[r]; ++t) {
            const int32_t s = tt_slots[(int64_t)tt_offsets[r] + t];
            if (s >= 0 && (int64_t)s < (int64_t)NB * S) {
                ++n_b[s / S];
                if (live_total) ++*live_total;
            }
        }
    }
    free(before);
    return rc;
}

int64_t vto_build_slot_mapping(int32_t R, const int32_t *tt_offsets, const int32_t *tt_slots,
                               const uint8_t *keep, const uint8_t *select, int32_t *out_slots,
                               int32_t *out_token_ids, int32_t *out_offsets, int64_t capacity)
{
    if (R < 0 || !tt_offsets || !tt_slots || !out_offsets) return VTO_EINVAL;
    int64_t n = 0;
    for (int32_t r = 0; r < R; ++r) {
        out_offsets[r] = (int32_t)n;
        if (select != NULL && select[r] == 0) continue;
        for (int64_t t = tt_offsets[r]; t < tt_offsets[r + 1]; ++t) {
            if (!is_live(tt_slots, keep, t)) continue;  /* evicted tokens are left out (Sec. 3.2) */
            if (n >= capacity) return VTO_EINVAL;
            if (out_slots) out_slots[n] = tt_slots[t];  /* the table already stores block * S + offset */
            if (out_token_ids) out_token_ids[n] = (int32_t)(t - tt_offsets[r]);
            ++n;
        }
    }
    out_offsets[R] = (int32_t)n;
    return n;
}

int vto_apply_moves(int32_t R, int32_t S, const int32_t *tt_offsets, int32_t *tt_slots, uint8_t *keep,
                    int32_t *phys_len, const int32_t *new_tt_slots, const int32_t *req_status,
                    const int32_t *new_bt_offsets, const int32_t *append_pos)
{
    if (R < 0 || S < 1 || !tt_offsets || !tt_slots || !keep || !new_tt_slots) return VTO_EINVAL;
    for (int32_t r = 0; r < R; ++r) {
        int32_t with_slot = 0, moved = 0;
        for (int64_t t = tt_offsets[r]; t < tt_offsets[r + 1]; ++t) {
            moved += new_tt_slots[t] >= 0 && new_tt_slots[t] != tt_slots[t];   /* destinations are never sources */
            tt_slots[t] = new_tt_slots[t];              /* source entry cleared, destination written (I2) */
            keep[t] = new_tt_slots[t] >= 0 ? 1 : 0;
            with_slot += new_tt_slots[t] >= 0;
        }
        if (phys_len && req_status && req_status[r] == VTO_REPACKED) {
            if (append_pos) {
                phys_len[r] = append_pos[r];            /* worked out by the repack in waves, wave by wave */
            } else if (new_bt_offsets) {
                /* new block list = blocks that stayed, then the destination blocks, which the moved
                 * tokens fill densely: the next token lands right behind them */
                const int32_t blocks = new_bt_offsets[r + 1] - new_bt_offsets[r];
                phys_len[r] = (blocks - ceil_div(moved, S)) * S + moved;
            } else {
                phys_len[r] = with_slot;                /* whole-request plans: nothing stayed */
            }
        }
    }
    return VTO_OK;
}

int vto_slot_cache_mark(int32_t R, uint8_t *dirty, const int32_t *victim_req, int32_t num_victims,
                        const int32_t *req_status)
{
    if (R < 0 || !dirty || num_victims < 0 || (num_victims > 0 && !victim_req)) return VTO_EINVAL;
    /* eviction and relocation are the structural changes that invalidate a cached array */
    for (int32_t i = 0; i < num_victims; ++i)
        if (victim_req[i] >= 0 && victim_req[i] < R) dirty[victim_req[i]] = 1;
    if (req_status)
        for (int32_t r = 0; r < R; ++r)
            if (req_status[r] == VTO_REPACKED) dirty[r] = 1;
    return VTO_OK;
}

int vto_slot_cache_update(int32_t R, const int32_t *tt_offsets, const int32_t *tt_slots, const uint8_t *keep,
                          const int32_t *tt_len, uint8_t *dirty, int32_t *cache_slots, int32_t *cache_ids,
                          int32_t *cache_len, int32_t *cache_seen, int32_t *num_rebuilt, int32_t *num_appended)
{
    if (R < 0 || !tt_offsets || !tt_slots || !tt_len || !dirty || !cache_slots || !cache_len || !cache_seen)
        return VTO_EINVAL;
    int32_t rebuilt = 0, appended = 0;
    for (int32_t r = 0; r < R; ++r) {
        const int64_t base = tt_offsets[r];
        int32_t first;                       /* first registered token the cache does not cover yet */
        if (dirty[r]) {                      /* structural change: start over */
            cache_len[r] = 0;
            first = 0;
            dirty[r] = 0;
            ++rebuilt;
        } else if (tt_len[r] > cache_seen[r]) {   /* append-only growth */
            first = cache_seen[r];
            ++appended;
        } else {
            continue;
        }
        for (int32_t t = first; t < tt_len[r]; ++t) {
            if (!is_live(tt_slots, keep, base + t)) continue;
            cache_slots[base + cache_len[r]] = tt_slots[base + t];
            if (cache_ids) cache_ids[base + cache_len[r]] = t;
            ++cache_len[r];
        }
        cache_seen[r] = tt_len[r];
    }
    if (num_rebuilt) *num_rebuilt = rebuilt;
    if (num_appended) *num_appended = appended;
    return VTO_OK;
}

int vto_block_liveness(int32_t R, int32_t S, int32_t NB, const int32_t *bt_offsets, const int32_t *bt_blocks,
                       const int32_t *tt_offsets, const int32_t *tt_slots, const uint8_t *keep,
                       int32_t *n_b, int64_t *hist, int64_t *live_total, int64_t *num_allocated)
{
    if (R < 0 || S < 1 || NB < 0 || !n_b) return VTO_EINVAL;
    for (int32_t b = 0; b < NB; ++b) n_b[b] = 0;
    int64_t live = 0;
    for (int64_t t = 0; t < tt_offsets[R]; ++t) {
        if (!is_live(tt_slots, keep, t)) continue;
        const int64_t b = tt_slots[t] / S;                 /* slot = block * S + offset */
        if (b >= NB) return VTO_EINVAL;
        ++n_b[b];                                          /* n_b: valid tokens stored in block b */
        ++live;
    }
    if (hist) {
        for (int32_t k = 0; k <= S; ++k) hist[k] = 0;
        for (int32_t j = 0; j < bt_offsets[R]; ++j) {
            const int32_t b = bt_blocks[j];
            if (b < 0 || b >= NB) return VTO_EINVAL;
            /* a block referenced by several requests (shared prefix) counts one per reference: clip */
            ++hist[n_b[b] > S ? S : n_b[b]];
        }
    }
    if (live_total) *live_total = live;
    if (num_allocated) *num_allocated = bt_offsets[R];
    return VTO_OK;
}

int vto_plan_partial(int32_t R, int32_t S, int32_t NB,
                     const int32_t *bt_offsets, const int32_t *bt_blocks,
                     const int32_t *tt_offsets, const int32_t *tt_slots, const uint8_t *keep,
                     const uint8_t *select, uint32_t thr_num, uint32_t thr_den,
                     const int32_t *free_blocks, int32_t num_free, const vto_partial_opts *opts,
                     int32_t *new_bt_offsets, int32_t *new_bt_blocks, int32_t *new_tt_slots,
                     int32_t *freed_blocks, int32_t *req_status,
                     int32_t *move_src, int32_t *move_dst, vto_counts *counts, int32_t *released_blocks)
{
    if (R < 0 || S < 1 || NB < 1 || num_free < 0 || !opts || !counts) return VTO_EINVAL;
    const int may_detach = opts->protect != NULL && opts->detach_den != 0;
    if (may_detach && !released_blocks) return VTO_EINVAL;
    if (opts->detach_rule > 2) return VTO_EINVAL;
    int32_t *n_b = (int32_t *)malloc(sizeof(int32_t) * (size_t)NB);
    uint8_t *is_source = (uint8_t *)malloc((size_t)NB);     /* per physical block, for the request at hand */
    int32_t *own_live = (int32_t *)calloc((size_t)NB, sizeof(int32_t));   /* n_rb: live tokens of the request at
                                                                             hand stored in block b */
    if (!n_b || !is_source || !own_live) { free(n_b); free(is_source); free(own_live); return VTO_EINVAL; }

    /* eligibility metadata: per-block liveness and the global waste ratio F (Sec. 3.3.1) */
    int64_t live_total = 0, N = 0;
    int rc = vto_block_liveness(R, S, NB, bt_offsets, bt_blocks, tt_offsets, tt_slots, keep, n_b, NULL,
                                &live_total, &N);
    if (rc != VTO_OK) { free(n_b); free(is_source); free(own_live); return rc; }
    /* F > theta  <=>  (N*S - live) * den > num * N*S, in integers */
    int triggered = 1;
    if (opts->theta_den != 0) {
        const uint64_t cap = (uint64_t)N * (uint64_t)S;
        triggered = N > 0 && (cap - (uint64_t)live_total) * opts->theta_den > (uint64_t)opts->theta_num * cap;
    }
    memset(is_source, 0, (size_t)NB);

    int32_t consumed = 0, num_freed = 0, num_moves = 0, num_admitted = 0, num_deferred = 0, new_bt_fill = 0;
    int32_t num_released = 0;
    int stop = 0;
    for (int32_t r = 0; r < R; ++r) {
        const int64_t t0 = tt_offsets[r], t1 = tt_offsets[r + 1];
        const int32_t b0 = bt_offsets[r], b1 = bt_offsets[r + 1];
        const int32_t nb = b1 - b0;

        /* copy-on-write detach: does the request leave its shared blocks?  It does when its own live
         * tokens fill less than detach_num / detach_den of them. */
        int detach = 0;
        if (may_detach) {
            int64_t ns_shared = 0, n_shared = 0;
            for (int32_t j = b0; j < b1; ++j) ns_shared += opts->protect[bt_blocks[j]] != 0;
            for (int64_t t = t0; t < t1; ++t)
                if (is_live(tt_slots, keep, t)) n_shared += opts->protect[tt_slots[t] / S] != 0;
            detach = ns_shared > 0 &&
                     (uint64_t)n_shared * opts->detach_den < (uint64_t)opts->detach_num * (uint64_t)ns_shared * (uint64_t)S;
            /* block by block instead: the census of the request's own live tokens per block */
            if (opts->detach_rule == 1)
                for (int64_t t = t0; t < t1; ++t)
                    if (is_live(tt_slots, keep, t)) ++own_live[tt_slots[t] / S];
        }

        /* source blocks: unprotected, low utilisation, at most B of them in table order (Sec. 3.3.3) */
        int32_t ns = 0, ns_unprotected = 0;
        for (int32_t j = b0; j < b1; ++j) {
            const int32_t b = bt_blocks[j];
            const int shared = opts->protect && opts->protect[b];
            int eligible = !shared;
            if (eligible && opts->util_den != 0)
                eligible = (uint64_t)n_b[b] * opts->util_den < (uint64_t)opts->util_num * (uint64_t)S;
            if (eligible && opts->max_source_blocks > 0 && ns_unprotected >= opts->max_source_blocks) eligible = 0;
            ns_unprotected += eligible;
            if (shared && may_detach) {
                if (opts->detach_rule == 1)                /* the shared blocks this request fills poorly */
                    eligible = (uint64_t)own_live[b] * opts->detach_den < (uint64_t)opts->detach_num * (uint64_t)S;
                else if (opts->detach_rule == 2)           /* the shared blocks all their holders together fill poorly */
                    eligible = (uint64_t)n_b[b] * opts->detach_den < (uint64_t)opts->detach_num * (uint64_t)S;
                else
                    eligible = detach;                     /* every shared block of a detaching request */
            }
            is_source[b] = (uint8_t)eligible;
            ns += eligible;
        }
        /* live tokens of the request, and those that sit in source blocks (T_live) */
        int64_t n = 0, n_src = 0;
        for (int64_t t = t0; t < t1; ++t) {
            if (!is_live(tt_slots, keep, t)) continue;
            ++n;
            n_src += is_source[tt_slots[t] / S];
        }
        const int32_t need = ceil_div(n_src, S);

        int sel = triggered && (select == NULL || select[r] != 0);
        if (sel && thr_den != 0)
            sel = (uint64_t)n * thr_den < (uint64_t)thr_num * (uint64_t)nb * (uint64_t)S;
        int32_t status;
        if (!sel) status = VTO_NOT_SELECTED;
        else if (!(need < ns)) status = VTO_NO_GAIN;        /* sources must release more than they consume */
        else if (stop || (int64_t)consumed + need > num_free) { status = VTO_DEFERRED_NO_FREE; stop = 1; }
        else status = VTO_REPACKED;
        req_status[r] = status;

        new_bt_offsets[r] = new_bt_fill;
        if (status == VTO_REPACKED) {
            const int32_t *dst = free_blocks + consumed;
            int64_t i = 0;
            for (int64_t t = t0; t < t1; ++t) {
                if (!is_live(tt_slots, keep, t)) { new_tt_slots[t] = -1; continue; }
                if (is_source[tt_slots[t] / S]) {
                    const int32_t slot = dst[i / S] * S + (int32_t)(i % S);
                    new_tt_slots[t] = slot;
                    move_src[num_moves] = tt_slots[t];
                    move_dst[num_moves] = slot;
                    ++num_moves;
                    ++i;
                } else {
                    new_tt_slots[t] = tt_slots[t];          /* its block stays in place */
                }
            }
            for (int32_t j = b0; j < b1; ++j)
                if (!is_source[bt_blocks[j]]) new_bt_blocks[new_bt_fill++] = bt_blocks[j];
            for (int32_t j = 0; j < need; ++j) new_bt_blocks[new_bt_fill++] = dst[j];
            for (int32_t j = b0; j < b1; ++j) {
                const int32_t b = bt_blocks[j];
                if (!is_source[b]) continue;
                if (opts->protect && opts->protect[b]) released_blocks[num_released++] = b;   /* a reference less */
                else freed_blocks[num_freed++] = b;
            }
            consumed += need;
            ++num_admitted;
        } else {
            if (status == VTO_DEFERRED_NO_FREE) ++num_deferred;
            for (int64_t t = t0; t < t1; ++t)
                new_tt_slots[t] = is_live(tt_slots, keep, t) ? tt_slots[t] : -1;
            for (int32_t j = b0; j < b1; ++j) new_bt_blocks[new_bt_fill++] = bt_blocks[j];
        }
        for (int32_t j = b0; j < b1; ++j) is_source[bt_blocks[j]] = 0;
        if (may_detach && opts->detach_rule == 1)
            for (int64_t t = t0; t < t1; ++t)
                if (is_live(tt_slots, keep, t)) own_live[tt_slots[t] / S] = 0;
    }
    new_bt_offsets[R] = new_bt_fill;
    counts->num_moves = num_moves;
    counts->num_dst_blocks = consumed;
    counts->num_freed = num_freed;
    counts->num_free_consumed = consumed;
    counts->num_admitted = num_admitted;
    counts->num_deferred = num_deferred;
    counts->num_released = num_released;
    free(n_b); free(is_source); free(own_live);
    return VTO_OK;
}

static uint64_t mix64(uint64_t x)                           /* splitmix64 finaliser */
{
    x ^= x >> 30;
    x *= 0xBF58476D1CE4E5B9ull;
    x ^= x >> 27;
    x *= 0x94D049BB133111EBull;
    x ^= x >> 31;
    return x;
}

int vto_digest_logical(const uint8_t *k_pool, const uint8_t *v_pool, int64_t layer_stride_bytes, int64_t num_slots,
                       int64_t row_bytes, int32_t layer_begin, int32_t layer_end, const int32_t *tt_slots,
                       const uint8_t *keep, int32_t len, uint64_t *digest, int32_t *num_active)
{
    if (!k_pool || !v_pool || !tt_slots || !digest || row_bytes < 16 || row_bytes % 16 != 0) return VTO_EINVAL;
    if (layer_begin < 0 || layer_end <= layer_begin || len < 0) return VTO_EINVAL;
    if (layer_stride_bytes == 0) layer_stride_bytes = num_slots * row_bytes;
    const uint64_t A = 0x9E3779B97F4A7C15ull, B = 0xD1B54A32D192ED03ull, C = 0x8CB92BA72F3D8DD7ull,
                   D = 0xA0761D6478BD642Full;
    const int32_t nl = layer_end - layer_begin;
    uint64_t sum = 0;
    int32_t i = 0;                                           /* rank among the active tokens */
    for (int32_t t = 0; t < len; ++t) {
        if (!is_live(tt_slots, keep, t)) continue;
        if (tt_slots[t] >= num_slots) return VTO_EINVAL;
        for (int32_t s = 0; s < 2 * nl; ++s) {               /* K layers, then V layers */
            const uint8_t *pool = s < nl ? k_pool : v_pool;
            const int32_t layer = layer_begin + (s < nl ? s : s - nl);
            const uint8_t *row = pool + (int64_t)layer * layer_stride_bytes + (int64_t)tt_slots[t] * row_bytes;
            /* key of this (rank, id, slab): binds the row's words to their place in the logical view */
            const uint64_t key = mix64((((uint64_t)i * A + (uint64_t)t) * B + (uint64_t)s) * C);
            /* 32-byte groups of four little-endian words; a row of 16 (mod 32) bytes ends with a
             * half group of two words.  Every word is bound to its place by its own key. */
            const int64_t nwords = row_bytes / 8;
            for (int64_t g = 0; g * 4 < nwords; ++g) {
                uint64_t a = 0, b = 0;
                for (int64_t j = 4 * g; j < 4 * g + 4 && j < nwords; ++j) {
                    uint64_t w = 0;
                    for (int q = 7; q >= 0; --q) w = (w << 8) | row[j * 8 + q];
                    const uint64_t x = w ^ (key + (uint64_t)j * D);
                    if ((j & 1) == 0) a += x;                /* words 4g, 4g+2 */
                    else b += x;                             /* words 4g+1, 4g+3 */
                }
                const unsigned __int128 prod = (unsigned __int128)a * b;      /* full 128-bit product */
                sum += (uint64_t)prod ^ (uint64_t)(prod >> 64);
            }
        }
        ++i;
    }
    *digest = sum;
    if (num_active) *num_active = i;
    return VTO_OK;
}

int vto_plan_waves(int32_t R, int32_t S, int32_t NB,
                   const int32_t *bt_offsets, const int32_t *bt_blocks,
                   const int32_t *tt_offsets, const int32_t *tt_slots, const uint8_t *keep,
                   const uint8_t *select, uint32_t thr_num, uint32_t thr_den,
                   const int32_t *free_blocks, int32_t num_free, const vto_partial_opts *opts,
                   int32_t num_waves,
                   int32_t *new_bt_offsets, int32_t *new_bt_blocks, int32_t *new_tt_slots,
                   int32_t *req_status, int32_t *req_wave, int32_t *req_append_pos, int32_t *free_out,
                   int32_t *num_free_out, int32_t *move_src, int32_t *move_dst, int64_t move_capacity,
                   int64_t *wave_move_offsets, vto_counts *wave_counts, int32_t *released_blocks)
{
    if (R < 0 || S < 1 || num_free < 0 || num_waves < 1 || !bt_offsets || !tt_offsets || !num_free_out ||
        !wave_move_offsets || !wave_counts)
        return VTO_EINVAL;
    if (opts && opts->detach_den != 0 && !released_blocks) return VTO_EINVAL;   /* a detach needs its list */
    const int64_t T = tt_offsets[R], nbt = bt_offsets[R];
    const size_t nT = (size_t)(T > 0 ? T : 1), nB = (size_t)(nbt > 0 ? nbt : 1), nR = (size_t)R + 1;
    const size_t nP = (size_t)num_free + nB;

    /* the committed state a wave plans on (cur_*) and the state it proposes (nxt_*) */
    int32_t *cur_bto = malloc(nR * sizeof(int32_t)), *nxt_bto = malloc(nR * sizeof(int32_t));
    int32_t *cur_btb = malloc(nB * sizeof(int32_t)), *nxt_btb = malloc(nB * sizeof(int32_t));
    int32_t *cur_tts = malloc(nT * sizeof(int32_t)), *nxt_tts = malloc(nT * sizeof(int32_t));
    int32_t *pool = malloc(nP * sizeof(int32_t)), *pool_next = malloc(nP * sizeof(int32_t));
    int32_t *freed = malloc(nB * sizeof(int32_t)), *status = malloc(nR * sizeof(int32_t));
    int32_t *msrc = malloc(nT * sizeof(int32_t)), *mdst = malloc(nT * sizeof(int32_t));
    int32_t *rel = malloc(nB * sizeof(int32_t));
    int64_t total_released = 0;
    int rc = VTO_OK;
    if (!cur_bto || !nxt_bto || !cur_btb || !nxt_btb || !cur_tts || !nxt_tts || !pool || !pool_next || !freed ||
        !status || !msrc || !mdst || !rel) {
        rc = VTO_EINVAL;
        goto done;
    }
    memcpy(cur_bto, bt_offsets, nR * sizeof(int32_t));
    if (nbt > 0) memcpy(cur_btb, bt_blocks, (size_t)nbt * sizeof(int32_t));
    if (T > 0) memcpy(cur_tts, tt_slots, (size_t)T * sizeof(int32_t));
    if (num_free > 0) memcpy(pool, free_blocks, (size_t)num_free * sizeof(int32_t));
    int32_t pool_n = num_free;
    for (int32_t r = 0; r < R; ++r) {
        req_status[r] = VTO_NOT_SELECTED;
        req_wave[r] = -1;
        if (req_append_pos) req_append_pos[r] = -1;
    }
    int64_t total_moves = 0;
    wave_move_offsets[0] = 0;

    for (int32_t k = 0; k < num_waves; ++k) {
        vto_counts c;
        /* one planning round against the pool as it stands (Sec. 3.3.2 admission, 3.3.3 planning) */
        if (opts)
            rc = vto_plan_partial(R, S, NB, cur_bto, cur_btb, tt_offsets, cur_tts, keep, select, thr_num, thr_den,
                                  pool, pool_n, opts, nxt_bto, nxt_btb, nxt_tts, freed, status, msrc, mdst, &c, rel);
        else
            rc = vto_plan(R, S, cur_bto, cur_btb, tt_offsets, cur_tts, keep, select, thr_num, thr_den, pool, pool_n,
                          nxt_bto, nxt_btb, nxt_tts, freed, status, msrc, mdst, &c);
        if (rc != VTO_OK) goto done;
        wave_counts[k] = c;
        /* references to shared blocks dropped by this wave's detaches, in wave order (a request that has left
         * its shared blocks no longer lists them, so no reference is dropped twice) */
        for (int32_t i = 0; opts && released_blocks && i < c.num_released; ++i) released_blocks[total_released++] = rel[i];
        /* its copies, in wave order */
        if (total_moves + c.num_moves > move_capacity) {
            rc = VTO_EINVAL;
            goto done;
        }
        for (int32_t m = 0; m < c.num_moves; ++m) {
            move_src[total_moves + m] = msrc[m];
            move_dst[total_moves + m] = mdst[m];
        }
        total_moves += c.num_moves;
        wave_move_offsets[k + 1] = total_moves;
        /* where a request repacked by this wave appends from now on: behind the tokens this wave
         * moved, which fill its destination blocks at the end of its new block list */
        if (req_append_pos) {
            for (int32_t r = 0; r < R; ++r) {
                if (status[r] != VTO_REPACKED) continue;
                int32_t moved = 0;
                for (int64_t t = tt_offsets[r]; t < tt_offsets[r + 1]; ++t)
                    moved += nxt_tts[t] >= 0 && nxt_tts[t] != cur_tts[t];
                const int32_t blocks = nxt_bto[r + 1] - nxt_bto[r];
                req_append_pos[r] = (blocks - ceil_div(moved, S)) * S + moved;
            }
        }
        /* commit: the proposed tables become the state (apply_moves, Sec. 3.2) ... */
        memcpy(cur_bto, nxt_bto, nR * sizeof(int32_t));
        if (nxt_bto[R] > 0) memcpy(cur_btb, nxt_btb, (size_t)nxt_bto[R] * sizeof(int32_t));
        if (T > 0) memcpy(cur_tts, nxt_tts, (size_t)T * sizeof(int32_t));
        for (int32_t r = 0; r < R; ++r) {
            if (status[r] == VTO_REPACKED) {
                req_status[r] = VTO_REPACKED;
                req_wave[r] = k;
            } else if (req_status[r] != VTO_REPACKED) {
                req_status[r] = status[r];
            }
        }
        /* ... and only then do the sources return to the pool (Sec. 3.3.4): the unconsumed part of
         * the pool keeps its order, the reclaimed blocks follow */
        int32_t n = 0;
        for (int32_t i = c.num_free_consumed; i < pool_n; ++i) pool_next[n++] = pool[i];
        for (int32_t i = 0; i < c.num_freed; ++i) pool_next[n++] = freed[i];
        int32_t *tmp = pool;
        pool = pool_next;
        pool_next = tmp;
        pool_n = n;
    }
    memcpy(new_bt_offsets, cur_bto, nR * sizeof(int32_t));
    if (cur_bto[R] > 0) memcpy(new_bt_blocks, cur_btb, (size_t)cur_bto[R] * sizeof(int32_t));
    if (T > 0) memcpy(new_tt_slots, cur_tts, (size_t)T * sizeof(int32_t));
    if (pool_n > 0) memcpy(free_out, pool, (size_t)pool_n * sizeof(int32_t));
    *num_free_out = pool_n;
done:
    free(cur_bto); free(nxt_bto); free(cur_btb); free(nxt_btb); free(cur_tts); free(nxt_tts);
    free(pool); free(pool_next); free(freed); free(status); free(msrc); free(mdst); free(rel);
    return rc;
}

int vto_openmp_threads(void)
{
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}
