"""Pins of the oracle's token-table runtime (evict_token, sync_new_tokens, slot mapping,
apply_moves) against library routines, closed forms and a dictionary-based simulation of a
serving loop (no GPU)."""
import numpy as np
import pytest

from oracle import vto

from runtime_sim import DictCache, ServingState, random_serving_steps


def test_slot_mapping_reduces_to_the_direct_formula_without_eviction():
    """No eviction, no relocation: the token-table lookup equals the direct computation
    slot = block_id * block_size + offset over the block table (Sec. 3.4)."""
    S = 16
    bt = np.array([7, 3, 11, 5], np.int32)
    n = 55
    st = ServingState.empty(S, capacities=[64], block_lists=[bt])
    assert vto.sync_new_tokens(S, st.tt_offsets, st.tt_slots, st.keep, st.tt_len, st.phys_len,
                               st.bt_offsets, st.bt_blocks, [n]) == 0
    slots, ids, off = vto.build_slot_mapping(st.tt_offsets, st.tt_slots, st.keep)
    pos = np.arange(n)
    assert np.array_equal(slots, bt[pos // S] * S + pos % S)
    assert np.array_equal(ids, pos) and off.tolist() == [0, n]
    assert st.tt_len.tolist() == [n] and st.phys_len.tolist() == [n]
    assert (st.tt_slots[n:] == -1).all() and (st.keep[n:] == 0).all()


def test_slot_mapping_is_numpy_boolean_selection():
    rng = np.random.default_rng(0)
    lens = [40, 0, 77, 5]
    off = np.concatenate([[0], np.cumsum(lens)]).astype(np.int32)
    tt = rng.permutation(400)[:off[-1]].astype(np.int32)
    tt[rng.random(off[-1]) < 0.2] = -1
    keep = (rng.random(off[-1]) < 0.6).astype(np.uint8)
    sel = np.array([1, 1, 0, 1], np.uint8)
    slots, ids, o = vto.build_slot_mapping(off, tt, keep, sel)
    live = (tt >= 0) & (keep != 0)
    exp_s, exp_i, exp_o = [], [], [0]
    for r in range(4):
        m = live[off[r]:off[r + 1]] if sel[r] else np.zeros(lens[r], bool)
        exp_s.append(tt[off[r]:off[r + 1]][m])
        exp_i.append(np.flatnonzero(m))
        exp_o.append(exp_o[-1] + int(m.sum()))
    assert np.array_equal(slots, np.concatenate(exp_s)) and np.array_equal(ids, np.concatenate(exp_i))
    assert o.tolist() == exp_o


def test_evict_is_a_scatter_of_zeros_and_skips_bad_victims():
    off = np.array([0, 10, 30], np.int32)
    tt_len = np.array([10, 12], np.int32)
    keep = np.ones(30, np.uint8)
    bad = vto.evict_tokens(off, tt_len, keep, [0, 1, 1, 0, 2, 1, -1], [3, 0, 11, 10, 0, 12, 0])
    exp = np.ones(30, np.uint8)
    exp[[3, 10, 21]] = 0
    assert np.array_equal(keep, exp)
    assert bad == 4          # token 10 of request 0, request 2, token 12 of request 1, request -1


def test_sync_appends_in_batches_and_stops_at_capacity_or_block_list():
    S = 4
    st = ServingState.empty(S, capacities=[10, 6], block_lists=[np.array([2, 9], np.int32), np.array([5], np.int32)])
    assert vto.sync_new_tokens(S, st.tt_offsets, st.tt_slots, st.keep, st.tt_len, st.phys_len,
                               st.bt_offsets, st.bt_blocks, [3, 2]) == 0
    assert vto.sync_new_tokens(S, st.tt_offsets, st.tt_slots, st.keep, st.tt_len, st.phys_len,
                               st.bt_offsets, st.bt_blocks, [7, 2]) == 0       # request 1 unchanged
    assert st.tt_slots[:7].tolist() == [8, 9, 10, 11, 36, 37, 38]
    assert st.tt_slots[10:12].tolist() == [20, 21]
    # request 0 asks for 12 tokens but its block list holds 8 and its table 10; request 1 for 6 with one block
    bad = vto.sync_new_tokens(S, st.tt_offsets, st.tt_slots, st.keep, st.tt_len, st.phys_len,
                              st.bt_offsets, st.bt_blocks, [12, 6])
    assert bad == 2
    assert st.tt_len.tolist() == [8, 4] and st.phys_len.tolist() == [8, 4]
    assert st.tt_slots[7] == 39 and st.tt_slots[8:10].tolist() == [-1, -1]


def test_apply_moves_commits_slots_liveness_and_append_position():
    S = 4
    st = ServingState.empty(S, capacities=[12], block_lists=[np.array([0, 1, 2], np.int32)])
    vto.sync_new_tokens(S, st.tt_offsets, st.tt_slots, st.keep, st.tt_len, st.phys_len, st.bt_offsets,
                        st.bt_blocks, [10])
    vto.evict_tokens(st.tt_offsets, st.tt_len, st.keep, [0] * 7, [0, 2, 3, 5, 6, 7, 9])
    p = vto.plan(S, st.bt_offsets, st.bt_blocks, st.tt_offsets, st.tt_slots, st.keep, np.array([6, 7], np.int32))
    assert p.req_status.tolist() == [vto.REPACKED] and p.num_moves == 3
    vto.apply_moves(st.tt_offsets, st.tt_slots, st.keep, st.phys_len, p.new_tt_slots, p.req_status)
    assert st.tt_slots[:10].tolist() == [-1, 24, -1, -1, 25, -1, -1, -1, 26, -1]
    assert st.keep[:10].tolist() == [0, 1, 0, 0, 1, 0, 0, 0, 1, 0]
    assert st.phys_len.tolist() == [3]
    # the request now owns block 6 only; the next token lands right behind the three survivors
    st.set_block_lists([p.new_bt_blocks])
    vto.sync_new_tokens(S, st.tt_offsets, st.tt_slots, st.keep, st.tt_len, st.phys_len, st.bt_offsets,
                        st.bt_blocks, [11])
    assert st.tt_slots[10] == 27 and st.tt_len.tolist() == [11] and st.phys_len.tolist() == [4]


@pytest.mark.parametrize("seed,S", [(0, 4), (1, 16), (2, 3)])
def test_serving_loop_against_a_dictionary_cache(seed, S):
    """Several decode steps of append -> evict -> slot mapping -> (sometimes) repack + commit on
    the oracle, mirrored by a cache that is just a dict {(request, token id): payload}.  After
    every step the oracle's logical view (slot mapping into the pool) must return exactly the
    payloads the dictionary holds, in token order (token conservation, unique mapping)."""
    rng = np.random.default_rng(seed)
    R = 5
    st = ServingState.random(rng, S, R, capacity=200, num_blocks=400)
    truth = DictCache()
    pool = np.zeros((st.num_blocks * S, 2), np.int64)      # one "layer": payload = (request, token id)
    for step in random_serving_steps(rng, st, steps=25):
        step.run_on_oracle(st, pool, truth)
        slots, ids, off = vto.build_slot_mapping(st.tt_offsets, st.tt_slots, st.keep)
        assert len(np.unique(slots)) == len(slots)                       # unique mapping
        for r in range(R):
            want = truth.live_tokens(r)
            got_ids = ids[off[r]:off[r + 1]].tolist()
            assert got_ids == want
            assert pool[slots[off[r]:off[r + 1]]].tolist() == [[r, t] for t in want]
        # blocks in use are exactly what the block lists say, and nothing is both free and used
        used = set(st.bt_blocks.tolist())
        assert len(used) == len(st.bt_blocks) and not (used & set(st.free))
        live_blocks = set((slots // S).tolist())
        assert live_blocks <= used


# ---- cached slot-translation arrays ---------------------------------------------------------------
def _new_cache(st):
    n = int(st.tt_offsets[-1])
    return dict(dirty=np.zeros(st.R, np.uint8), slots=np.full(n, -77, np.int32), ids=np.full(n, -77, np.int32),
                len=np.zeros(st.R, np.int32), seen=np.zeros(st.R, np.int32))


def _update(st, c):
    return vto.slot_cache_update(st.tt_offsets, st.tt_slots, st.keep, st.tt_len, c["dirty"], c["slots"], c["ids"],
                                 c["len"], c["seen"])


@pytest.mark.parametrize("seed,S", [(0, 4), (1, 16), (2, 3)])
def test_slot_cache_follows_a_serving_loop(seed, S):
    """Marks after evictions and commits, one update per step: every request's cached array must
    equal its slot mapping (a separately pinned routine) and the dictionary's live ids; requests
    that were neither marked nor grown are not touched at all; the numbers of rebuilt / appended
    requests are the ones the test's own bookkeeping predicts."""
    from runtime_sim import Append, Evict, Repack
    rng = np.random.default_rng(seed)
    R = 6
    st = ServingState.random(rng, S, R, capacity=200, num_blocks=500)
    truth = DictCache()
    c = _new_cache(st)
    saw_append_only = saw_rebuild = False
    for step in random_serving_steps(rng, st, steps=30):
        before_len = st.tt_len.copy()
        step.run_on_oracle(st, None, truth)
        touched = set()
        if isinstance(step, Evict):
            vto.slot_cache_mark(c["dirty"], victim_req=step.victim_req)
            touched = {int(r) for r in step.victim_req if 0 <= r < R}
        elif isinstance(step, Repack):
            vto.slot_cache_mark(c["dirty"], req_status=step.last_plan.req_status)
            touched = set(np.flatnonzero(step.last_plan.req_status == vto.REPACKED).tolist())
        assert set(np.flatnonzero(c["dirty"]).tolist()) == touched
        grown = {r for r in range(R) if st.tt_len[r] > c["seen"][r]} - touched
        snapshot = {k: v.copy() for k, v in c.items()}
        nr, na = _update(st, c)
        assert (nr, na) == (len(touched), len(grown)) and not c["dirty"].any()
        saw_append_only |= bool(grown) and isinstance(step, Append)
        saw_rebuild |= bool(touched)
        slots, ids, off = vto.build_slot_mapping(st.tt_offsets, st.tt_slots, st.keep)
        for r in range(R):
            b = int(st.tt_offsets[r])
            n = int(c["len"][r])
            assert c["slots"][b:b + n].tolist() == slots[off[r]:off[r + 1]].tolist()
            assert c["ids"][b:b + n].tolist() == ids[off[r]:off[r + 1]].tolist() == truth.live_tokens(r)
            assert c["seen"][r] == st.tt_len[r]
            if r not in touched and r not in grown:
                e = int(st.tt_offsets[r + 1])
                assert np.array_equal(c["slots"][b:e], snapshot["slots"][b:e])
                assert np.array_equal(c["ids"][b:e], snapshot["ids"][b:e])
            elif r in grown:                    # append-only: the old prefix stays, entries are added behind it
                n0 = int(snapshot["len"][r])
                assert n >= n0 and np.array_equal(c["slots"][b:b + n0], snapshot["slots"][b:b + n0])
    assert saw_append_only and saw_rebuild


def test_slot_cache_is_stale_until_the_change_is_marked():
    """The update must not rebuild on its own: an eviction that nobody marked leaves the cached
    array as it was (that is the point of refreshing only after structural changes), and the mark
    repairs it."""
    S = 4
    st = ServingState.empty(S, capacities=[16], block_lists=[np.array([3, 1, 2], np.int32)])
    vto.sync_new_tokens(S, st.tt_offsets, st.tt_slots, st.keep, st.tt_len, st.phys_len, st.bt_offsets, st.bt_blocks, [9])
    c = _new_cache(st)
    assert _update(st, c) == (0, 1)
    assert c["slots"][:9].tolist() == [12, 13, 14, 15, 4, 5, 6, 7, 8] and c["len"].tolist() == [9]
    vto.evict_tokens(st.tt_offsets, st.tt_len, st.keep, [0, 0], [1, 6])
    assert _update(st, c) == (0, 0) and c["len"].tolist() == [9]          # unmarked: untouched
    vto.sync_new_tokens(S, st.tt_offsets, st.tt_slots, st.keep, st.tt_len, st.phys_len, st.bt_offsets, st.bt_blocks, [11])
    assert _update(st, c) == (0, 1)
    assert c["slots"][:11].tolist() == [12, 13, 14, 15, 4, 5, 6, 7, 8, 9, 10]   # appended behind the stale entries
    vto.slot_cache_mark(c["dirty"], victim_req=[0, 0, 5, -1])                   # out-of-range requests are skipped
    assert _update(st, c) == (1, 0)
    assert c["slots"][:9].tolist() == [12, 14, 15, 4, 5, 7, 8, 9, 10] and c["len"].tolist() == [9]
    assert c["ids"][:9].tolist() == [0, 2, 3, 4, 5, 7, 8, 9, 10] and c["seen"].tolist() == [11]


PARTIAL_MIX = (None, dict(util=(1, 1)), dict(util=(1, 2)), dict(util=(3, 4), max_source_blocks=3), dict())


@pytest.mark.parametrize("seed,S,wave_options", [(3, 4, ()), (4, 16, ()), (5, 3, ()), (6, 4, (0, 2, 3, 4)),
                                                 (7, 8, (2, 3, 5)), (8, 3, (0, 3, 4)), (9, 4, (3, 4))])
def test_serving_loop_with_partial_plans_against_a_dictionary_cache(seed, S, wave_options):
    """The same loop with the partial planner in the mix (blocks that stay, a source bound), as
    single plans and as repacks in waves: the commit must put the append position behind the moved
    tokens -- blocks that stayed may have holes, and after several waves a partly filled
    destination block of an early wave may sit in the middle of the list -- or new tokens
    overwrite live ones."""
    rng = np.random.default_rng(seed)
    R = 5
    st = ServingState.random(rng, S, R, capacity=260, num_blocks=600)
    truth = DictCache()
    pool = np.zeros((st.num_blocks * S, 2), np.int64)
    kinds = set()
    for step in random_serving_steps(rng, st, steps=36, partial_options=PARTIAL_MIX, wave_options=wave_options):
        step.run_on_oracle(st, pool, truth)
        if hasattr(step, "partial") and len(step.last_plan.move_src):
            kinds.add((step.waves > 0, None if step.partial is None else tuple(sorted(step.partial))))
        slots, ids, off = vto.build_slot_mapping(st.tt_offsets, st.tt_slots, st.keep)
        assert len(np.unique(slots)) == len(slots)
        for r in range(R):
            want = truth.live_tokens(r)
            assert ids[off[r]:off[r + 1]].tolist() == want
            assert pool[slots[off[r]:off[r + 1]]].tolist() == [[r, t] for t in want]
        used = set(st.bt_blocks.tolist())
        assert len(used) == len(st.bt_blocks) and not (used & set(st.free))
        assert set((slots // S).tolist()) <= used
        assert vto.check_tables(S, st.num_blocks, st.bt_offsets, st.bt_blocks, st.tt_offsets, st.tt_slots,
                                np.asarray(st.free, np.int32)) == 0
    assert len(kinds) >= 2


def test_append_position_after_a_partial_plan():
    """Hand case, S = 4: blocks [A full, B 1 of 4 live, C 3 of 4 live, D 2 of 4 (tail, 2 written)];
    sources = blocks under 100 % utilisation = B, C, D -> 6 moved tokens -> 2 destinations.  New list
    [A, X, Y]; the next token lands at position 1*4 + 6 = 10, i.e. offset 2 of Y."""
    S = 4
    st = ServingState.empty(S, capacities=[20], block_lists=[np.array([10, 11, 12, 13], np.int32)], num_blocks=20)
    vto.sync_new_tokens(S, st.tt_offsets, st.tt_slots, st.keep, st.tt_len, st.phys_len, st.bt_offsets, st.bt_blocks, [14])
    vto.evict_tokens(st.tt_offsets, st.tt_len, st.keep, [0] * 4, [4, 5, 6, 9])
    p = vto.plan_partial(S, 20, st.bt_offsets, st.bt_blocks, st.tt_offsets, st.tt_slots, st.keep,
                         np.array([2, 3, 5], np.int32), util=(1, 1))
    assert p.req_status.tolist() == [vto.REPACKED] and p.num_moves == 6 and p.new_bt_blocks.tolist() == [10, 2, 3]
    vto.apply_moves(st.tt_offsets, st.tt_slots, st.keep, st.phys_len, p.new_tt_slots, p.req_status, S=S,
                    new_bt_offsets=p.new_bt_offsets)
    assert st.phys_len.tolist() == [10]
    st.set_block_lists([p.new_bt_blocks])
    vto.sync_new_tokens(S, st.tt_offsets, st.tt_slots, st.keep, st.tt_len, st.phys_len, st.bt_offsets, st.bt_blocks, [15])
    assert st.tt_slots[14] == 3 * S + 2 and st.phys_len.tolist() == [11]
    # without the block table the old rule counts live entries: the same number only when nothing stayed
    whole = ServingState.empty(S, capacities=[20], block_lists=[np.array([10, 11, 12, 13], np.int32)], num_blocks=20)
    vto.sync_new_tokens(S, whole.tt_offsets, whole.tt_slots, whole.keep, whole.tt_len, whole.phys_len,
                        whole.bt_offsets, whole.bt_blocks, [14])
    vto.evict_tokens(whole.tt_offsets, whole.tt_len, whole.keep, [0] * 4, [4, 5, 6, 9])
    q = vto.plan(S, whole.bt_offsets, whole.bt_blocks, whole.tt_offsets, whole.tt_slots, whole.keep,
                 np.array([2, 3, 5], np.int32))
    a, b = whole.phys_len.copy(), whole.phys_len.copy()
    tt1, k1 = whole.tt_slots.copy(), whole.keep.copy()
    vto.apply_moves(whole.tt_offsets, tt1, k1, a, q.new_tt_slots, q.req_status)
    tt2, k2 = whole.tt_slots.copy(), whole.keep.copy()
    vto.apply_moves(whole.tt_offsets, tt2, k2, b, q.new_tt_slots, q.req_status, S=S, new_bt_offsets=q.new_bt_offsets)
    assert a.tolist() == b.tolist() == [10]


# ---- per-block liveness kept current by the runtime interfaces --------------------------------------
@pytest.mark.parametrize("seed,S", [(10, 4), (11, 16), (12, 3)])
def test_incremental_block_liveness_equals_the_recount(seed, S):
    """n_b and the live total maintained by the counted evict / append interfaces (recounted only
    after repacks) must equal vto_block_liveness -- itself pinned by numpy.bincount -- after every
    step of a serving loop whose victim batches contain repeats and already evicted tokens."""
    rng = np.random.default_rng(seed)
    R = 5
    st = ServingState.random(rng, S, R, capacity=260, num_blocks=600)
    st.enable_counters()
    changed_without_repack = 0
    for step in random_serving_steps(rng, st, steps=36, partial_options=PARTIAL_MIX, wave_options=(0, 0, 3)):
        before = st.counters["n_b"].copy()
        step.run_on_oracle(st, None, None)
        n_b, _, live, _ = vto.block_liveness(S, st.num_blocks, st.bt_offsets, st.bt_blocks, st.tt_offsets,
                                             st.tt_slots, st.keep)
        assert np.array_equal(st.counters["n_b"], n_b) and st.counters["live"][0] == live
        if not hasattr(step, "partial"):
            changed_without_repack += int(not np.array_equal(before, n_b))
    assert changed_without_repack >= 10


def test_counted_eviction_counts_a_token_once():
    S = 4
    st = ServingState.empty(S, capacities=[12, 8], block_lists=[np.array([3, 1], np.int32), np.array([5], np.int32)],
                            num_blocks=8)
    st.enable_counters()
    vto.sync_new_tokens_counted(S, st.tt_offsets, st.tt_slots, st.keep, st.tt_len, st.phys_len, st.bt_offsets,
                                st.bt_blocks, [7, 3], st.counters["n_b"], st.counters["live"])
    assert st.counters["n_b"].tolist() == [0, 3, 0, 4, 0, 3, 0, 0] and st.counters["live"][0] == 10
    # token (0, 1) twice in one batch, (0, 5) once, two victims out of range
    bad = vto.evict_tokens_counted(S, st.tt_offsets, st.tt_len, st.tt_slots, st.keep, [0, 0, 0, 0, 2], [1, 1, 5, 7, 0],
                                   st.counters["n_b"], st.counters["live"])
    assert bad == 2 and st.counters["n_b"].tolist() == [0, 2, 0, 3, 0, 3, 0, 0] and st.counters["live"][0] == 8
    # evicting them again changes nothing
    vto.evict_tokens_counted(S, st.tt_offsets, st.tt_len, st.tt_slots, st.keep, [0, 0], [1, 5], st.counters["n_b"],
                             st.counters["live"])
    assert st.counters["n_b"].tolist() == [0, 2, 0, 3, 0, 3, 0, 0] and st.counters["live"][0] == 8
    assert st.keep[:7].tolist() == [1, 0, 1, 1, 1, 0, 1]
