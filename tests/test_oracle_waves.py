"""Pins of the oracle's repack in waves, where blocks reclaimed by one wave are the destinations
of the next (no GPU).

Nothing here retypes the oracle's loop: the wave index of every request is predicted from block
arithmetic alone, the physical effect is replayed on a dictionary cache {slot: (request, token)}
wave by wave with the definition twin, and single waves reduce to the one-shot planner."""
import itertools
from fractions import Fraction

import numpy as np
import pytest

from definition_twin import repack_definition, repack_partial_definition
from oracle import vto
from harness import workloads as wl


def workloads():
    yield wl.tiny(seed=0)
    yield wl.llama8b_h2o(seed=1, requests=5, lo=100, hi=400, layers=1, heads=1, head_dim=8)
    yield wl.mistral7b_random(seed=2, requests=9, lo=20, hi=200, layers=1, heads=1, head_dim=8)
    yield wl.steady_state(seed=4, requests=12, lo=100, hi=600, layers=1, heads=1, head_dim=8)
    yield wl.longctx_scissor(seed=3, requests=3, lo=900, hi=1500, layers=1, heads=1, head_dim=8)
    yield wl.streaming_window(seed=6, requests=6, lo=60, hi=400, window=48, layers=1, heads=1, head_dim=8)


def waves(w, free, num_waves, partial=None):
    return vto.plan_waves(w.block_size, w.num_blocks, w.bt_offsets, w.bt_blocks, w.tt_offsets, w.tt_slots, w.keep,
                          free, num_waves, w.select, w.thr_num, w.thr_den, partial)


def per_request(w):
    """(live tokens, blocks, candidate?) of every request from the inputs alone."""
    S = w.block_size
    live = (w.tt_slots >= 0) & (w.keep != 0)
    out = []
    for r in range(w.num_requests):
        n = int(live[w.tt_offsets[r]:w.tt_offsets[r + 1]].sum())
        nb = int(w.bt_offsets[r + 1] - w.bt_offsets[r])
        sel = w.select is None or bool(w.select[r])
        if sel and w.thr_den:
            sel = nb > 0 and Fraction(n, nb * S) < Fraction(w.thr_num, w.thr_den)
        out.append((n, nb, sel and -(-n // S) < nb))
    return out


@pytest.mark.parametrize("w", list(workloads()), ids=lambda w: w.name)
def test_one_wave_is_the_one_shot_plan(w):
    for nf in (0, 3, len(w.free_blocks)):
        free = w.free_blocks[:nf]
        p = vto.plan_workload(w, num_free=nf)
        v = waves(w, free, 1)
        assert np.array_equal(v.new_bt_offsets, p.new_bt_offsets) and np.array_equal(v.new_bt_blocks, p.new_bt_blocks)
        assert np.array_equal(v.new_tt_slots, p.new_tt_slots) and np.array_equal(v.req_status, p.req_status)
        assert np.array_equal(v.move_src, p.move_src) and np.array_equal(v.move_dst, p.move_dst)
        assert v.free_out.tolist() == free[p.num_free_consumed:].tolist() + p.freed_blocks.tolist()
        assert np.array_equal(v.req_wave, np.where(p.req_status == vto.REPACKED, 0, -1))


@pytest.mark.parametrize("w", list(workloads()), ids=lambda w: w.name)
def test_wave_of_every_request_follows_from_block_arithmetic(w):
    """Pool size after a wave = size before + sum over admitted (blocks - ceil(n/S)); a wave admits
    the longest prefix of the still pending candidates whose cumulative ceil(n/S) fits the pool."""
    S = w.block_size
    facts = per_request(w)
    cands = [r for r, (_, _, c) in enumerate(facts) if c]
    biggest = max((-(-facts[r][0] // S) for r in cands), default=0)
    for nf in sorted({0, 1, biggest - 1, biggest, biggest + 3, 2 * biggest}):
        if nf < 0 or nf > len(w.free_blocks):
            continue
        W = 6
        v = waves(w, w.free_blocks[:nf], W)
        pool, pending, expect = nf, list(cands), {}
        for k in range(W):
            cum, admitted = 0, []
            for r in pending:
                cum += -(-facts[r][0] // S)
                if cum > pool:
                    break
                admitted.append(r)
            for r in admitted:
                expect[r] = k
                pool += facts[r][1] - -(-facts[r][0] // S)        # its blocks come back, its demand is consumed
            pending = pending[len(admitted):]
            assert v.wave_counts[k]["num_admitted"] == len(admitted)
            assert v.wave_counts[k]["num_deferred"] == len(pending)
        assert len(v.free_out) == pool
        for r in range(w.num_requests):
            assert v.req_wave[r] == expect.get(r, -1)
            assert (v.req_status[r] == vto.REPACKED) == (r in expect)
            if r in pending:
                assert v.req_status[r] == vto.DEFERRED_NO_FREE


@pytest.mark.parametrize("w", list(workloads()), ids=lambda w: w.name)
def test_headroom_of_the_largest_request_is_enough(w):
    """With a pool as large as the largest single demand and one wave per candidate, every
    candidate is repacked and ends with ceil(n/S) blocks -- the result a one-shot plan needs the
    SUM of all demands for."""
    S = w.block_size
    facts = per_request(w)
    cands = [r for r, (_, _, c) in enumerate(facts) if c]
    if not cands:
        pytest.skip("no candidate")
    biggest = max(-(-facts[r][0] // S) for r in cands)
    total = sum(-(-facts[r][0] // S) for r in cands)
    v = waves(w, w.free_blocks[:biggest], len(cands))
    one_shot = vto.plan_workload(w, num_free=total)
    assert np.array_equal(v.req_status, one_shot.req_status)
    assert np.array_equal(np.diff(v.new_bt_offsets), np.diff(one_shot.new_bt_offsets))
    assert len(v.move_src) == one_shot.num_moves
    assert len(v.free_out) == biggest + one_shot.num_freed - one_shot.num_dst_blocks
    if biggest < total:
        short = vto.plan_workload(w, num_free=biggest)
        assert short.num_admitted < len(cands)          # the same pool does not serve a single wave


def replay_on_cache(w, free, num_waves, twin, **twin_kw):
    """Dictionary cache {slot: (r, t)}; every wave planned by the definition twin and executed by
    moving payloads; returns the final state."""
    S, R = w.block_size, w.num_requests
    bt = [w.bt_blocks[w.bt_offsets[r]:w.bt_offsets[r + 1]].tolist() for r in range(R)]
    tt = [w.tt_slots[w.tt_offsets[r]:w.tt_offsets[r + 1]].tolist() for r in range(R)]
    keeps = [w.keep[w.tt_offsets[r]:w.tt_offsets[r + 1]].tolist() for r in range(R)]
    cache = {s: (r, t) for r in range(R) for t, s in enumerate(tt[r]) if s >= 0}
    pool = list(free)
    status, wave = [0] * R, [-1] * R
    for k in range(num_waves):
        d = twin(S, bt, tt, keeps, pool, **twin_kw)
        for src, dst in d["moves"]:
            cache[dst] = cache[src]
        for r in range(R):
            if d["status"][r] == 1:
                status[r], wave[r] = 1, k
            elif status[r] != 1:
                status[r] = d["status"][r]
        bt, tt = d["new_bt"], d["new_tt"]
        pool = pool[d["consumed"]:] + d["freed"]
    return bt, tt, pool, status, wave, cache, keeps


def check_against_replay(w, v, free_in, replay):
    bt, tt, pool, status, wave, cache, keeps = replay
    R = w.num_requests
    for r in range(R):
        assert v.new_bt_blocks[v.new_bt_offsets[r]:v.new_bt_offsets[r + 1]].tolist() == bt[r]
        assert v.new_tt_slots[w.tt_offsets[r]:w.tt_offsets[r + 1]].tolist() == tt[r]
    assert v.free_out.tolist() == pool and v.req_status.tolist() == status and v.req_wave.tolist() == wave
    # the oracle's move list, applied in its order to the same cache, shows every live token its own payload
    mine = {s: (r, t) for r in range(R) for t, s in enumerate(w.tt_slots[w.tt_offsets[r]:w.tt_offsets[r + 1]].tolist())
            if s >= 0}
    for s, d in zip(v.move_src.tolist(), v.move_dst.tolist()):
        mine[d] = mine[s]
    seen = set()
    for r in range(R):
        for t, s in enumerate(tt[r]):
            if s >= 0:
                assert keeps[r][t] and mine[s] == (r, t) and cache[s] == (r, t) and s not in seen
                seen.add(s)
    # block conservation: tables and pool partition the blocks that tables and pool held before
    after = [b for r in range(R) for b in bt[r]] + pool
    before = w.bt_blocks.tolist() + list(free_in)
    assert sorted(after) == sorted(before) and len(set(after)) == len(after)



@pytest.mark.parametrize("w", list(workloads()), ids=lambda w: w.name)
@pytest.mark.parametrize("nf_frac", [0.0, 0.1, 0.35, 1.0])
def test_waves_against_a_dictionary_cache_replay(w, nf_frac):
    need_total = vto.plan_workload(w).num_dst_blocks
    nf = int(round(nf_frac * need_total))
    free = w.free_blocks[:nf]
    thr = Fraction(w.thr_num, w.thr_den) if w.thr_den else None
    sel = None if w.select is None else w.select.tolist()
    v = waves(w, free, 4)
    check_against_replay(w, v, free.tolist(), replay_on_cache(w, free.tolist(), 4, repack_definition, select=sel, thr=thr))


@pytest.mark.parametrize("w", list(workloads()), ids=lambda w: w.name)
def test_partial_waves_with_a_source_bound_walk_through_the_request(w):
    """B sources per request and wave: a request is repacked in several waves, B blocks at a time."""
    need_total = vto.plan_workload(w).num_dst_blocks
    free = w.free_blocks[:max(2, need_total // 5)]
    thr = Fraction(w.thr_num, w.thr_den) if w.thr_den else None
    sel = None if w.select is None else w.select.tolist()
    opts = dict(util=(1, 1), max_source_blocks=4)
    v = waves(w, free, 5, partial=opts)
    check_against_replay(w, v, free.tolist(), replay_on_cache(w, free.tolist(), 5, repack_partial_definition, select=sel, thr=thr,
                                               util=Fraction(1, 1), max_sources=4))
    assert any(c["num_admitted"] for c in v.wave_counts[1:]) or v.wave_counts[0]["num_admitted"] == 0


def test_every_mask_of_two_small_requests_every_pool_size():
    """Brute force: 2 requests x 6 tokens, S = 2, every keep mask, every pool size 0..6, 3 waves."""
    S, n_tok = 2, 6
    bt = [[5, 1, 7], [2, 9, 0]]
    free_all = [3, 8, 4, 6, 10, 11]
    tt = [[b * S + o for b in blocks for o in range(S)] for blocks in bt]

    class W:
        pass
    for m0, m1 in itertools.product(range(1 << n_tok), repeat=2):
        if (m0 * 7 + m1 * 13) % 5:        # a fifth of the 4096 mask pairs keeps the test quick
            continue
        keeps = [[(m >> t) & 1 for t in range(n_tok)] for m in (m0, m1)]
        w = W()
        w.block_size, w.num_blocks, w.num_requests = S, 12, 2
        w.bt_offsets = np.array([0, 3, 6], np.int32)
        w.bt_blocks = np.array(bt[0] + bt[1], np.int32)
        w.tt_offsets = np.array([0, n_tok, 2 * n_tok], np.int32)
        w.tt_slots = np.array(tt[0] + tt[1], np.int32)
        w.keep = np.array(keeps[0] + keeps[1], np.uint8)
        w.select, w.thr_num, w.thr_den = None, 0, 0
        for nf in range(0, 7):
            free = np.array(free_all[:nf], np.int32)
            v = waves(w, free, 3)
            check_against_replay(w, v, free.tolist(), replay_on_cache(w, free.tolist(), 3, repack_definition))


def test_move_list_order_matters_when_blocks_are_reused():
    """The waves' lists overlap (a destination of wave 1 is a source of wave 0), so applying them out
    of order corrupts the view -- the reason the copies of consecutive waves are ordered."""
    w = wl.mistral7b_random(seed=5, requests=6, lo=80, hi=160, layers=1, heads=1, head_dim=8)
    need = [int(x) for x in np.diff(vto.plan_workload(w).new_bt_offsets)]
    free = w.free_blocks[:max(need)]
    v = waves(w, free, 6)
    o = v.wave_move_offsets
    assert (np.diff(o) > 0).sum() >= 2
    reused = set((v.move_dst[o[1]:] // w.block_size).tolist()) & set((v.move_src[:o[1]] // w.block_size).tolist())
    assert reused, "a later wave writes into blocks wave 0 has evacuated"
    rows = np.arange(w.num_blocks * w.block_size, dtype=np.int64).reshape(-1, 1).copy()
    good = rows.copy()
    vto.apply_moves_slab(good, v.move_src, v.move_dst)
    live = v.new_tt_slots >= 0
    assert np.array_equal(good[v.new_tt_slots[live], 0], w.tt_slots[live])      # row content = original slot
    bad = rows.copy()
    order = np.concatenate([np.arange(o[1], o[-1]), np.arange(0, o[1])])       # wave 0 last
    vto.apply_moves_slab(bad, v.move_src[order], v.move_dst[order])
    assert not np.array_equal(bad[v.new_tt_slots[live], 0], w.tt_slots[live])


@pytest.mark.parametrize("degree", [1, 2, 4])
@pytest.mark.parametrize("detach", [Fraction(1, 1), Fraction(1, 2), Fraction(1, 8)])
@pytest.mark.parametrize("rule", [0, 1, 2])
def test_waves_with_copy_on_write_detach_against_a_replay(degree, detach, rule):
    """Repack in waves on the shared-prefix workload with a detach threshold: wave by wave the definition
    twin plans on what the previous wave committed; tables, pool, statuses and the list of dropped
    references (wave after wave, each reference once) must be the oracle's, one wave must equal the single
    partial plan, and every request must still see exactly its own payloads -- shared blocks keep their
    bytes for the sharers that stayed.  All three forms of the rule: all protected blocks of a request at
    once, block by block on its own tokens, block by block on all holders' tokens (later waves then see
    requests that still hold part of their prefix)."""
    w, protect = wl.shared_prefix(seed=3, groups=2, degree=degree, prefix_len=48, suffix_len=150, layers=1, heads=1,
                                  head_dim=8, block_size=4)
    S, R = w.block_size, w.num_requests
    prot = set(np.flatnonzero(protect).tolist())
    opts = dict(protect=protect, util=(1, 1), max_source_blocks=6, detach=(detach.numerator, detach.denominator),
                detach_rule=rule)
    twin_kw = dict(protect=prot, util=Fraction(1, 1), max_sources=6, detach=detach, detach_rule=rule)
    one = vto.plan_partial(S, w.num_blocks, w.bt_offsets, w.bt_blocks, w.tt_offsets, w.tt_slots, w.keep,
                           w.free_blocks, **opts)
    v1 = vto.plan_waves(S, w.num_blocks, w.bt_offsets, w.bt_blocks, w.tt_offsets, w.tt_slots, w.keep, w.free_blocks, 1,
                        partial=opts)
    assert np.array_equal(v1.new_tt_slots, one.new_tt_slots) and np.array_equal(v1.new_bt_blocks, one.new_bt_blocks)
    assert np.array_equal(v1.released_blocks, one.released_blocks) and v1.wave_counts[0]["num_released"] == len(one.released_blocks)

    need = vto.plan_partial(S, w.num_blocks, w.bt_offsets, w.bt_blocks, w.tt_offsets, w.tt_slots, w.keep,
                            w.free_blocks, **opts).num_dst_blocks
    for nf in sorted({max(1, need // 5), max(2, need // 2), need}):
        free = w.free_blocks[:nf].tolist()
        v = vto.plan_waves(S, w.num_blocks, w.bt_offsets, w.bt_blocks, w.tt_offsets, w.tt_slots, w.keep, free, 5,
                           partial=opts)
        # the replay: dictionary of slot contents (a slot's content is named by the slot it was filled in)
        bt = [w.bt_blocks[w.bt_offsets[r]:w.bt_offsets[r + 1]].tolist() for r in range(R)]
        tt = [w.tt_slots[w.tt_offsets[r]:w.tt_offsets[r + 1]].tolist() for r in range(R)]
        keeps = [w.keep[w.tt_offsets[r]:w.tt_offsets[r + 1]].tolist() for r in range(R)]
        content = {s: s for s in range(w.slots_per_layer)}
        pool, released, status = list(free), [], [0] * R
        per_wave = []
        for k in range(5):
            d = repack_partial_definition(S, bt, tt, keeps, pool, **twin_kw)
            for src, dst in d["moves"]:
                content[dst] = content[src]
            for r in range(R):
                status[r] = 1 if d["status"][r] == 1 else (status[r] if status[r] == 1 else d["status"][r])
            bt, tt = d["new_bt"], d["new_tt"]
            pool = pool[d["consumed"]:] + d["freed"]
            released += d["released"]
            per_wave.append(len(d["released"]))
        for r in range(R):
            assert v.new_bt_blocks[v.new_bt_offsets[r]:v.new_bt_offsets[r + 1]].tolist() == bt[r]
            assert v.new_tt_slots[w.tt_offsets[r]:w.tt_offsets[r + 1]].tolist() == tt[r]
        assert v.free_out.tolist() == pool and v.req_status.tolist() == status
        assert v.released_blocks.tolist() == released
        assert [c["num_released"] for c in v.wave_counts] == per_wave
        # the oracle's own move list, in its order, leaves every live token with the content of its old slot
        mine = {s: s for s in range(w.slots_per_layer)}
        for s, dd in zip(v.move_src.tolist(), v.move_dst.tolist()):
            mine[dd] = mine[s]
        for r in range(R):
            old = w.tt_slots[w.tt_offsets[r]:w.tt_offsets[r + 1]].tolist()
            for t, s in enumerate(tt[r]):
                if s >= 0:
                    assert keeps[r][t] and mine[s] == old[t] and content[s] == old[t]
        # a reference is dropped at most once per request and block, and only to protected blocks
        assert all(b in prot for b in released)
        if detach == Fraction(1, 1) and nf == need:
            assert released, "with this threshold and a full pool some request leaves its prefix"
        # shared blocks are never reclaimed nor handed out
        assert not (set(pool) & prot)
