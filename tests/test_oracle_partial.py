"""Pins of the oracle's eligibility metadata (per-block liveness, F) and of partial plans that
evacuate only low-utilisation, unprotected blocks (no GPU)."""
import itertools
from fractions import Fraction

import numpy as np
import pytest

from definition_twin import repack_partial_definition, to_csr
from oracle import vto
from harness import workloads as wl


def workloads():
    yield wl.tiny(seed=0)
    yield wl.llama8b_h2o(seed=1, requests=5, lo=100, hi=400, layers=1, heads=1, head_dim=8)
    yield wl.mistral7b_random(seed=2, requests=9, lo=20, hi=200, layers=1, heads=1, head_dim=8)
    yield wl.steady_state(seed=4, requests=12, lo=100, hi=600, layers=1, heads=1, head_dim=8)
    yield wl.longctx_scissor(seed=3, requests=3, lo=900, hi=1500, layers=1, heads=1, head_dim=8)
    yield wl.streaming_window(seed=6, requests=6, lo=60, hi=400, window=48, layers=1, heads=1, head_dim=8)


def plan_p(w, **kw):
    return vto.plan_partial(w.block_size, w.num_blocks, w.bt_offsets, w.bt_blocks, w.tt_offsets, w.tt_slots, w.keep,
                            w.free_blocks, w.select, w.thr_num, w.thr_den, **kw)


def same_plan(a, b):
    return all(np.array_equal(getattr(a, f), getattr(b, f)) for f in
               ("new_bt_offsets", "new_bt_blocks", "new_tt_slots", "freed_blocks", "req_status", "move_src", "move_dst")) \
        and (a.num_moves, a.num_free_consumed, a.num_freed, a.num_admitted, a.num_deferred) == \
            (b.num_moves, b.num_free_consumed, b.num_freed, b.num_admitted, b.num_deferred)


@pytest.mark.parametrize("w", list(workloads()), ids=lambda w: w.name)
def test_block_liveness_is_a_bincount_and_F_matches(w):
    S = w.block_size
    n_b, hist, live, alloc = vto.block_liveness(S, w.num_blocks, w.bt_offsets, w.bt_blocks, w.tt_offsets, w.tt_slots, w.keep)
    is_live = (w.tt_slots >= 0) & (w.keep != 0)
    assert np.array_equal(n_b, np.bincount(w.tt_slots[is_live] // S, minlength=w.num_blocks))
    assert np.array_equal(hist, np.bincount(n_b[w.bt_blocks], minlength=S + 1))
    assert live == int(is_live.sum()) and alloc == len(w.bt_blocks) and hist.sum() == alloc
    # F = 1 - (1/N) sum u_b over allocated blocks (Sec. 2.3.1), and the oracle's own waste ratio
    F = 1 - live / (alloc * S)
    assert F == pytest.approx(1 - np.mean(n_b[w.bt_blocks] / S))
    assert F == pytest.approx(vto.waste_ratio(S, alloc, w.tt_slots, w.keep))


@pytest.mark.parametrize("w", list(workloads()), ids=lambda w: w.name)
def test_default_options_reduce_to_whole_request_plan(w):
    assert same_plan(plan_p(w), vto.plan_workload(w))
    for c in (0, 1, 5):
        assert same_plan(plan_p(w, num_free=c), vto.plan_workload(w, num_free=c))


@pytest.mark.parametrize("w", list(workloads()), ids=lambda w: w.name)
def test_keeping_full_blocks_gives_the_same_block_count_with_fewer_moves(w):
    """Sources = blocks that are not fully live (n_b < S).  Block demand f + ceil(p / S) equals
    ceil((f*S + p) / S): the packed footprint of Sec. 5's block arithmetic, reached with p moves
    instead of f*S + p."""
    S = w.block_size
    whole = vto.plan_workload(w)
    part = plan_p(w, util=(1, 1))
    n_b, _, _, _ = vto.block_liveness(S, w.num_blocks, w.bt_offsets, w.bt_blocks, w.tt_offsets, w.tt_slots, w.keep)
    live = (w.tt_slots >= 0) & (w.keep != 0)
    moves = 0
    for r in range(w.num_requests):
        blocks = w.bt_blocks[w.bt_offsets[r]:w.bt_offsets[r + 1]]
        full = int((n_b[blocks] == S).sum())
        n = int(live[w.tt_offsets[r]:w.tt_offsets[r + 1]].sum())
        p = n - full * S
        after = part.new_bt_offsets[r + 1] - part.new_bt_offsets[r]
        if part.req_status[r] == vto.REPACKED:
            assert after == full + -(-p // S) == -(-n // S)
            moves += p
            if whole.req_status[r] == vto.REPACKED:
                assert after == whole.new_bt_offsets[r + 1] - whole.new_bt_offsets[r]
            # fully live blocks stay where they are, in their old order, ahead of the destinations
            kept = [b for b in blocks if n_b[b] == S]
            assert part.new_bt_blocks[part.new_bt_offsets[r]:part.new_bt_offsets[r] + full].tolist() == kept
    assert part.num_moves == moves <= whole.num_moves or part.num_admitted != whole.num_admitted
    # token conservation and unique mapping still hold
    assert np.array_equal(part.new_tt_slots >= 0, live)
    occ = part.new_tt_slots[part.new_tt_slots >= 0]
    assert len(np.unique(occ)) == len(occ)
    assert not (set(part.move_src.tolist()) & set(part.move_dst.tolist()))


def test_protected_blocks_never_move_or_get_reclaimed():
    """Shared-prefix blocks are excluded from plans (I4); here: the first blocks of every request."""
    w = wl.mistral7b_random(seed=6, requests=6, lo=80, hi=200, layers=1, heads=1, head_dim=8, block_size=4)
    protect = np.zeros(w.num_blocks, np.uint8)
    prefix = []
    for r in range(w.num_requests):
        blocks = w.bt_blocks[w.bt_offsets[r]:w.bt_offsets[r + 1]]
        prefix += blocks[:5].tolist()
    protect[prefix] = 1
    p = plan_p(w, protect=protect)
    assert p.num_admitted > 0
    assert not (set(p.freed_blocks.tolist()) & set(prefix))
    assert not (set((p.move_src // w.block_size).tolist()) & set(prefix))
    for r in range(w.num_requests):
        blocks = w.bt_blocks[w.bt_offsets[r]:w.bt_offsets[r + 1]]
        assert p.new_bt_blocks[p.new_bt_offsets[r]:p.new_bt_offsets[r] + 5].tolist() == blocks[:5].tolist()
    live = (w.tt_slots >= 0) & (w.keep != 0)
    in_prefix = np.isin(w.tt_slots // w.block_size, prefix) & live
    assert np.array_equal(p.new_tt_slots[in_prefix], w.tt_slots[in_prefix])
    # everything protected: nothing can be gained
    q = plan_p(w, protect=np.ones(w.num_blocks, np.uint8))
    assert q.num_moves == 0 and set(q.req_status.tolist()) <= {vto.NO_GAIN}


def test_global_trigger_threshold_is_strict_and_exact():
    S = 4
    bt = np.arange(4, dtype=np.int32)
    tt = np.arange(16, dtype=np.int32)
    keep = np.zeros(16, np.uint8)
    keep[[0, 4, 8, 12]] = 1                                 # F = 1 - 4/16 = 3/4 exactly
    free = np.array([10, 11], np.int32)
    args = (S, 12, [0, 4], bt, [0, 16], tt, keep, free)
    assert vto.plan_partial(*args, theta=(3, 4)).req_status.tolist() == [vto.NOT_SELECTED]      # F > 3/4 is false
    assert vto.plan_partial(*args, theta=(74, 100)).req_status.tolist() == [vto.REPACKED]
    assert vto.plan_partial(*args, theta=(1, 4)).req_status.tolist() == [vto.REPACKED]          # the paper's default 0.25


def test_source_bound_B_takes_the_first_eligible_blocks_in_table_order():
    S = 4
    bt = np.array([3, 0, 2, 1, 5], np.int32)
    tt = (bt[np.arange(20) // S] * S + np.arange(20) % S).astype(np.int32)
    keep = np.zeros(20, np.uint8)
    keep[[0, 5, 9, 14, 17]] = 1                             # one survivor per block
    free = np.array([8, 9], np.int32)
    p = vto.plan_partial(S, 10, [0, 5], bt, [0, 20], tt, keep, free, max_source_blocks=3)
    assert p.freed_blocks.tolist() == [3, 0, 2] and p.num_free_consumed == 1
    assert p.new_bt_blocks.tolist() == [1, 5, 8]
    assert p.new_tt_slots[[0, 5, 9]].tolist() == [32, 33, 34] and p.new_tt_slots[[14, 17]].tolist() == tt[[14, 17]].tolist()
    # B = 1: one source block cannot release more than the one destination it needs
    assert vto.plan_partial(S, 10, [0, 5], bt, [0, 20], tt, keep, free, max_source_blocks=1).req_status.tolist() == [vto.NO_GAIN]


def _compare(S, bts, tts, keeps, free, select, thr, protect, util, B, theta, NB, detach=None, rule=0):
    bt_off, bt_flat = to_csr(bts)
    tt_off, tt_flat = to_csr(tts)
    _, keep_flat = to_csr(keeps)
    prot = np.zeros(NB, np.uint8)
    prot[list(protect)] = 1
    fr = lambda f: (f.numerator, f.denominator) if f is not None else (0, 0)
    p = vto.plan_partial(S, NB, bt_off, bt_flat, tt_off, tt_flat, keep_flat, free,
                         select=None if select is None else np.array(select, np.uint8),
                         thr_num=fr(thr)[0], thr_den=fr(thr)[1], protect=prot if protect else None,
                         util=fr(util), max_source_blocks=B, theta=fr(theta), detach=fr(detach),
                         detach_rule=rule)
    d = repack_partial_definition(S, bts, tts, keeps, list(free), select, thr, set(protect), util, B, theta, detach,
                                  rule)
    assert p.released_blocks.tolist() == d["released"]
    nbo, nbf = to_csr(d["new_bt"])
    _, ntf = to_csr(d["new_tt"])
    assert p.new_bt_offsets.tolist() == nbo and p.new_bt_blocks.tolist() == nbf
    assert p.new_tt_slots.tolist() == ntf and p.freed_blocks.tolist() == d["freed"]
    assert p.req_status.tolist() == d["status"]
    assert list(zip(p.move_src.tolist(), p.move_dst.tolist())) == d["moves"]
    assert p.num_free_consumed == d["consumed"]


def test_bruteforce_against_the_definition_twin():
    rng = np.random.default_rng(3)
    S = 2
    bts = [[4, 1, 6], [0, 7, 3], []]
    tts = [[8, -1, 3, 2, 12, 13], [1, 0, -1, 14, 6, -1, 7], [-1, -1]]
    NB = 12
    for _ in range(40):
        keeps = [rng.integers(0, 2, len(t)).tolist() for t in tts]
        for util in (None, Fraction(1, 1), Fraction(1, 2)):
            for protect in ((), (1,), (4, 7)):
                for B in (0, 1, 2):
                    for theta in (None, Fraction(1, 4), Fraction(3, 4)):
                        for c in (0, 1, 3):
                            _compare(S, bts, tts, keeps, np.array([9, 5, 10][:c], np.int32), None,
                                     None if c else Fraction(3, 4), protect, util, B, theta, NB)


def test_bruteforce_all_masks_one_request():
    S = 3
    bt = [2, 0, 1]
    tt = [bt[t // S] * S + t % S for t in range(8)]
    for mask in itertools.product([0, 1], repeat=8):
        for util in (None, Fraction(1, 1), Fraction(2, 3), Fraction(1, 3)):
            for c in range(3):
                _compare(S, [bt], [tt], [list(mask)], np.array([5, 4][:c], np.int32), None, None, (), util, 0, None, 8)


def test_shared_prefix_blocks_are_skipped_and_private_suffixes_reclaimed():
    """Prefix-cache compatibility (Sec. 5, Table 1): every shared-prefix block is left in place for
    every sharing degree, private suffix blocks are reclaimed, and each request's logical view is
    unchanged."""
    for degree in (1, 2, 4):
        w, protect = wl.shared_prefix(seed=degree, groups=2, degree=degree, prefix_len=64, suffix_len=96, layers=1,
                                      heads=1, head_dim=8, block_size=4)
        S = w.block_size
        p = vto.plan_partial(S, w.num_blocks, w.bt_offsets, w.bt_blocks, w.tt_offsets, w.tt_slots, w.keep,
                             w.free_blocks, protect=protect)
        shared = set(np.flatnonzero(protect).tolist())
        assert p.num_admitted == w.num_requests
        assert not (set(p.freed_blocks.tolist()) & shared)                       # 100 % of shared candidates skipped
        assert not (set((p.move_src // S).tolist()) & shared)
        assert not (set((p.move_dst // S).tolist()) & shared)
        pre = w.notes["prefix_blocks"]
        live = (w.tt_slots >= 0) & (w.keep != 0)
        slab = np.arange(w.slots_per_layer * 2, dtype=np.int64).reshape(-1, 2)
        before = slab.copy()
        vto.apply_moves_slab(slab, p.move_src, p.move_dst)
        for r in range(w.num_requests):
            t0, t1 = w.tt_offsets[r], w.tt_offsets[r + 1]
            old = w.bt_blocks[w.bt_offsets[r]:w.bt_offsets[r + 1]]
            new = p.new_bt_blocks[p.new_bt_offsets[r]:p.new_bt_offsets[r + 1]]
            assert new[:pre].tolist() == old[:pre].tolist()                      # the prefix stays, in order
            n_private = int(live[t0 + 64:t1].sum())
            assert len(new) == pre + -(-n_private // S)                          # suffix packed densely
            a = vto.gather_logical(before, w.tt_slots[t0:t1], w.keep[t0:t1])
            b = vto.gather_logical(slab, p.new_tt_slots[t0:t1])
            assert np.array_equal(a, b)
        # the shared slots are referenced once per sharing request, private slots exactly once
        occ = p.new_tt_slots[p.new_tt_slots >= 0]
        counts = np.bincount(occ, minlength=w.slots_per_layer)
        assert counts[np.isin(np.arange(w.slots_per_layer) // S, list(shared))].max() <= degree
        assert counts[~np.isin(np.arange(w.slots_per_layer) // S, list(shared))].max() <= 1


# ---- copy-on-write detach from shared blocks --------------------------------------------------------
def test_detach_bruteforce_against_the_definition_twin():
    """Two requests sharing blocks 4 and 1 (protected), private blocks behind them; every keep mask
    of a random sample, several detach thresholds, source bounds and pool sizes."""
    rng = np.random.default_rng(5)
    S = 2
    bts = [[4, 1, 6, 2], [4, 1, 7, 3], [8]]
    tts = [[8, 9, 2, 3, 12, -1, 4, 5], [8, 9, 2, 3, 14, 15, 6, -1], [16, 17]]
    NB = 14
    for _ in range(60):
        keeps = [rng.integers(0, 2, len(t)).tolist() for t in tts]
        for detach in (None, Fraction(1, 1), Fraction(1, 2), Fraction(3, 4), Fraction(1, 4)):
            for util in (None, Fraction(1, 1)):
                for B in (0, 1):
                    for c in (0, 1, 2, 5):
                        _compare(S, bts, tts, keeps, np.array([9, 5, 10, 11, 12][:c], np.int32), None, None, (4, 1),
                                 util, B, None, NB, detach)


def test_detach_threshold_is_strict_and_counts_the_requests_own_tokens():
    """S = 4, two shared blocks (8 slots): the request keeps 4 of its 8 prefix tokens.  It leaves the
    prefix for thresholds above 1/2 and stays at exactly 1/2; the other sharer's tokens do not count."""
    S = 4
    bts = [[0, 1, 5], [0, 1, 6]]
    tts = [[0, 1, 2, 3, 4, 5, 6, 7, 20, 21], [0, 1, 2, 3, 4, 5, 6, 7, 24]]
    keeps = [[1, 0, 1, 0, 1, 0, 1, 0, 1, 1], [1] * 9]
    bt_off, bt_flat = to_csr(bts)
    tt_off, tt_flat = to_csr(tts)
    _, keep_flat = to_csr(keeps)
    protect = np.zeros(10, np.uint8)
    protect[[0, 1]] = 1
    free = np.array([7, 8, 9], np.int32)
    run = lambda d: vto.plan_partial(S, 10, bt_off, bt_flat, tt_off, tt_flat, keep_flat, free, protect=protect,
                                     util=(1, 1), detach=d)
    stay = run((1, 2))
    assert stay.released_blocks.tolist() == [] and stay.req_status.tolist() == [vto.NO_GAIN, vto.NO_GAIN]
    go = run((5, 8))
    # request 0: sources = shared 0, 1 and private 5 (2 of 4 live) -> 6 tokens -> 2 destinations < 3 sources
    assert go.req_status.tolist() == [vto.REPACKED, vto.NO_GAIN]
    assert go.released_blocks.tolist() == [0, 1] and go.freed_blocks.tolist() == [5]
    assert go.new_bt_blocks.tolist() == [7, 8, 0, 1, 6]
    assert go.new_tt_slots[:10].tolist() == [28, -1, 29, -1, 30, -1, 31, -1, 32, 33]
    assert go.new_tt_slots[10:].tolist() == tts[1]                         # the other sharer is untouched
    assert sorted(go.move_src.tolist()) == [0, 2, 4, 6, 20, 21]            # copies out of the shared blocks too


@pytest.mark.parametrize("degree", [1, 2, 4])
def test_detach_on_the_shared_prefix_workload(degree):
    """Every request of the prefix-cache workload leaves its shared prefix (H2O keeps about a fifth of
    it): its table shrinks to ceil(live / S), the prefix blocks are released once per sharer and never
    put on the free list or written to, and every request still sees exactly its own tokens."""
    w, protect = wl.shared_prefix(seed=degree, groups=2, degree=degree, prefix_len=64, suffix_len=96, layers=1,
                                  heads=1, head_dim=8, block_size=4)
    S = w.block_size
    p = vto.plan_partial(S, w.num_blocks, w.bt_offsets, w.bt_blocks, w.tt_offsets, w.tt_slots, w.keep, w.free_blocks,
                         protect=protect, detach=(1, 1))
    shared = set(np.flatnonzero(protect).tolist())
    live = (w.tt_slots >= 0) & (w.keep != 0)
    assert p.num_admitted == w.num_requests
    assert not (set(p.freed_blocks.tolist()) & shared) and not (set((p.move_dst // S).tolist()) & shared)
    assert sorted(np.bincount(p.released_blocks, minlength=w.num_blocks)[sorted(shared)].tolist()) == \
           [degree] * len(shared)
    slab = np.arange(w.slots_per_layer * 2, dtype=np.int64).reshape(-1, 2)
    before = slab.copy()
    vto.apply_moves_slab(slab, p.move_src, p.move_dst)
    shared_rows = np.isin(np.arange(w.slots_per_layer) // S, sorted(shared))
    assert np.array_equal(slab[shared_rows], before[shared_rows])            # the shared blocks keep their bytes
    for r in range(w.num_requests):
        t0, t1 = w.tt_offsets[r], w.tt_offsets[r + 1]
        new = p.new_bt_blocks[p.new_bt_offsets[r]:p.new_bt_offsets[r + 1]]
        assert len(new) == -(-int(live[t0:t1].sum()) // S) and not (set(new.tolist()) & shared)
        assert np.array_equal(vto.gather_logical(before, w.tt_slots[t0:t1], w.keep[t0:t1]),
                              vto.gather_logical(slab, p.new_tt_slots[t0:t1]))
    occ = p.new_tt_slots[p.new_tt_slots >= 0]
    assert np.bincount(occ).max() == 1                                       # every slot is private now
    # without detach the result is the conservative one of the paper's Table 1
    q = vto.plan_partial(S, w.num_blocks, w.bt_offsets, w.bt_blocks, w.tt_offsets, w.tt_slots, w.keep, w.free_blocks,
                         protect=protect)
    assert q.released_blocks.tolist() == [] and len(q.new_bt_blocks) > len(p.new_bt_blocks)


# ---- copy-on-write detach decided per shared block -------------------------------------------------
def test_per_block_detach_bruteforce_against_the_definition_twin():
    """Three requests over three protected blocks (0, 4 and 1; request 2 holds only one of them) with
    private blocks behind them, S = 3 so that a block can be 0/3 .. 3/3 full of one request's tokens;
    random keep masks x thresholds x utilisation x source bounds x pool sizes, block-by-block rule."""
    rng = np.random.default_rng(17)
    S = 3
    bts = [[0, 4, 1, 6], [0, 4, 1, 7, 3], [4, 8]]
    tts = [[0, 1, 2, 12, 13, 14, 3, 4, 5, 18, 19, -1], [0, 1, 2, 12, 13, 14, 3, 4, 5, 21, 22, 23, 9, -1, 11],
           [12, 13, 14, 24, 25]]
    NB = 16
    seen = set()
    for _ in range(50):
        keeps = [rng.integers(0, 2, len(t)).tolist() for t in tts]
        for detach in (Fraction(1, 3), Fraction(1, 2), Fraction(2, 3), Fraction(1, 1), Fraction(4, 3)):
            for util in (None, Fraction(1, 1)):
                for B in (0, 1):
                    for c in (0, 1, 3, 6):
                        free = np.array([9, 5, 10, 11, 12, 13][:c], np.int32)
                        _compare(S, bts, tts, keeps, free, None, None, (0, 4, 1), util, B, None, NB, detach, 1)
            d = repack_partial_definition(S, bts, tts, keeps, [9, 5, 10, 11, 12, 13], protect={0, 4, 1}, detach=detach,
                                          detach_rule=1)
            for r in range(3):
                shared = [b for b in bts[r] if b in (0, 4, 1)]
                seen.add((len(shared), sum(b in d["new_bt"][r] for b in shared)))
    # the sample really holds requests that left some of their shared blocks and stayed in others
    assert {(3, 1), (3, 2), (3, 0), (3, 3), (1, 0), (1, 1)} <= seen


def test_per_block_detach_by_hand():
    """S = 4.  Request 0 holds shared blocks 0, 1, 2 and private block 5; of its prefix tokens it keeps
    3 in block 0, 1 in block 1 and 2 in block 2; request 1 keeps everything.  At threshold 1/2 it leaves
    block 1 only (1/4 < 1/2; 2/4 is not below 1/2: strict); at 3/4 blocks 1 and 2; the request-level
    rule at 1/2 would have kept all three (6 of 12 slots)."""
    S = 4
    bts = [[0, 1, 2, 5], [0, 1, 2, 6]]
    tts = [list(range(12)) + [20, 21, 22], list(range(12)) + [24]]
    keeps = [[1, 1, 1, 0,  0, 1, 0, 0,  1, 0, 0, 1,  1, 0, 1], [1] * 13]
    bt_off, bt_flat = to_csr(bts)
    tt_off, tt_flat = to_csr(tts)
    _, keep_flat = to_csr(keeps)
    protect = np.zeros(12, np.uint8)
    protect[[0, 1, 2]] = 1
    free = np.array([7, 8, 9], np.int32)
    run = lambda d, pb: vto.plan_partial(S, 12, bt_off, bt_flat, tt_off, tt_flat, keep_flat, free, protect=protect,
                                         util=(1, 1), detach=d, detach_rule=int(pb))
    whole = run((1, 2), False)
    assert whole.released_blocks.tolist() == [] and whole.req_status.tolist() == [vto.NO_GAIN, vto.NO_GAIN]
    half = run((1, 2), True)
    # sources: shared 1 (1 live) and private 5 (2 of 4 live) -> 3 tokens -> 1 destination < 2 sources
    assert half.req_status.tolist() == [vto.REPACKED, vto.NO_GAIN]
    assert half.released_blocks.tolist() == [1] and half.freed_blocks.tolist() == [5]
    assert half.new_bt_blocks.tolist() == [0, 2, 7, 0, 1, 2, 6]
    assert half.new_tt_slots[:15].tolist() == [0, 1, 2, -1, -1, 28, -1, -1, 8, -1, -1, 11, 29, -1, 30]
    assert half.new_tt_slots[15:].tolist() == tts[1]                       # the other sharer is untouched
    assert list(zip(half.move_src.tolist(), half.move_dst.tolist())) == [(5, 28), (20, 29), (22, 30)]
    more = run((3, 4), True)
    # blocks 1 and 2 and private 5: 1 + 2 + 2 = 5 tokens -> 2 destinations < 3 sources
    assert more.released_blocks.tolist() == [1, 2] and more.freed_blocks.tolist() == [5]
    assert more.new_bt_blocks.tolist() == [0, 7, 8, 0, 1, 2, 6]
    assert more.new_tt_slots[:15].tolist() == [0, 1, 2, -1, -1, 28, -1, -1, 29, -1, -1, 30, 31, -1, 32]
    assert len(more.released_blocks) == 2 and more.num_moves == 5


def test_per_block_detach_meets_the_request_level_rule_where_the_two_must_agree():
    """(a) A threshold above one empties every protected block under either rule.  (b) With one
    protected block per request the block is the request's whole shared part.  (c) Threshold 0/1:
    nothing is below it, both equal the conservative plan."""
    w, protect = wl.shared_prefix(seed=3, groups=3, degree=2, prefix_len=48, suffix_len=80, layers=1, heads=1,
                                  head_dim=8, block_size=4)
    S = w.block_size
    run = lambda **kw: vto.plan_partial(S, w.num_blocks, w.bt_offsets, w.bt_blocks, w.tt_offsets, w.tt_slots, w.keep,
                                        w.free_blocks, util=(1, 1), **kw)
    same = lambda p, q: all(np.array_equal(getattr(p, f), getattr(q, f)) for f in
                            ("new_bt_offsets", "new_bt_blocks", "new_tt_slots", "freed_blocks", "released_blocks",
                             "req_status", "move_src", "move_dst"))
    assert same(run(protect=protect, detach=(5, 4)), run(protect=protect, detach=(5, 4), detach_rule=1))
    assert len(run(protect=protect, detach=(5, 4)).released_blocks) > 0
    one = np.zeros_like(protect)                 # protect only the first block of every request's table
    one[w.bt_blocks[w.bt_offsets[:-1]]] = 1
    # (the other prefix blocks are then unprotected blocks in several tables: plan request by request)
    for r in range(w.num_requests):
        sel = np.zeros(w.num_requests, np.uint8)
        sel[r] = 1
        for d in ((1, 4), (1, 2), (3, 4), (1, 1)):
            assert same(run(protect=one, detach=d, select=sel), run(protect=one, detach=d, select=sel,
                                                                    detach_rule=1))
    cons = run(protect=protect)
    assert same(cons, run(protect=protect, detach=(0, 1), detach_rule=1))
    assert same(cons, run(protect=protect, detach=(0, 1)))


@pytest.mark.parametrize("degree", [1, 2, 4])
@pytest.mark.parametrize("detach", [(1, 4), (1, 2), (3, 4)])
def test_per_block_detach_on_the_shared_prefix_workload(degree, detach):
    """Block-by-block detach on the prefix-cache workload: a request leaves exactly the prefix blocks it
    fills below the threshold (counted from its own mask), keeps the others at the head of its table,
    the shared blocks are never freed, written to or changed, and every request sees its own tokens."""
    w, protect = wl.shared_prefix(seed=10 + degree, groups=2, degree=degree, prefix_len=64, suffix_len=96, layers=1,
                                  heads=1, head_dim=8, block_size=4)
    S = w.block_size
    p = vto.plan_partial(S, w.num_blocks, w.bt_offsets, w.bt_blocks, w.tt_offsets, w.tt_slots, w.keep, w.free_blocks,
                         protect=protect, detach=detach, detach_rule=1)
    shared = set(np.flatnonzero(protect).tolist())
    live = (w.tt_slots >= 0) & (w.keep != 0)
    assert not (set(p.freed_blocks.tolist()) & shared) and not (set((p.move_dst // S).tolist()) & shared)
    assert set(p.released_blocks.tolist()) <= shared
    slab = np.arange(w.slots_per_layer * 2, dtype=np.int64).reshape(-1, 2)
    before = slab.copy()
    vto.apply_moves_slab(slab, p.move_src, p.move_dst)
    shared_rows = np.isin(np.arange(w.slots_per_layer) // S, sorted(shared))
    assert np.array_equal(slab[shared_rows], before[shared_rows])
    released = p.released_blocks.tolist()
    cursor = 0
    some_left = some_stayed = False
    for r in range(w.num_requests):
        t0, t1 = w.tt_offsets[r], w.tt_offsets[r + 1]
        old = w.bt_blocks[w.bt_offsets[r]:w.bt_offsets[r + 1]].tolist()
        new = p.new_bt_blocks[p.new_bt_offsets[r]:p.new_bt_offsets[r + 1]].tolist()
        assert np.array_equal(vto.gather_logical(before, w.tt_slots[t0:t1], w.keep[t0:t1]),
                              vto.gather_logical(slab, p.new_tt_slots[t0:t1]))
        if p.req_status[r] != vto.REPACKED:
            assert new == old
            continue
        mine = np.bincount(w.tt_slots[t0:t1][live[t0:t1]] // S, minlength=w.num_blocks)
        leaves = [b for b in old if b in shared and mine[b] * detach[1] < detach[0] * S]
        stays = [b for b in old if b in shared and b not in leaves]
        assert released[cursor:cursor + len(leaves)] == leaves
        cursor += len(leaves)
        assert new[:len(stays)] == stays and not (set(new) & set(leaves))
        # its tokens in the blocks it stays in keep their slots; those in the blocks it left were copied out
        slots, now = w.tt_slots[t0:t1], p.new_tt_slots[t0:t1]
        in_stay = live[t0:t1] & np.isin(slots // S, stays)
        in_left = live[t0:t1] & np.isin(slots // S, leaves)
        assert np.array_equal(now[in_stay], slots[in_stay]) and not np.isin(now[in_left] // S, sorted(shared)).any()
        some_left |= bool(leaves)
        some_stayed |= bool(stays)
    assert cursor == len(released)
    if detach == (1, 2):
        assert some_left and some_stayed            # the threshold really splits the prefix


# ---- copy-on-write detach decided per shared block from the live tokens of all its holders ----------
def test_all_holders_detach_bruteforce_against_the_definition_twin():
    """The tables of the per-block brute force (three requests over three protected blocks, S = 3), rule 2:
    a protected block is left by every planned holder when everything stored in it -- one count per
    referencing token-table entry -- fills less than the threshold of a block."""
    rng = np.random.default_rng(23)
    S = 3
    bts = [[0, 4, 1, 6], [0, 4, 1, 7, 3], [4, 8]]
    tts = [[0, 1, 2, 12, 13, 14, 3, 4, 5, 18, 19, -1], [0, 1, 2, 12, 13, 14, 3, 4, 5, 21, 22, 23, 9, -1, 11],
           [12, 13, 14, 24, 25]]
    NB = 16
    verdicts = set()
    for _ in range(50):
        keeps = [(rng.random(len(t)) < rng.choice([0.15, 0.4, 0.8])).astype(int).tolist() for t in tts]
        for detach in (Fraction(1, 3), Fraction(2, 3), Fraction(1, 1), Fraction(4, 3), Fraction(7, 3)):
            for util in (None, Fraction(1, 1)):
                for B in (0, 1):
                    for c in (0, 1, 3, 6):
                        free = np.array([9, 5, 10, 11, 12, 13][:c], np.int32)
                        _compare(S, bts, tts, keeps, free, None, None, (0, 4, 1), util, B, None, NB, detach, 2)
            d = repack_partial_definition(S, bts, tts, keeps, [9, 5, 10, 11, 12, 13], protect={0, 4, 1}, detach=detach,
                                          detach_rule=2)
            # every admitted holder of a block reaches the same verdict on it
            for b in (0, 4, 1):
                held = [r for r in range(3) if b in bts[r] and d["status"][r] == 1]
                gone = [r for r in held if b not in d["new_bt"][r]]
                assert len(gone) in (0, len(held))
                if held:
                    verdicts.add(bool(gone))
    assert verdicts == {True, False}


def test_all_holders_detach_by_hand():
    """S = 4, blocks 0 and 1 shared by two requests.  Block 0: request 0 keeps one token, request 1 keeps
    two -> n_b = 3 < 4: both leave it at threshold 1/1.  Block 1: one + three -> n_b = 4: not below a block,
    both stay -- although request 0 alone fills a quarter of it (rule 1 would let it go).  At 3/4 nobody
    leaves block 0 either (3/4 is not below 3/4)."""
    S = 4
    bts = [[0, 1, 5], [0, 1, 6]]
    tts = [list(range(8)) + [20, 21, 22, 23], list(range(8)) + [24, 25, 26, 27]]
    keeps = [[1, 0, 0, 0,  0, 1, 0, 0,  1, 0, 0, 0], [0, 1, 1, 0,  1, 0, 1, 1,  0, 0, 1, 0]]
    bt_off, bt_flat = to_csr(bts)
    tt_off, tt_flat = to_csr(tts)
    _, keep_flat = to_csr(keeps)
    protect = np.zeros(12, np.uint8)
    protect[[0, 1]] = 1
    free = np.array([7, 8, 9, 10], np.int32)
    run = lambda d, rule: vto.plan_partial(S, 12, bt_off, bt_flat, tt_off, tt_flat, keep_flat, free, protect=protect,
                                           util=(1, 1), detach=d, detach_rule=rule)
    p = run((1, 1), 2)
    assert p.req_status.tolist() == [vto.REPACKED, vto.REPACKED]
    assert p.released_blocks.tolist() == [0, 0] and p.freed_blocks.tolist() == [5, 6]
    # request 0: tokens 0 (block 0) and 20 (block 5) move to block 7; it stays in block 1
    assert p.new_bt_blocks.tolist() == [1, 7, 1, 8]
    assert p.new_tt_slots[:12].tolist() == [28, -1, -1, -1, -1, 5, -1, -1, 29, -1, -1, -1]
    assert p.new_tt_slots[12:].tolist() == [-1, 32, 33, -1, 4, -1, 6, 7, -1, -1, 34, -1]
    assert list(zip(p.move_src.tolist(), p.move_dst.tolist())) == [(0, 28), (20, 29), (1, 32), (2, 33), (26, 34)]
    own = run((1, 1), 1)                       # by its own tokens request 0 would leave block 1 as well
    assert own.released_blocks.tolist()[:2] == [0, 1]
    strict = run((3, 4), 2)
    assert strict.released_blocks.tolist() == []


@pytest.mark.parametrize("degree", [1, 2, 4, 8])
def test_all_holders_detach_on_the_shared_prefix_workload(degree):
    """Threshold 1/1 on the prefix-cache workload (H2O keeps about a fifth per request): what is left is
    decided by bincount over all holders' live tokens; a block every holder left appears once per holder in
    the released list and in no new table, shared bytes stay, every request sees its tokens.  With degree 1
    the rule equals the per-block rule on own tokens."""
    w, protect = wl.shared_prefix(seed=20 + degree, groups=2, degree=degree, prefix_len=64, suffix_len=96, layers=1,
                                  heads=1, head_dim=8, block_size=4)
    S = w.block_size
    extra = 400                                     # room for every private copy
    NB = w.num_blocks + extra
    free = np.concatenate([w.free_blocks, np.arange(w.num_blocks, NB, dtype=np.int32)])
    prot = np.concatenate([protect, np.zeros(extra, np.uint8)])
    run = lambda rule: vto.plan_partial(S, NB, w.bt_offsets, w.bt_blocks, w.tt_offsets, w.tt_slots, w.keep, free,
                                        protect=prot, detach=(1, 1), detach_rule=rule)
    p = run(2)
    live = (w.tt_slots >= 0) & (w.keep != 0)
    n_b = np.bincount(w.tt_slots[live] // S, minlength=NB)
    shared = np.flatnonzero(prot)
    leaves = {int(b) for b in shared if n_b[b] < S}
    assert p.num_admitted == w.num_requests
    assert sorted(p.released_blocks.tolist()) == sorted(b for b in leaves for _ in range(degree))
    assert not (set(p.new_bt_blocks.tolist()) & leaves)
    for b in set(shared.tolist()) - leaves:
        assert (p.new_bt_blocks == b).sum() == degree
    slab = np.arange(NB * S * 2, dtype=np.int64).reshape(-1, 2)
    before = slab.copy()
    vto.apply_moves_slab(slab, p.move_src, p.move_dst)
    rows = np.isin(np.arange(NB * S) // S, shared)
    assert np.array_equal(slab[rows], before[rows])
    for r in range(w.num_requests):
        t0, t1 = w.tt_offsets[r], w.tt_offsets[r + 1]
        assert np.array_equal(vto.gather_logical(before, w.tt_slots[t0:t1], w.keep[t0:t1]),
                              vto.gather_logical(slab, p.new_tt_slots[t0:t1]))
    if degree == 1:
        q = run(1)
        assert np.array_equal(p.new_tt_slots, q.new_tt_slots) and np.array_equal(p.released_blocks, q.released_blocks)
    if degree == 8:
        assert len(leaves) < len(shared)            # eight holders fill most prefix blocks beyond one block's worth
