"""Pins of the CPU oracle against what the paper and the mathematics fix (no GPU).

Each test is chosen so that a plausible slip in the oracle (a dropped term, an off-by-one in
ceil, a transposed src/dst, a wrong order) fails at least one of them.
"""
import itertools
from fractions import Fraction

import numpy as np
import pytest

from conftest import read_golden
from definition_twin import repack_definition, to_csr
from oracle import vto
from harness import workloads as wl


# ------------------------------------------------------------------------------------------
# helpers
# ------------------------------------------------------------------------------------------
def identity_request(n_tokens, S, first_block=0):
    nb = -(-n_tokens // S)
    bt = np.arange(first_block, first_block + nb, dtype=np.int32)
    tt = (bt[np.arange(n_tokens) // S] * S + np.arange(n_tokens) % S).astype(np.int32)
    return bt, tt


def host_pools(w, seed=1):
    """K and V pools [L, NB*S, row_elems] uint16 from the shared fill generator."""
    k = np.stack([wl.fill_slab(seed, 0, l, w.num_layers, w.slots_per_layer, w.row_elems)
                  for l in range(w.num_layers)])
    v = np.stack([wl.fill_slab(seed, 1, l, w.num_layers, w.slots_per_layer, w.row_elems)
                  for l in range(w.num_layers)])
    return k, v


def small_workloads():
    yield wl.tiny(seed=0)
    yield wl.tiny(seed=3, requests=7, lo=1, hi=70, block_size=3, heads=1, head_dim=8)
    yield wl.llama8b_h2o(seed=1, requests=5, lo=100, hi=400, layers=2, heads=1, head_dim=16)
    yield wl.mistral7b_random(seed=2, requests=9, lo=20, hi=200, layers=2, heads=1, head_dim=16)
    yield wl.longctx_scissor(seed=3, requests=3, lo=900, hi=1500, layers=1, heads=1, head_dim=8)
    yield wl.steady_state(seed=4, requests=12, lo=100, hi=600, layers=1, heads=1, head_dim=8)
    yield wl.steady_state(seed=5, requests=12, lo=100, hi=600, layers=1, heads=1, head_dim=8,
                          block_size=32)
    yield wl.streaming_window(seed=6, requests=6, lo=60, hi=400, window=48, layers=1, heads=1, head_dim=8)


# ------------------------------------------------------------------------------------------
# values the paper prints
# ------------------------------------------------------------------------------------------
def test_capacity_frontier_block_arithmetic():
    """Sec. 5 capacity frontier: a 16,320-token request holds 1,020 blocks of 16; its 8,192
    retained tokens pack into 512; 22 such requests fit 11,519 usable blocks, 23 do not."""
    g = read_golden("capacity_frontier.txt")
    S = g["block_size"]
    n_tokens = g["full_request_blocks"] * S
    bt, tt = identity_request(n_tokens, S)
    assert len(bt) == g["full_request_blocks"]
    keep = np.zeros(n_tokens, np.uint8)
    keep[np.random.default_rng(0).permutation(n_tokens)[:g["packed_request_blocks"] * S]] = 1
    free = np.arange(len(bt), len(bt) + 600, dtype=np.int32)
    p = vto.plan(S, [0, len(bt)], bt, [0, n_tokens], tt, keep, free)
    assert p.num_free_consumed == g["packed_request_blocks"]
    assert p.num_freed == g["full_request_blocks"]
    assert p.req_status.tolist() == [vto.REPACKED]
    assert g["six_full_requests_blocks"] == 6 * g["full_request_blocks"] > g["usable_blocks_mem_util_0_35"]
    assert g["usable_blocks_mem_util_0_35"] // g["full_request_blocks"] == g["native_max_concurrency_0_35"]
    assert g["usable_blocks_mem_util_0_50"] // g["full_request_blocks"] == g["native_max_concurrency_0_50"]

    # 23 identical requests, a free list as long as the paper's usable pool: exactly 22 are admitted.
    C = g["vtoken_max_concurrency_0_50"] + 1
    bts, tts, keeps = [], [], []
    for c in range(C):
        b, t = identity_request(n_tokens, S, first_block=c * g["full_request_blocks"])
        bts.append(b), tts.append(t), keeps.append(keep)
    bt_off = np.arange(C + 1) * g["full_request_blocks"]
    tt_off = np.arange(C + 1) * n_tokens
    first_free = C * g["full_request_blocks"]
    free = np.arange(first_free, first_free + g["usable_blocks_mem_util_0_50"], dtype=np.int32)
    p = vto.plan(S, bt_off, np.concatenate(bts), tt_off, np.concatenate(tts),
                 np.concatenate(keeps), free)
    assert p.num_admitted == g["vtoken_max_concurrency_0_50"]
    assert p.num_deferred == 1
    assert p.num_free_consumed == g["vtoken_max_concurrency_0_50"] * g["packed_request_blocks"]
    assert p.req_status.tolist() == [vto.REPACKED] * (C - 1) + [vto.DEFERRED_NO_FREE]


def test_kv_bytes_per_token_paper_figures():
    """Sec. 2.1: 2*L*H*D*dtype; 13B LLaMA ~0.8 MB per token; Sec. 4: ~2 GB per 16K tokens (7B/8B)."""
    g = read_golden("kv_bytes_per_token.txt")
    assert wl.kv_bytes_per_token(g["llama13b_layers"], 1, g["llama13b_hidden"], 2) == g["llama13b_bytes_per_token"]
    assert abs(g["llama13b_bytes_per_token"] / 1e6 - 0.8) < 0.05
    assert wl.kv_bytes_per_token(32, 8, 128, 2) * 16384 == g["llama8b_bytes_16k_tokens"]
    assert 16 * 16384 == g["token_table_bytes_16k"]


# ------------------------------------------------------------------------------------------
# special case that reduces to library routines: one request, identity layout
# ------------------------------------------------------------------------------------------
@pytest.mark.parametrize("S,n_tokens,seed", [(16, 1000, 0), (1, 37, 1), (3, 100, 2), (32, 4097, 3), (48, 48 * 5, 4)])
def test_single_request_matches_numpy_compaction(S, n_tokens, seed):
    rng = np.random.default_rng(seed)
    bt, tt = identity_request(n_tokens, S)
    nb = len(bt)
    keep = (rng.random(n_tokens) < 0.4).astype(np.uint8)
    n = int(keep.sum())
    need = -(-n // S)
    free = np.arange(nb, nb + need + 3, dtype=np.int32)[::-1].copy()   # descending: order matters
    p = vto.plan(S, [0, nb], bt, [0, n_tokens], tt, keep, free)
    if need < nb:
        ranks = np.cumsum(keep, dtype=np.int64) - 1
        expect = np.where(keep != 0, free[np.maximum(ranks, 0) // S] * S + ranks % S, -1)
        assert np.array_equal(p.new_tt_slots, expect)
        assert np.array_equal(p.new_bt_blocks, free[:need])
        assert np.array_equal(p.freed_blocks, bt)
        assert np.array_equal(p.move_src, tt[np.flatnonzero(keep)])
        # bytes: packed rows == boolean-mask row selection of the slab
        NBtot = nb + need + 3
        slab = rng.integers(0, 2 ** 16, size=(NBtot * S, 8), dtype=np.uint16)
        before = slab.copy()
        vto.apply_moves_slab(slab, p.move_src, p.move_dst)
        packed = slab[p.new_tt_slots[keep != 0]]
        assert np.array_equal(packed, before[:n_tokens][keep != 0])
        # nothing but the destination rows changed
        changed = np.flatnonzero((slab != before).any(axis=1))
        assert set(changed) <= set(p.move_dst.tolist())
        assert np.array_equal(vto.gather_logical(slab, p.new_tt_slots), before[:n_tokens][keep != 0])
    else:
        assert p.req_status.tolist() == [vto.NO_GAIN]


def test_moves_are_src_to_dst_not_transposed():
    """row[dst] = row[src]: a swapped memcpy would overwrite live rows with free-block bytes."""
    S = 2
    bt, tt = identity_request(4, S)           # slots 0..3 in blocks 0,1
    keep = np.array([1, 0, 0, 0], np.uint8)
    p = vto.plan(S, [0, 2], bt, [0, 4], tt, keep, np.array([5], np.int32))
    assert p.move_src.tolist() == [0] and p.move_dst.tolist() == [10]
    slab = np.arange(12 * 4, dtype=np.uint16).reshape(12, 4)
    before = slab.copy()
    vto.apply_moves_slab(slab, p.move_src, p.move_dst)
    assert np.array_equal(slab[10], before[0]) and np.array_equal(slab[0], before[0])
    assert np.array_equal(np.delete(slab, 10, 0), np.delete(before, 10, 0))


# ------------------------------------------------------------------------------------------
# brute force on tiny pools against the definition-level twin
# ------------------------------------------------------------------------------------------
def _compare_with_twin(S, bts, tts, keeps, free, select, thr):
    bt_off, bt_flat = to_csr(bts)
    tt_off, tt_flat = to_csr(tts)
    _, keep_flat = to_csr(keeps)
    thr_num, thr_den = (thr.numerator, thr.denominator) if thr is not None else (0, 0)
    p = vto.plan(S, bt_off, bt_flat, tt_off, tt_flat, keep_flat, free,
                 select=None if select is None else np.array(select, np.uint8),
                 thr_num=thr_num, thr_den=thr_den)
    d = repack_definition(S, bts, tts, keeps, list(free), select, thr)
    nbo, nbf = to_csr(d["new_bt"])
    _, ntf = to_csr(d["new_tt"])
    assert p.new_bt_offsets.tolist() == nbo
    assert p.new_bt_blocks.tolist() == nbf
    assert p.new_tt_slots.tolist() == ntf
    assert p.freed_blocks.tolist() == d["freed"]
    assert p.req_status.tolist() == d["status"]
    assert list(zip(p.move_src.tolist(), p.move_dst.tolist())) == d["moves"]
    assert p.num_free_consumed == d["consumed"] == p.num_dst_blocks
    assert p.num_admitted == d["status"].count(1) and p.num_deferred == d["status"].count(3)


@pytest.mark.parametrize("S", [1, 2, 3, 4])
def test_bruteforce_all_masks_tiny(S):
    """Every keep mask of a two-request pool with 9 tokens, every free-list length."""
    lens = [5, 4]
    bts, tts, nxt = [], [], 0
    for n in lens:
        nb = -(-n // S)
        blocks = list(range(nxt, nxt + nb))[::-1]           # non-monotone physical order
        nxt += nb
        bts.append(blocks)
        tts.append([blocks[t // S] * S + t % S for t in range(n)])
    total_need_max = sum(-(-n // S) for n in lens)
    free_all = list(range(nxt + 2, nxt + 2 + total_need_max))[::-1]
    for mask in itertools.product([0, 1], repeat=sum(lens)):
        keeps = [list(mask[:lens[0]]), list(mask[lens[0]:])]
        for c in range(len(free_all) + 1):
            _compare_with_twin(S, bts, tts, keeps, np.array(free_all[:c], np.int32), None, None)


def test_bruteforce_select_threshold_holes():
    """Three requests with -1 holes, every select subset, several thresholds, short free lists."""
    rng = np.random.default_rng(7)
    S = 2
    bts = [[4, 1], [0, 7, 3], []]
    tts = [[8, -1, 3, 2], [1, 0, -1, 14, 6, -1, 7], [-1, -1]]
    for _ in range(60):
        keeps = [rng.integers(0, 2, len(t)).tolist() for t in tts]
        for select in [None] + [list(s) for s in itertools.product([0, 1], repeat=3)]:
            for thr in [None, Fraction(1, 4), Fraction(1, 2), Fraction(3, 4), Fraction(1, 1)]:
                for c in range(0, 4):
                    _compare_with_twin(S, bts, tts, keeps, np.array([9, 5, 8][:c], np.int32), select, thr)


def test_threshold_equality_is_not_selected():
    """n / (nb*S) == thr exactly -> not below the threshold (strict integer comparison)."""
    S = 4
    bt, tt = identity_request(16, S)
    keep = np.zeros(16, np.uint8)
    keep[:8] = 1                                            # live fraction exactly 1/2
    free = np.array([10, 11], np.int32)
    assert vto.plan(S, [0, 4], bt, [0, 16], tt, keep, free, thr_num=1, thr_den=2).req_status.tolist() == [vto.NOT_SELECTED]
    keep[7] = 0                                             # 7/16 < 1/2
    assert vto.plan(S, [0, 4], bt, [0, 16], tt, keep, free, thr_num=1, thr_den=2).req_status.tolist() == [vto.REPACKED]


# ------------------------------------------------------------------------------------------
# invariants on the synthetic workloads (I1, I2, block conservation, untouched bytes)
# ------------------------------------------------------------------------------------------
@pytest.mark.parametrize("w", list(small_workloads()), ids=lambda w: f"{w.name}-S{w.block_size}-seed{w.seed}")
def test_invariants_on_workloads(w):
    S = w.block_size
    assert vto.validate(S, w.num_blocks, w.bt_offsets, w.bt_blocks, w.tt_offsets, w.tt_slots,
                        w.keep, w.free_blocks) == 0
    p = vto.plan_workload(w)
    R = w.num_requests
    live = (w.tt_slots >= 0) & (w.keep != 0)
    # token conservation (I1): same active ids before and after
    assert np.array_equal(p.new_tt_slots >= 0, live)
    # unique mapping (I2)
    occupied = p.new_tt_slots[p.new_tt_slots >= 0]
    assert len(np.unique(occupied)) == len(occupied)
    # blocks per repacked request = ceil(live / S); order and complete fill
    for r in range(R):
        t0, t1 = w.tt_offsets[r], w.tt_offsets[r + 1]
        n = int(live[t0:t1].sum())
        nbt = p.new_bt_blocks[p.new_bt_offsets[r]:p.new_bt_offsets[r + 1]]
        old = w.bt_blocks[w.bt_offsets[r]:w.bt_offsets[r + 1]]
        if p.req_status[r] == vto.REPACKED:
            assert len(nbt) == -(-n // S) < len(old)
            i = np.arange(n)
            assert np.array_equal(p.new_tt_slots[t0:t1][live[t0:t1]], nbt[i // S] * S + i % S)
        else:
            assert np.array_equal(nbt, old)
            assert np.array_equal(p.new_tt_slots[t0:t1][live[t0:t1]], w.tt_slots[t0:t1][live[t0:t1]])
    adm = np.flatnonzero(p.req_status == vto.REPACKED)
    # conservation of blocks
    assert np.array_equal(w.free_blocks[:p.num_free_consumed],
                          np.concatenate([p.new_bt_blocks[p.new_bt_offsets[r]:p.new_bt_offsets[r + 1]] for r in adm] + [np.zeros(0, np.int32)]))
    assert np.array_equal(p.freed_blocks,
                          np.concatenate([w.bt_blocks[w.bt_offsets[r]:w.bt_offsets[r + 1]] for r in adm] + [np.zeros(0, np.int32)]))
    assert p.num_freed - p.num_free_consumed >= p.num_admitted
    assert p.num_moves == int(sum(live[w.tt_offsets[r]:w.tt_offsets[r + 1]].sum() for r in adm))
    assert vto.check_semantics(S, w.bt_offsets, w.bt_blocks, w.tt_offsets, w.tt_slots, w.keep, w.free_blocks,
                               p.new_bt_offsets, p.new_bt_blocks, p.new_tt_slots, p.freed_blocks,
                               p.num_free_consumed, p.req_status, w.select, w.thr_num, w.thr_den) == 0
    # sources and destinations are disjoint sets
    assert not (set(p.move_src.tolist()) & set(p.move_dst.tolist()))

    # bytes: logical view identical before and after, everything but destinations untouched
    k, v = host_pools(w)
    k0, v0 = k.copy(), v.copy()
    vto.apply_moves_pools(k, v, p.move_src, p.move_dst, threads=2)
    for pool, pool0 in ((k, k0), (v, v0)):
        for l in range(w.num_layers):
            for r in range(R):
                t0, t1 = w.tt_offsets[r], w.tt_offsets[r + 1]
                a = vto.gather_logical(pool0[l], w.tt_slots[t0:t1], w.keep[t0:t1])
                b = vto.gather_logical(pool[l], p.new_tt_slots[t0:t1])
                assert np.array_equal(a, b)
                # independent of the oracle's own gather: numpy fancy indexing
                assert np.array_equal(a, pool0[l][w.tt_slots[t0:t1][live[t0:t1]]])
            changed = np.flatnonzero((pool[l] != pool0[l]).any(axis=1))
            assert set(changed.tolist()) <= set(p.move_dst.tolist())

    # idempotence: adopt the new state, keep everything that is left -> nothing to gain
    keep2 = (p.new_tt_slots >= 0).astype(np.uint8)
    left = w.free_blocks[p.num_free_consumed:]
    if p.num_deferred == 0 and w.thr_den == 0:
        q = vto.plan(S, p.new_bt_offsets, p.new_bt_blocks, w.tt_offsets, p.new_tt_slots, keep2, left)
        assert set(q.req_status.tolist()) <= {vto.NO_GAIN}
        assert np.array_equal(q.new_tt_slots, p.new_tt_slots)
        assert np.array_equal(q.new_bt_blocks, p.new_bt_blocks)
        assert q.num_moves == 0 and q.num_freed == 0


def test_free_list_cut_at_every_length_prefix_rule():
    """Free list of every length: the admitted set is the longest candidate prefix; later
    candidates are deferred even when they would fit."""
    w = wl.mistral7b_random(seed=11, requests=6, lo=30, hi=90, layers=1, heads=1, head_dim=8, block_size=4)
    full = vto.plan_workload(w)
    assert full.num_deferred == 0
    needs = [full.new_bt_offsets[r + 1] - full.new_bt_offsets[r] for r in range(w.num_requests)]
    for c in range(full.num_free_consumed + 1):
        p = vto.plan_workload(w, num_free=c)
        cum, cut = 0, False
        for r in range(w.num_requests):
            if full.req_status[r] != vto.REPACKED:
                assert p.req_status[r] == full.req_status[r]
                continue
            cum += needs[r]
            cut = cut or cum > c
            assert p.req_status[r] == (vto.DEFERRED_NO_FREE if cut else vto.REPACKED)


def test_edge_cases():
    S = 4
    # all-keep on a fresh identity layout: nothing to gain, outputs equal inputs
    bt, tt = identity_request(10, S)
    p = vto.plan(S, [0, 3], bt, [0, 10], tt, np.ones(10, np.uint8), np.array([7, 8, 9], np.int32))
    assert p.req_status.tolist() == [vto.NO_GAIN] and p.num_moves == 0
    assert np.array_equal(p.new_tt_slots, tt) and np.array_equal(p.new_bt_blocks, bt)
    # all-evict: frees every block, consumes none
    p = vto.plan(S, [0, 3], bt, [0, 10], tt, np.zeros(10, np.uint8), np.zeros(0, np.int32))
    assert p.req_status.tolist() == [vto.REPACKED] and p.num_free_consumed == 0
    assert p.freed_blocks.tolist() == bt.tolist() and (p.new_tt_slots == -1).all()
    assert p.new_bt_offsets.tolist() == [0, 0]
    # empty request without blocks: no gain
    p = vto.plan(S, [0, 0], np.zeros(0, np.int32), [0, 0], np.zeros(0, np.int32), np.zeros(0, np.uint8),
                 np.array([1], np.int32))
    assert p.req_status.tolist() == [vto.NO_GAIN]
    # kept flag on an entry without a physical copy is not live
    tt2 = tt.copy()
    tt2[5] = -1
    p = vto.plan(S, [0, 3], bt, [0, 10], tt2, np.ones(10, np.uint8), np.array([7, 8, 9], np.int32))
    assert p.new_tt_slots[5] == -1
    # live counts around a block boundary: k*S-1, k*S, k*S+1
    bt, tt = identity_request(40, S)
    for n in (7, 8, 9):
        keep = np.zeros(40, np.uint8)
        keep[np.arange(n) * 4] = 1
        p = vto.plan(S, [0, 10], bt, [0, 40], tt, keep, np.arange(20, 30, dtype=np.int32))
        assert p.num_free_consumed == -(-n // S)
    # worst fragmentation: one survivor per block -> nb - ceil(nb/S) blocks gained
    keep = np.zeros(40, np.uint8)
    keep[::S] = 1
    p = vto.plan(S, [0, 10], bt, [0, 40], tt, keep, np.arange(20, 30, dtype=np.int32))
    assert p.num_freed - p.num_free_consumed == 10 - 3


def test_validate_flags_broken_inputs():
    S = 4
    bt, tt = identity_request(10, S)
    ok = dict(S=S, NB=8, bt_offsets=[0, 3], bt_blocks=bt, tt_offsets=[0, 10], tt_slots=tt,
              keep=np.ones(10, np.uint8), free_blocks=np.array([5, 6], np.int32))
    assert vto.validate(**ok) == 0
    assert vto.validate(**{**ok, "free_blocks": np.array([2], np.int32)}) == 5      # free block allocated
    assert vto.validate(**{**ok, "free_blocks": np.array([9], np.int32)}) == 4      # out of range
    t = tt.copy(); t[1] = t[0]
    assert vto.validate(**{**ok, "tt_slots": t}) == 8                                # slot twice (I2)
    t = tt.copy(); t[0] = 5 * S
    assert vto.validate(**{**ok, "tt_slots": t}) == 7                                # outside own blocks
    assert vto.validate(**{**ok, "bt_blocks": np.array([0, 1, 1], np.int32)}) == 3   # shared block


def test_semantic_checker_accepts_permuted_reclaimed_list_and_rejects_defects():
    w = wl.mistral7b_random(seed=5, requests=5, lo=30, hi=90, layers=1, heads=1, head_dim=8, block_size=4)
    p = vto.plan_workload(w)
    args = (w.block_size, w.bt_offsets, w.bt_blocks, w.tt_offsets, w.tt_slots, w.keep, w.free_blocks)
    assert vto.check_semantics(*args, p.new_bt_offsets, p.new_bt_blocks, p.new_tt_slots,
                               p.freed_blocks[::-1].copy(), p.num_free_consumed, p.req_status) == 0
    bad_tt = p.new_tt_slots.copy()
    i, j = np.flatnonzero(bad_tt >= 0)[:2]
    bad_tt[i], bad_tt[j] = bad_tt[j], bad_tt[i]                                      # logical order broken
    assert vto.check_semantics(*args, p.new_bt_offsets, p.new_bt_blocks, bad_tt,
                               p.freed_blocks, p.num_free_consumed, p.req_status) != 0
    assert vto.check_semantics(*args, p.new_bt_offsets, p.new_bt_blocks, p.new_tt_slots,
                               p.freed_blocks[:-1], p.num_free_consumed, p.req_status) != 0


# ------------------------------------------------------------------------------------------
# waste ratio F (Sec. 2.3.1)
# ------------------------------------------------------------------------------------------
def test_waste_ratio_definition_and_expectation():
    S = 16
    # by hand: 3 blocks, 10 + 0 + 2 live tokens -> F = 1 - 12/48
    bt, tt = identity_request(48, S)
    keep = np.zeros(48, np.uint8)
    keep[:10] = 1
    keep[32:34] = 1
    assert vto.waste_ratio(S, 3, tt, keep) == pytest.approx(1 - 12 / 48)
    # per-block form 1 - mean(u_b) gives the same number
    n_b = np.bincount(tt[keep != 0] // S, minlength=3)
    assert vto.waste_ratio(S, 3, tt, keep) == pytest.approx(1 - np.mean(n_b / S))
    # i.i.d. keep probability p on full blocks: E[F] = 1 - p
    rng = np.random.default_rng(0)
    bt, tt = identity_request(16 * 4000, S)
    keep = (rng.random(len(tt)) < 0.3).astype(np.uint8)
    assert vto.waste_ratio(S, 4000, tt, keep) == pytest.approx(0.7, abs=0.01)
    # after a repack the only waste left is the tail of each request's last block
    p = vto.plan(S, [0, 4000], bt, [0, len(tt)], tt, keep, np.arange(4000, 8000, dtype=np.int32))
    n = int(keep.sum())
    assert vto.waste_ratio(S, p.num_free_consumed, p.new_tt_slots) == pytest.approx(1 - n / (-(-n // S) * S))
