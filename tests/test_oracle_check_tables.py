"""Pins of the oracle's order-free table checker (every violated precondition as a bit): a
set-based Python statement of the same definitions, the relation to the first-failure validator,
one planted defect per bit on every workload recipe, and random corruptions (no GPU)."""
from collections import Counter

import numpy as np
import pytest

from oracle import vto
from harness import workloads as wl

BIT = {"offsets": 1, "block_range": 2, "block_twice": 4, "free_range": 8, "free_twice_or_held": 16,
       "slot_range": 32, "foreign_slot": 64, "slot_twice": 128}
# code of vto_validate (first failure) -> bit of vto_check_tables
FIRST_TO_BIT = {1: 1, 2: 2, 3: 4, 4: 8, 5: 16, 6: 32, 7: 64, 8: 128}


def check(w, **over):
    a = dict(S=w.block_size, NB=w.num_blocks, bt_offsets=w.bt_offsets, bt_blocks=w.bt_blocks, tt_offsets=w.tt_offsets,
             tt_slots=w.tt_slots, free_blocks=w.free_blocks)
    a.update(over)
    return vto.check_tables(**a), a


def twin(S, NB, bt_offsets, bt_blocks, tt_offsets, tt_slots, free_blocks, protect=None):
    """The definitions with Counters and sets."""
    R = len(tt_offsets) - 1
    f = 0
    if any(bt_offsets[r + 1] < bt_offsets[r] or tt_offsets[r + 1] < tt_offsets[r] for r in range(R)):
        return 1
    tables = [[int(b) for b in bt_blocks[bt_offsets[r]:bt_offsets[r + 1]]] for r in range(R)]
    flat = [b for t in tables for b in t]
    if any(not 0 <= b < NB for b in flat):
        f |= 2
    held = Counter(b for b in flat if 0 <= b < NB)
    if any(c > 1 and not (protect is not None and protect[b]) for b, c in held.items()):
        f |= 4
    free = [int(b) for b in free_blocks]
    if any(not 0 <= b < NB for b in free):
        f |= 8
    fc = Counter(b for b in free if 0 <= b < NB)
    if any(c > 1 or b in held for b, c in fc.items()):
        f |= 16
    holders = {}
    for r, t in enumerate(tables):
        for b in set(t):
            holders.setdefault(b, set()).add(r)
    refs = Counter()
    for r in range(R):
        for s in tt_slots[tt_offsets[r]:tt_offsets[r + 1]]:
            s = int(s)
            if s < 0:
                continue
            if s >= NB * S:
                f |= 32
                continue
            h = holders.get(s // S, set())
            if len(h) == 0 or (len(h) == 1 and r not in h):
                f |= 64
            refs[s] += 1
    if any(c > 1 and not (protect is not None and protect[s // S]) for s, c in refs.items()):
        f |= 128
    return f


def recipes():
    yield wl.tiny(seed=0)
    yield wl.llama8b_h2o(seed=1, requests=5, lo=100, hi=400, layers=1, heads=1, head_dim=8)
    yield wl.mistral7b_random(seed=2, requests=9, lo=20, hi=200, layers=1, heads=1, head_dim=8)
    yield wl.steady_state(seed=4, requests=12, lo=100, hi=600, layers=1, heads=1, head_dim=8)
    yield wl.longctx_scissor(seed=3, requests=3, lo=900, hi=1500, layers=1, heads=1, head_dim=8)


def plant(w, kind, rng):
    """One defect of the named kind; returns the overriding arguments."""
    bt, tt, free = w.bt_blocks.copy(), w.tt_slots.copy(), w.free_blocks.copy()
    live = np.flatnonzero(tt >= 0)
    if kind == "block_range":
        bt[rng.integers(len(bt))] = w.num_blocks + 3
        return dict(bt_blocks=bt)
    if kind == "block_twice":
        r = int(np.argmax(np.diff(w.bt_offsets) >= 2))
        bt[w.bt_offsets[r]] = bt[w.bt_offsets[r] + 1]            # one of its own blocks twice
        return dict(bt_blocks=bt)
    if kind == "free_range":
        free[rng.integers(len(free))] = -1
        return dict(free_blocks=free)
    if kind == "free_twice_or_held":
        if rng.random() < 0.5:
            free[0] = free[1]
        else:
            free[0] = bt[rng.integers(len(bt))]
        return dict(free_blocks=free)
    if kind == "slot_range":
        tt[live[rng.integers(len(live))]] = w.num_blocks * w.block_size + 1
        return dict(tt_slots=tt)
    if kind == "foreign_slot":
        tt[live[rng.integers(len(live))]] = int(free[0]) * w.block_size    # a slot in a free block
        return dict(tt_slots=tt)
    if kind == "slot_twice":
        i, j = rng.choice(len(live), 2, replace=False)
        r_of = np.searchsorted(w.tt_offsets, live, side="right") - 1
        same = np.flatnonzero(r_of == r_of[i])
        j = same[0] if same[0] != i else same[1]
        tt[live[j]] = tt[live[i]]                                          # two tokens of one request, one slot
        return dict(tt_slots=tt)
    raise KeyError(kind)


@pytest.mark.parametrize("w", list(recipes()), ids=lambda w: w.name)
def test_valid_inputs_and_one_planted_defect_per_bit(w):
    rng = np.random.default_rng(7)
    bits, a = check(w)
    assert bits == 0 == twin(**a) and vto.validate(w.block_size, w.num_blocks, w.bt_offsets, w.bt_blocks,
                                                   w.tt_offsets, w.tt_slots, w.keep, w.free_blocks) == 0
    for kind in ("block_range", "block_twice", "free_range", "free_twice_or_held", "slot_range", "foreign_slot",
                 "slot_twice"):
        bits, a = check(w, **plant(w, kind, rng))
        assert bits & BIT[kind], kind
        assert bits == twin(**a), kind
        # the first-failure validator names one of the reported bits
        first = vto.validate(a["S"], a["NB"], a["bt_offsets"], a["bt_blocks"], a["tt_offsets"], a["tt_slots"],
                             np.ones(len(a["tt_slots"]), np.uint8), a["free_blocks"])
        assert first != 0 and bits & FIRST_TO_BIT[first], (kind, first, bits)


def test_offsets_and_empty_inputs():
    assert vto.check_tables(4, 8, [0, 3, 2], [0, 1, 2], [0, 1, 2], [0, 4], []) == 1
    assert vto.check_tables(4, 8, [0, 1, 2], [0, 1], [0, 2, 1], [0, 4], []) == 1
    assert vto.check_tables(4, 8, [0], [], [0], [], []) == 0
    assert vto.check_tables(4, 8, [0, 0], [], [0, 3], [-1, -1, -1], [1, 2]) == 0


def test_shared_blocks_with_and_without_protection():
    """A block held by two requests: bit 4 unless protected; slots inside it are not 'foreign' for
    anybody (the check does not apply), slots in a block held by one other request are."""
    S, NB = 4, 10
    bt_offsets, bt_blocks = [0, 2, 4], [7, 1, 7, 2]
    tt_offsets = [0, 3, 6]
    tt_slots = [28, 29, 4, 30, 8, 5]         # request 1: slot 30 in shared block 7, slot 8 own, slot 5 in block 1
    protect = np.zeros(NB, np.uint8)
    args = (S, NB, bt_offsets, bt_blocks, tt_offsets, tt_slots, [3])
    assert vto.check_tables(*args) == 4 | 64 == twin(*args)
    protect[7] = 1
    assert vto.check_tables(*args, protect=protect) == 64 == twin(*args, protect=protect)
    tt_ok = [28, 29, 4, 30, 8, -1]
    assert vto.check_tables(S, NB, bt_offsets, bt_blocks, tt_offsets, tt_ok, [3], protect=protect) == 0
    w, p = wl.shared_prefix(seed=1, groups=2, degree=3, prefix_len=64, suffix_len=80, layers=1, heads=1, head_dim=8)
    assert vto.check_tables(w.block_size, w.num_blocks, w.bt_offsets, w.bt_blocks, w.tt_offsets, w.tt_slots,
                            w.free_blocks, protect=p) == 0
    assert vto.check_tables(w.block_size, w.num_blocks, w.bt_offsets, w.bt_blocks, w.tt_offsets, w.tt_slots,
                            w.free_blocks) == 4 | 128      # unprotected: blocks held and slots mapped several times


def test_boundaries_of_the_slot_checks():
    S, NB = 4, 6
    # the first slot beyond the pool is out of range; the last slot of the pool is not
    assert vto.check_tables(S, NB, [0, 1], [5], [0, 2], [23, 24], []) == 32
    assert vto.check_tables(S, NB, [0, 1], [5], [0, 2], [23, 20], []) == 0
    # a block listed twice by ONE request has one holder: another request's slot in it is foreign
    args = (S, NB, [0, 2, 3], [3, 3, 1], [0, 1, 2], [12, 13], [])
    assert vto.check_tables(*args) == 4 | 64 == twin(*args)


def test_random_corruptions_against_the_twin():
    rng = np.random.default_rng(11)
    w = wl.mistral7b_random(seed=9, requests=6, lo=10, hi=60, layers=1, heads=1, head_dim=8, block_size=4)
    seen = set()
    for _ in range(300):
        bt, tt, free = w.bt_blocks.copy(), w.tt_slots.copy(), w.free_blocks[:12].copy()
        for _ in range(int(rng.integers(1, 4))):
            which = rng.integers(3)
            if which == 0:
                bt[rng.integers(len(bt))] = rng.integers(-2, w.num_blocks + 2)
            elif which == 1:
                tt[rng.integers(len(tt))] = rng.integers(-1, w.num_blocks * 4 + 3)
            else:
                free[rng.integers(len(free))] = rng.integers(-1, w.num_blocks + 1)
        a = dict(S=4, NB=w.num_blocks, bt_offsets=w.bt_offsets, bt_blocks=bt, tt_offsets=w.tt_offsets, tt_slots=tt,
                 free_blocks=free)
        bits = vto.check_tables(**a)
        assert bits == twin(**a)
        seen.add(bits)
    assert len(seen) > 10
