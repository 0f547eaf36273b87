"""GPU parity of the input-precondition checker against the oracle's order-free checker: valid
workloads, one planted defect per bit, random corruptions, shared prefixes, full-size tables."""
import numpy as np
import pytest

from oracle import vto
from paper_2608_13263_b200 import binding as vt
from harness import workloads as wl

from test_oracle_check_tables import BIT, plant, recipes

pytestmark = pytest.mark.gpu


class Checker:
    """A context over a one-layer dummy pool (the checker reads tables only) and device buffers
    sized for a workload, re-uploadable with corrupted tables."""

    def __init__(self, w, slack=8):
        import torch
        self.torch = torch
        self.w = w
        dev = torch.device("cuda:0")
        self.dev = dev
        self.pool = torch.zeros((1, w.slots_per_layer, 8), dtype=torch.int16, device=dev)
        self.cap_bt = len(w.bt_blocks) + slack
        self.cap_tt = w.num_tokens + slack
        self.cap_free = len(w.free_blocks) + slack
        self.ctx = vt.vtoken_create(1, w.num_blocks, w.block_size, 1, 8, self.pool, self.pool, w.num_requests,
                                    self.cap_tt, self.cap_bt, self.cap_free)
        i32 = dict(dtype=torch.int32, device=dev)
        self.bt_offsets = torch.zeros(w.num_requests + 1, **i32)
        self.tt_offsets = torch.zeros(w.num_requests + 1, **i32)
        self.bt_blocks = torch.zeros(self.cap_bt, **i32)
        self.tt_slots = torch.zeros(self.cap_tt, **i32)
        self.free_blocks = torch.zeros(self.cap_free, **i32)
        self.num_free = torch.zeros(1, **i32)
        self.num_requests = torch.tensor([w.num_requests], **i32)
        self.bits = torch.full((1,), 0x7fffffff, **i32)
        self.protect = torch.zeros(w.num_blocks, dtype=torch.uint8, device=dev)

    def run(self, bt_offsets=None, bt_blocks=None, tt_offsets=None, tt_slots=None, free_blocks=None, protect=None,
            **_):
        t, w = self.torch, self.w
        up = lambda dst, a: dst[:len(a)].copy_(t.from_numpy(np.ascontiguousarray(a, np.int32)))
        up(self.bt_offsets, w.bt_offsets if bt_offsets is None else bt_offsets)
        up(self.tt_offsets, w.tt_offsets if tt_offsets is None else tt_offsets)
        up(self.bt_blocks, w.bt_blocks if bt_blocks is None else bt_blocks)
        up(self.tt_slots, w.tt_slots if tt_slots is None else tt_slots)
        free = w.free_blocks if free_blocks is None else free_blocks
        up(self.free_blocks, free)
        self.num_free.fill_(len(free))
        if protect is not None:
            self.protect.copy_(t.from_numpy(protect))
        vt.vtoken_check_tables(self.ctx, num_requests=self.num_requests, bt_offsets=self.bt_offsets,
                               bt_blocks=self.bt_blocks, tt_offsets=self.tt_offsets, tt_slots=self.tt_slots,
                               free_blocks=self.free_blocks, num_free=self.num_free, out_bits=self.bits,
                               protect=self.protect if protect is not None else None)
        t.cuda.synchronize()
        return int(self.bits.item())

    def close(self):
        self.torch.cuda.synchronize()
        vt.vtoken_destroy(self.ctx)


def oracle_bits(w, protect=None, **over):
    a = dict(S=w.block_size, NB=w.num_blocks, bt_offsets=w.bt_offsets, bt_blocks=w.bt_blocks, tt_offsets=w.tt_offsets,
             tt_slots=w.tt_slots, free_blocks=w.free_blocks, protect=protect)
    a.update(over)
    return vto.check_tables(**a)


@pytest.mark.parametrize("w", list(recipes()), ids=lambda w: w.name)
def test_valid_and_planted_defects(w):
    rng = np.random.default_rng(7)
    ck = Checker(w)
    assert ck.run() == 0 == oracle_bits(w)
    for kind in ("block_range", "block_twice", "free_range", "free_twice_or_held", "slot_range", "foreign_slot",
                 "slot_twice"):
        over = plant(w, kind, rng)
        got = ck.run(**over)
        assert got == oracle_bits(w, **over) and got & BIT[kind], kind
    # broken offsets: only that bit
    off = w.tt_offsets.copy()
    off[1], off[2] = off[2], off[1] + 0
    if off[2] < off[1]:
        assert ck.run(tt_offsets=off) == 1 == oracle_bits(w, tt_offsets=off)
    assert ck.run() == 0                      # the scratch is reset by every call
    ck.close()


def test_random_corruptions():
    rng = np.random.default_rng(11)
    w = wl.mistral7b_random(seed=9, requests=6, lo=10, hi=60, layers=1, heads=1, head_dim=8, block_size=4)
    ck = Checker(w)
    seen = set()
    for _ in range(200):
        bt, tt, free = w.bt_blocks.copy(), w.tt_slots.copy(), w.free_blocks[:12].copy()
        for _ in range(int(rng.integers(1, 4))):
            which = rng.integers(3)
            if which == 0:
                bt[rng.integers(len(bt))] = rng.integers(-2, w.num_blocks + 2)
            elif which == 1:
                tt[rng.integers(len(tt))] = rng.integers(-1, w.num_blocks * 4 + 3)
            else:
                free[rng.integers(len(free))] = rng.integers(-1, w.num_blocks + 1)
        got = ck.run(bt_blocks=bt, tt_slots=tt, free_blocks=free)
        assert got == oracle_bits(w, bt_blocks=bt, tt_slots=tt, free_blocks=free)
        seen.add(got)
    assert len(seen) > 10
    ck.close()


def test_shared_prefix_needs_the_protect_mask():
    w, p = wl.shared_prefix(seed=1, groups=2, degree=3, prefix_len=64, suffix_len=80, layers=1, heads=1, head_dim=8)
    ck = Checker(w)
    assert ck.run(protect=p) == 0 == oracle_bits(w, protect=p)
    assert ck.run() == (4 | 128) == oracle_bits(w)
    ck.close()


def test_full_size_tables_and_a_single_duplicate_slot():
    """Steady-state tables (2.2 M entries, 48 k blocks): valid; then one slot duplicated in one
    request is found (I2), and nothing else is reported."""
    w = wl.steady_state(seed=0)
    ck = Checker(w)
    assert ck.run() == 0
    tt = w.tt_slots.copy()
    live = np.flatnonzero(tt >= 0)
    r_of = np.searchsorted(w.tt_offsets, live, side="right") - 1
    i = len(live) // 2
    j = i + 1 if r_of[i + 1] == r_of[i] else i - 1
    tt[live[j]] = tt[live[i]]
    assert ck.run(tt_slots=tt) == 128 == oracle_bits(w, tt_slots=tt)
    ck.close()
