"""Pins of the oracle's relocation digest: an independent vectorised numpy evaluation of the
same formula, invariance under a repack, and sensitivity to every defect it exists to catch."""
import numpy as np

from oracle import vto
from paper_2608_13263_b200 import workloads as wl

A, B, C, D = 0x9E3779B97F4A7C15, 0xD1B54A32D192ED03, 0x8CB92BA72F3D8DD7, 0xA0761D6478BD642F


def mix(x):
    x = x.astype(np.uint64, copy=True)
    with np.errstate(over="ignore"):
        x ^= x >> np.uint64(30)
        x *= np.uint64(0xBF58476D1CE4E5B9)
        x ^= x >> np.uint64(27)
        x *= np.uint64(0x94D049BB133111EB)
        x ^= x >> np.uint64(31)
    return x


def numpy_digest(k, v, tt_slots, keep, l0, l1):
    live = np.flatnonzero((tt_slots >= 0) & (keep != 0))
    slots = tt_slots[live]
    rows = np.concatenate([k[l0:l1, slots], v[l0:l1, slots]], axis=0)          # [2*nl, n, row]
    words = np.ascontiguousarray(rows).view("<u8")                             # [2*nl, n, row_bytes / 8]
    S_, n, W = words.shape
    with np.errstate(over="ignore"):
        i = np.arange(n, dtype=np.uint64)[None, :, None]
        t = live.astype(np.uint64)[None, :, None]
        s = np.arange(S_, dtype=np.uint64)[:, None, None]
        j = np.arange(W, dtype=np.uint64)[None, None, :]
        key = mix(((i * np.uint64(A) + t) * np.uint64(B) + s) * np.uint64(C))       # per (token, slab)
        total = mix(words ^ (key + j * np.uint64(D))).sum(dtype=np.uint64)
    return int(total), n


def pools(w, seed=1):
    k = np.stack([wl.fill_slab(seed, 0, l, w.num_layers, w.slots_per_layer, w.row_elems) for l in range(w.num_layers)])
    v = np.stack([wl.fill_slab(seed, 1, l, w.num_layers, w.slots_per_layer, w.row_elems) for l in range(w.num_layers)])
    return k, v


def test_digest_equals_vectorised_numpy_evaluation():
    w = wl.steady_state(seed=2, requests=6, lo=50, hi=300, layers=3, heads=1, head_dim=8)
    k, v = pools(w)
    for r in range(w.num_requests):
        t0, t1 = w.tt_offsets[r], w.tt_offsets[r + 1]
        for l0, l1 in ((0, 3), (1, 2)):
            assert vto.digest_logical(k, v, w.tt_slots[t0:t1], w.keep[t0:t1], l0, l1) == \
                   numpy_digest(k, v, w.tt_slots[t0:t1], w.keep[t0:t1], l0, l1)


def test_digest_is_invariant_under_repack_and_catches_defects():
    w = wl.mistral7b_random(seed=4, requests=5, lo=60, hi=200, layers=2, heads=1, head_dim=8)
    k, v = pools(w)
    p = vto.plan_workload(w)
    k2, v2 = k.copy(), v.copy()
    vto.apply_moves_pools(k2, v2, p.move_src, p.move_dst)
    assert p.num_moves > 0
    for r in range(w.num_requests):
        t0, t1 = w.tt_offsets[r], w.tt_offsets[r + 1]
        before = vto.digest_logical(k, v, w.tt_slots[t0:t1], w.keep[t0:t1])
        after = vto.digest_logical(k2, v2, p.new_tt_slots[t0:t1])
        assert before == after                                           # token conservation (I1)
        new = p.new_tt_slots[t0:t1].copy()
        live = np.flatnonzero(new >= 0)
        if len(live) < 3:
            continue
        swapped = new.copy()
        swapped[live[0]], swapped[live[1]] = new[live[1]], new[live[0]]  # two tokens exchanged
        assert vto.digest_logical(k2, v2, swapped) != after
        lost = new.copy()
        lost[live[2]] = -1                                               # a token lost
        assert vto.digest_logical(k2, v2, lost) != after
        dup = new.copy()
        dup[live[2]] = new[live[1]]                                      # a slot referenced twice
        assert vto.digest_logical(k2, v2, dup) != after
        shifted = np.concatenate([[-1], new])[:len(new)]                 # same payloads under different ids
        assert vto.digest_logical(k2, v2, shifted) != after
        k3 = k2.copy()
        k3[1, new[live[0]], 3] ^= 1                                      # one bit of one K row
        assert vto.digest_logical(k3, v2, new) != after
