"""Pins of the oracle's relocation digest: an independent vectorised numpy evaluation of the
same formula, invariance under a repack, and sensitivity to every defect it exists to catch."""
import numpy as np

from oracle import vto
from harness import workloads as wl

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


M32 = np.uint64(0xFFFFFFFF)


def fold128(a, b):
    """low64(a*b) ^ high64(a*b) of uint64 arrays, from 32-bit halves (schoolbook product)."""
    with np.errstate(over="ignore"):
        al, ah, bl, bh = a & M32, a >> np.uint64(32), b & M32, b >> np.uint64(32)
        ll, lh, hl, hh = al * bl, al * bh, ah * bl, ah * bh
        mid = (ll >> np.uint64(32)) + (lh & M32) + (hl & M32)
        hi = hh + (lh >> np.uint64(32)) + (hl >> np.uint64(32)) + (mid >> np.uint64(32))
        return (a * b) ^ hi


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
        x = words ^ (key + j * np.uint64(D))
        if W % 4:                                      # a trailing half group: absent words add nothing
            x = np.concatenate([x, np.zeros(x.shape[:-1] + (4 - W % 4,), np.uint64)], axis=-1)
        a = x[..., 0::4] + x[..., 2::4]
        b = x[..., 1::4] + x[..., 3::4]
        total = fold128(a, b).sum(dtype=np.uint64)
    return int(total), n


def bigint_digest(k, v, tt_slots, keep):
    """The definition with Python integers (exact 128-bit products), one word pair at a time."""
    M = (1 << 64) - 1

    def mixi(x):
        x ^= x >> 30
        x = x * 0xBF58476D1CE4E5B9 & M
        x ^= x >> 27
        x = x * 0x94D049BB133111EB & M
        return x ^ x >> 31
    L = k.shape[0]
    total, i = 0, 0
    for t in range(len(tt_slots)):
        if tt_slots[t] < 0 or not keep[t]:
            continue
        for s in range(2 * L):
            row = (k if s < L else v)[s % L, tt_slots[t]].tobytes()
            key = mixi(((i * A + t) * B + s) * C & M)
            words = [int.from_bytes(row[8 * j:8 * j + 8], "little") ^ (key + j * D & M) for j in range(len(row) // 8)]
            for g in range(0, len(words), 4):
                a = sum(words[g:g + 4:2]) & M
                b = sum(words[g + 1:g + 4:2]) & M
                total = (total + ((a * b & M) ^ (a * b >> 64))) & M
        i += 1
    return total, i


def pools(w, seed=1):
    k = np.stack([wl.fill_slab(seed, 0, l, w.num_layers, w.slots_per_layer, w.row_elems) for l in range(w.num_layers)])
    v = np.stack([wl.fill_slab(seed, 1, l, w.num_layers, w.slots_per_layer, w.row_elems) for l in range(w.num_layers)])
    return k, v


def test_digest_equals_vectorised_numpy_evaluation():
    # rows of 16 bytes (half a group), 48 bytes (a group and a half) and 128 bytes (whole groups)
    for head_dim in (8, 24, 64):
        w = wl.steady_state(seed=2, requests=6, lo=50, hi=300, layers=3, heads=1, head_dim=head_dim)
        k, v = pools(w)
        for r in range(w.num_requests):
            t0, t1 = w.tt_offsets[r], w.tt_offsets[r + 1]
            for l0, l1 in ((0, 3), (1, 2)):
                assert vto.digest_logical(k, v, w.tt_slots[t0:t1], w.keep[t0:t1], l0, l1) == \
                       numpy_digest(k, v, w.tt_slots[t0:t1], w.keep[t0:t1], l0, l1)
    w = wl.tiny(seed=4, heads=1, head_dim=24)
    k, v = pools(w)
    t0, t1 = w.tt_offsets[0], w.tt_offsets[1]
    assert vto.digest_logical(k, v, w.tt_slots[t0:t1], w.keep[t0:t1]) == bigint_digest(k, v, w.tt_slots[t0:t1],
                                                                                       w.keep[t0:t1])


def test_digest_equals_exact_integer_evaluation_on_a_small_case():
    w = wl.tiny(seed=3)
    k, v = pools(w)
    for r in range(w.num_requests):
        t0, t1 = w.tt_offsets[r], w.tt_offsets[r + 1]
        assert vto.digest_logical(k, v, w.tt_slots[t0:t1], w.keep[t0:t1]) == \
               bigint_digest(k, v, w.tt_slots[t0:t1], w.keep[t0:t1])


def test_fold128_helper_against_python_integers():
    rng = np.random.default_rng(0)
    a = rng.integers(0, 2 ** 64, size=2000, dtype=np.uint64)
    b = rng.integers(0, 2 ** 64, size=2000, dtype=np.uint64)
    a[:4] = [0, 2 ** 64 - 1, 2 ** 32, 2 ** 64 - 1]
    b[:4] = [5, 2 ** 64 - 1, 2 ** 32, 1]
    want = [((int(x) * int(y)) & (2 ** 64 - 1)) ^ ((int(x) * int(y)) >> 64) for x, y in zip(a, b)]
    assert fold128(a, b).tolist() == want


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
