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


# ---- discriminating power: the digest definition is frozen; these pins say what it must tell apart ----
def _one_request(seed=9, tokens=40, layers=3, head_dim=32):
    """One request on an identity layout, everything kept: tt_slots, pools [L, slots, row] of 64-byte rows."""
    w = wl.tiny(seed=seed, requests=1, lo=tokens, hi=tokens, p_keep=1.0, layers=layers, heads=1, head_dim=head_dim)
    k, v = pools(w)
    tt = w.tt_slots[w.tt_offsets[0]:w.tt_offsets[1]].copy()
    return w, k, v, tt


def test_digest_tells_every_word_swap_inside_a_group_apart():
    """The four 8-byte words of a 32-byte group enter one product: each is bound to its place by its own
    key, so exchanging any two of them (within a group, across the two groups of a row, across rows)
    must change the digest."""
    w, k, v, tt = _one_request()
    base = vto.digest_logical(k, v, tt)[0]
    seen = {base}
    row = k[1, tt[5]].view("<u8")                      # 64-byte row: words 0..3 = group 0, 4..7 = group 1
    assert len(row) == 8 and len(set(row.tolist())) == 8
    for a in range(8):
        for b in range(a + 1, 8):
            k2 = k.copy()
            r2 = k2[1, tt[5]].view("<u8")
            r2[a], r2[b] = row[b], row[a]
            d = vto.digest_logical(k2, v, tt)[0]
            assert d not in seen, (a, b)
            seen.add(d)
    # the same word pair exchanged between two different rows of the slab
    k2 = k.copy()
    x, y = k2[0, tt[3]].view("<u8"), k2[0, tt[4]].view("<u8")
    x[2], y[2] = k[0, tt[4]].view("<u8")[2], k[0, tt[3]].view("<u8")[2]
    assert vto.digest_logical(k2, v, tt)[0] not in seen


def test_digest_tells_rows_slabs_and_layers_apart():
    w, k, v, tt = _one_request()
    base = vto.digest_logical(k, v, tt)[0]
    # a row exchanged between two requests: request A takes one slot of request B and the other way round
    w2 = wl.mistral7b_random(seed=8, requests=2, lo=30, hi=60, layers=2, heads=1, head_dim=16, rho_lo=1.0, rho_hi=1.0)
    k2, v2 = pools(w2)
    ta = w2.tt_slots[w2.tt_offsets[0]:w2.tt_offsets[1]].copy()
    tb = w2.tt_slots[w2.tt_offsets[1]:w2.tt_offsets[2]].copy()
    da, db = vto.digest_logical(k2, v2, ta)[0], vto.digest_logical(k2, v2, tb)[0]
    ta2, tb2 = ta.copy(), tb.copy()
    ta2[7], tb2[11] = tb[11], ta[7]
    assert vto.digest_logical(k2, v2, ta2)[0] != da and vto.digest_logical(k2, v2, tb2)[0] != db
    # K and V exchanged as a whole, and for one layer only
    assert vto.digest_logical(v, k, tt)[0] != base
    k3, v3 = k.copy(), v.copy()
    k3[1], v3[1] = v[1], k[1]
    assert vto.digest_logical(k3, v3, tt)[0] != base
    # layers permuted (both pools alike), every permutation of three layers
    import itertools
    seen = {base}
    for perm in itertools.permutations(range(3)):
        if perm == (0, 1, 2):
            continue
        d = vto.digest_logical(np.ascontiguousarray(k[list(perm)]), np.ascontiguousarray(v[list(perm)]), tt)[0]
        assert d not in seen, perm
        seen.add(d)
    # a sub-range of layers is a different digest from the whole
    assert vto.digest_logical(k, v, tt, 0, 2)[0] != base


def test_digest_of_ten_thousand_single_bit_flips_never_collides():
    """10 000 different single-bit flips of one request's K/V bytes: every one of them changes the digest
    (zero collisions with the intact digest).  Two DIFFERENT flips may give the same digest in exactly one
    way, which the definition implies and this test pins down: words j and j + 2 of a 32-byte group are
    added before the multiply, so flipping the same bit position in both moves the sum by the same power
    of two when the two bits agree (after the per-word keys); every collision among the flips must be of
    that kind.  (The digest is a relocation check -- rows, tokens, slabs, words in the wrong place -- not
    an error-correcting code.)  Evaluated incrementally: the digest is a sum over (token, slab, group)
    terms, so a flip changes exactly one term, recomputed here with numpy and checked against the oracle
    on a sample."""
    w, k, v, tt = _one_request(tokens=64, layers=4, head_dim=64)        # 128-byte rows, 8 slabs
    L, n = k.shape[0], len(tt)
    base = vto.digest_logical(k, v, tt)[0]
    rng = np.random.default_rng(5)
    M = (1 << 64) - 1
    row_bits = k.shape[2] * 16

    def term(kk, vv, tok, slab):
        """Digest contribution of (token tok, slab): numpy evaluation of the one row with its own key."""
        src = (kk if slab < L else vv)[slab % L, tt[tok]]
        words = np.ascontiguousarray(src).view("<u8").astype(np.uint64)[None, None, :]
        with np.errstate(over="ignore"):
            key = mix(np.array([((tok * A + tok) * B + slab) * C & M], dtype=np.uint64))[None, None, :]
            j = np.arange(words.shape[-1], dtype=np.uint64)[None, None, :]
            x = words ^ (key + j * np.uint64(D))
            a_, b_ = x[..., 0::4] + x[..., 2::4], x[..., 1::4] + x[..., 3::4]
            return int(fold128(a_, b_).sum(dtype=np.uint64))

    # the decomposition is exact: the sum of all terms is the oracle's digest (rank == id here: every token kept)
    assert sum(term(k, v, t, s) for t in range(n) for s in range(2 * L)) & M == base
    seen = {}
    checked_in_full = 0
    collisions = 0
    flips = rng.choice(n * 2 * L * row_bits, size=10000, replace=False)         # 10 000 different bits
    for trial, f in enumerate(flips.tolist()):
        tok, slab, bit = f // (2 * L * row_bits), f // row_bits % (2 * L), f % row_bits
        pool = k if slab < L else v
        old = term(k, v, tok, slab)
        pool[slab % L, tt[tok], bit // 16] ^= np.uint16(1 << (bit % 16))
        new = term(k, v, tok, slab)
        d = (base - old + new) & M
        if trial % 500 == 0:                                            # the shortcut against the oracle itself
            assert vto.digest_logical(k, v, tt)[0] == d
            checked_in_full += 1
        pool[slab % L, tt[tok], bit // 16] ^= np.uint16(1 << (bit % 16))
        assert d != base, (tok, slab, bit)                              # every flip is detected
        if d in seen:
            tok2, slab2, bit2 = seen[d]
            # same token, slab and group, same bit position, words two apart
            assert (tok2, slab2) == (tok, slab) and bit2 // 256 == bit // 256 and bit2 % 64 == bit % 64 and \
                abs(bit2 // 64 - bit // 64) == 2, ((tok, slab, bit), (tok2, slab2, bit2))
            collisions += 1
        seen[d] = (tok, slab, bit)
    assert checked_in_full == 20 and len(seen) + collisions == 10000
    assert collisions < 150                                             # about 50 expected from the pair count
