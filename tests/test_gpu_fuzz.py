"""Seeded fuzz of the whole path against the oracle: random shapes, block sizes, masks, table holes,
selections, thresholds, free-list lengths and partial-plan options, whole pools compared."""
import os

import numpy as np
import pytest

from oracle import vto
from harness import workloads as wl

pytestmark = pytest.mark.gpu

# more seeds for a soak run: VTOKEN_FUZZ_SCALE=10 runs ten times as many problems
FUZZ_SCALE = max(1, int(os.environ.get("VTOKEN_FUZZ_SCALE", "1")))


def random_problem(rng):
    S = int(rng.choice([1, 2, 3, 4, 8, 16, 32, 48]))
    heads, head_dim = [(1, 8), (1, 64), (2, 128), (4, 128), (8, 128)][int(rng.integers(0, 5))]
    R = int(rng.integers(1, 12))
    layers = int(rng.integers(1, 4))
    lens = rng.integers(0, 40 * S + 2, size=R)
    residents, keeps = [], []
    for n in lens:
        n = int(n)
        resident = np.flatnonzero(rng.random(n) < rng.choice([1.0, 0.9, 0.5]))       # -1 holes in the table
        keep = rng.random(n) < rng.uniform(0.0, 1.0)
        if rng.random() < 0.15:
            keep[:] = True
        if rng.random() < 0.1:
            keep[:] = False
        residents.append(resident.astype(np.int64))
        keeps.append(keep)                                                          # may keep a hole: not live
    gen = np.random.Generator(np.random.PCG64(int(rng.integers(0, 1 << 30))))
    w = wl._assemble("fuzz", (layers, heads, head_dim), S, lens, residents, keeps, gen, 0,
                     headroom=int(rng.integers(1, 6)))
    if rng.random() < 0.4:
        w.select = rng.integers(0, 2, size=R).astype(np.uint8)
    if rng.random() < 0.4:
        w.thr_num, w.thr_den = [(1, 4), (1, 2), (3, 4), (1, 1), (5, 7)][int(rng.integers(0, 5))]
    return w


@pytest.mark.parametrize("seed", range(60 * FUZZ_SCALE))
def test_fuzz_whole_and_partial_plans(seed):
    import torch
    from harness.device import DeviceProblem
    rng = np.random.default_rng(1000 + seed)
    w = random_problem(rng)
    S = w.block_size
    num_free = None if rng.random() < 0.5 else int(rng.integers(0, len(w.free_blocks) + 1))
    partial = rng.random() < 0.5
    opts = {}
    if partial:
        opts = dict(util=[(0, 0), (1, 1), (1, 2), (3, 4)][int(rng.integers(0, 4))],
                    max_source_blocks=int(rng.choice([0, 0, 1, 3, 10])),
                    theta=[(0, 0), (1, 4), (9, 10)][int(rng.integers(0, 3))])
        if rng.random() < 0.4:
            opts["protect"] = (rng.random(w.num_blocks) < 0.2).astype(np.uint8)
            if rng.random() < 0.6:
                opts["detach"] = [(1, 1), (1, 2), (3, 4)][int(rng.integers(0, 3))]
                # (a generator of its own: the problems of the other seeds stay what they were)
                opts["detach_rule"] = int(np.random.default_rng(5000 + seed).integers(0, 3))
    variant = int(rng.choice([0, 1, 2])) if w.row_bytes >= 16 else 1
    prob = DeviceProblem(w, fill_seed=seed, copy_variant=variant)
    from paper_2608_13263_b200 import binding as vt
    before = _digest(prob, vt, prob.tt_slots, prob.keep) if w.row_bytes % 16 == 0 else None
    nf_dev = None if num_free is None else torch.tensor([num_free], dtype=torch.int32, device=prob.device)
    if partial:
        dopts = dict(opts)
        if "protect" in opts:
            dopts["protect"] = torch.from_numpy(opts["protect"]).to(prob.device)
        prob.plan_partial(num_free=nf_dev, **dopts)
        p = vto.plan_partial(S, w.num_blocks, w.bt_offsets, w.bt_blocks, w.tt_offsets, w.tt_slots, w.keep,
                             w.free_blocks, w.select, w.thr_num, w.thr_den, num_free=num_free, **opts)
    else:
        prob.plan(num_free=nf_dev)
        p = vto.plan_workload(w, num_free=num_free)
    prob.repack()
    out = prob.outputs()
    assert out["error_flags"] == 0
    for n in ("num_moves", "num_dst_blocks", "num_freed", "num_free_consumed", "num_admitted", "num_deferred"):
        assert out[n] == getattr(p, n), n
    assert np.array_equal(out["req_status"], p.req_status)
    assert np.array_equal(out["new_bt_offsets"], p.new_bt_offsets)
    assert np.array_equal(out["new_bt_blocks"], p.new_bt_blocks)
    assert np.array_equal(out["new_tt_slots"], p.new_tt_slots)
    assert np.array_equal(out["freed_blocks"], p.freed_blocks)
    if partial:
        assert np.array_equal(out["released_blocks"], p.released_blocks)
    if before is not None:          # relocation check: same digest through the new table (token conservation)
        assert np.array_equal(before, _digest(prob, vt, prob.new_tt_slots, None))
    k = np.stack([wl.fill_slab(seed, 0, l, w.num_layers, w.slots_per_layer, w.row_elems) for l in range(w.num_layers)])
    v = np.stack([wl.fill_slab(seed, 1, l, w.num_layers, w.slots_per_layer, w.row_elems) for l in range(w.num_layers)])
    vto.apply_moves_pools(k, v, p.move_src, p.move_dst)
    assert np.array_equal(prob.k_pool.cpu().numpy().view(np.uint16), k)
    assert np.array_equal(prob.v_pool.cpu().numpy().view(np.uint16), v)
    prob.close()


@pytest.mark.parametrize("seed", range(24 * FUZZ_SCALE))
def test_fuzz_repack_in_waves(seed):
    """Random problems through vtoken_repack_waves (short pools, whole and partial planners): all
    outputs and whole pools against the oracle's wave plan, and the relocation digest of every
    request is the same before and after."""
    import torch
    from paper_2608_13263_b200 import binding as vt
    from harness.device import DeviceProblem
    rng = np.random.default_rng(5000 + seed)
    w = random_problem(rng)
    S = w.block_size
    num_free = int(rng.integers(0, min(len(w.free_blocks), 12) + 1))
    waves = int(rng.integers(1, 6))
    partial = None
    if rng.random() < 0.5:
        partial = dict(util=[(0, 0), (1, 1), (1, 2), (3, 4)][int(rng.integers(0, 4))],
                       max_source_blocks=int(rng.choice([0, 1, 2, 5])),
                       theta=[(0, 0), (1, 4)][int(rng.integers(0, 2))])
    variant = int(rng.choice([0, 1, 2])) if w.row_bytes >= 16 else 1
    prob = DeviceProblem(w, fill_seed=seed, copy_variant=variant, wave_capacity=True)
    digest = lambda tt, keep: _digest(prob, vt, tt, keep)
    before = digest(prob.tt_slots, prob.keep) if w.row_bytes % 16 == 0 else None
    prob.repack_waves(waves, num_free=torch.tensor([num_free], dtype=torch.int32, device=prob.device), partial=partial)
    out = prob.waves_outputs(waves)
    v = vto.plan_waves(S, w.num_blocks, w.bt_offsets, w.bt_blocks, w.tt_offsets, w.tt_slots, w.keep,
                       w.free_blocks[:num_free], waves, w.select, w.thr_num, w.thr_den, partial)
    for k in range(waves):
        assert out["wave_counts"][k]["error_flags"] == 0
        for n in ("num_moves", "num_dst_blocks", "num_freed", "num_free_consumed", "num_admitted", "num_deferred"):
            assert out["wave_counts"][k][n] == v.wave_counts[k][n], (k, n)
    for n in ("req_status", "req_wave", "req_append_pos", "new_bt_offsets", "new_bt_blocks", "new_tt_slots", "free_out"):
        assert np.array_equal(out[n], getattr(v, n)), n
    kp = np.stack([wl.fill_slab(seed, 0, l, w.num_layers, w.slots_per_layer, w.row_elems) for l in range(w.num_layers)])
    vp = np.stack([wl.fill_slab(seed, 1, l, w.num_layers, w.slots_per_layer, w.row_elems) for l in range(w.num_layers)])
    vto.apply_moves_pools(kp, vp, v.move_src, v.move_dst)
    assert np.array_equal(prob.k_pool.cpu().numpy().view(np.uint16), kp)
    assert np.array_equal(prob.v_pool.cpu().numpy().view(np.uint16), vp)
    if before is not None:
        assert np.array_equal(before, digest(prob.new_tt_slots, None))
    prob.close()


def _digest(prob, vt, tt_slots, keep):
    import torch
    dig = torch.zeros(prob.max_requests, dtype=torch.int64, device=prob.device)
    vt.vtoken_digest_logical(prob.ctx, num_requests=prob.num_requests, tt_offsets=prob.tt_offsets, tt_slots=tt_slots,
                             keep=keep, select=None, layer_begin=0, layer_end=prob.w.num_layers, out_digest=dig)
    torch.cuda.synchronize()
    return dig.cpu().numpy()[:prob.w.num_requests].copy()
