"""GPU parity of the eligibility metadata (per-block liveness, histogram, F) and of partial
plans (low-utilisation sources, protected blocks, source bound, global trigger) against the
oracle: tables, lists, counts and whole pools, bit-exact."""
import os

import numpy as np
import pytest

from oracle import vto
from paper_2608_13263_b200 import binding as vt
from harness import workloads as wl

pytestmark = pytest.mark.gpu

FILL_SEED = 1


def host_pools(w):
    k = np.stack([wl.fill_slab(FILL_SEED, 0, l, w.num_layers, w.slots_per_layer, w.row_elems)
                  for l in range(w.num_layers)])
    v = np.stack([wl.fill_slab(FILL_SEED, 1, l, w.num_layers, w.slots_per_layer, w.row_elems)
                  for l in range(w.num_layers)])
    return k, v


def small_configs():
    return [
        wl.tiny(seed=0),
        wl.llama8b_h2o(seed=0, requests=6, lo=300, hi=900, layers=2),
        wl.mistral7b_random(seed=0, requests=17, lo=100, hi=500, layers=2, rho_lo=0.6, rho_hi=0.97),
        wl.longctx_scissor(seed=0, requests=3, lo=3000, hi=6000, layers=1),
        wl.steady_state(seed=0, requests=24, lo=100, hi=1500, layers=2),
        wl.steady_state(seed=1, requests=24, lo=100, hi=1500, layers=1, block_size=32),
        wl.streaming_window(seed=0, requests=9, lo=200, hi=1500, window=100, layers=1),
    ]


OPTION_SETS = [
    dict(),                                               # reduces to the whole-request plan
    dict(util=(1, 1)),                                    # fully live blocks stay
    dict(util=(1, 2)),                                    # only blocks under 50 % utilisation move
    dict(util=(1, 1), max_source_blocks=7),
    dict(util=(3, 4), theta=(1, 4)),                      # the paper's default trigger
    dict(theta=(99, 100)),                                # trigger never holds
    dict(protect="prefix"),
    dict(protect="prefix", util=(1, 1), max_source_blocks=20),
]


def run_partial(w, opts, num_free=None, whole_pool=True):
    import torch
    from harness.device import DeviceProblem
    opts = dict(opts)
    protect = None
    if opts.get("protect") == "prefix":
        protect = np.zeros(w.num_blocks, np.uint8)
        for r in range(w.num_requests):
            protect[w.bt_blocks[w.bt_offsets[r]:w.bt_offsets[r + 1]][:3]] = 1
        opts["protect"] = protect
    prob = DeviceProblem(w, fill_seed=FILL_SEED)
    dopts = dict(opts)
    if protect is not None:
        dopts["protect"] = torch.from_numpy(protect).to(prob.device)
    nf_dev = None if num_free is None else torch.tensor([num_free], dtype=torch.int32, device=prob.device)
    prob.plan_partial(num_free=nf_dev, **dopts)
    prob.repack()
    out = prob.outputs()
    p = vto.plan_partial(w.block_size, w.num_blocks, w.bt_offsets, w.bt_blocks, w.tt_offsets, w.tt_slots, w.keep,
                         w.free_blocks, w.select, w.thr_num, w.thr_den, num_free=num_free, **opts)
    assert out["error_flags"] == 0
    for n in ("num_moves", "num_dst_blocks", "num_freed", "num_free_consumed", "num_admitted", "num_deferred"):
        assert out[n] == getattr(p, n), n
    assert np.array_equal(out["req_status"], p.req_status)
    assert np.array_equal(out["new_bt_offsets"], p.new_bt_offsets)
    assert np.array_equal(out["new_bt_blocks"], p.new_bt_blocks)
    assert np.array_equal(out["new_tt_slots"], p.new_tt_slots)
    assert np.array_equal(out["freed_blocks"], p.freed_blocks)
    if whole_pool:
        k, v = host_pools(w)
        vto.apply_moves_pools(k, v, p.move_src, p.move_dst, threads=2)
        assert np.array_equal(prob.k_pool.cpu().numpy().view(np.uint16), k)
        assert np.array_equal(prob.v_pool.cpu().numpy().view(np.uint16), v)
    prob.close()
    return out, p


@pytest.mark.parametrize("opts", OPTION_SETS, ids=[str(i) for i in range(len(OPTION_SETS))])
@pytest.mark.parametrize("w", small_configs(), ids=lambda w: f"{w.name}-S{w.block_size}")
def test_partial_plans_small_whole_pool(w, opts):
    run_partial(w, opts)


def test_partial_plan_moves_fewer_rows_for_the_same_block_count():
    w = wl.mistral7b_random(seed=3, requests=12, lo=200, hi=600, layers=1, rho_lo=0.8, rho_hi=0.98)
    out_p, p = run_partial(w, dict(util=(1, 1)))
    out_w, q = run_partial(w, dict())
    both = (p.req_status == vto.REPACKED) & (q.req_status == vto.REPACKED)
    assert both.any()
    assert out_p["num_moves"] < out_w["num_moves"]
    for r in np.flatnonzero(both):
        assert (out_p["new_bt_offsets"][r + 1] - out_p["new_bt_offsets"][r]) == \
               (out_w["new_bt_offsets"][r + 1] - out_w["new_bt_offsets"][r])


def test_partial_free_list_cut():
    w = wl.mistral7b_random(seed=11, requests=6, lo=30, hi=90, layers=1, heads=1, head_dim=8, block_size=4)
    total = vto.plan_partial(w.block_size, w.num_blocks, w.bt_offsets, w.bt_blocks, w.tt_offsets, w.tt_slots, w.keep,
                             w.free_blocks, util=(1, 1)).num_free_consumed
    for c in range(total + 1):
        run_partial(w, dict(util=(1, 1)), num_free=c, whole_pool=(c % 5 == 0))


@pytest.mark.parametrize("w", small_configs(), ids=lambda w: f"{w.name}-S{w.block_size}")
def test_block_liveness_matches_oracle(w):
    import torch
    from harness.device import DeviceProblem
    prob = DeviceProblem(w, fill_seed=FILL_SEED)
    n_b = torch.full((w.num_blocks,), -1, dtype=torch.int32, device=prob.device)
    hist = torch.full((w.block_size + 1,), -1, dtype=torch.int64, device=prob.device)
    summary = torch.full((2,), -1, dtype=torch.int64, device=prob.device)
    vt.vtoken_block_liveness(prob.ctx, num_requests=prob.num_requests, bt_offsets=prob.bt_offsets,
                             bt_blocks=prob.bt_blocks, tt_offsets=prob.tt_offsets, tt_slots=prob.tt_slots,
                             keep=prob.keep, n_b=n_b, hist=hist, summary=summary)
    torch.cuda.synchronize()
    o_nb, o_hist, o_live, o_alloc = vto.block_liveness(w.block_size, w.num_blocks, w.bt_offsets, w.bt_blocks,
                                                       w.tt_offsets, w.tt_slots, w.keep)
    assert np.array_equal(n_b.cpu().numpy(), o_nb)
    assert np.array_equal(hist.cpu().numpy(), o_hist)
    assert summary.cpu().numpy().tolist() == [o_live, o_alloc]
    prob.close()


def test_partial_plan_full_size_steady_state_tables():
    """The partial planner at the benchmark's largest table size (512 requests, 2.2 M entries):
    all tables and lists against the oracle; pools verified through the origin map."""
    import torch
    from harness.device import DeviceProblem, origin_map
    free_bytes, _ = torch.cuda.mem_get_info()
    requests = 512
    while True:
        w = wl.steady_state(seed=0, requests=requests)
        if 2 * w.pool_bytes + (3 << 30) < free_bytes or requests == 1:
            break
        requests //= 2
    prob = DeviceProblem(w, fill_seed=FILL_SEED)
    prob.plan_partial(util=(1, 1), theta=(1, 4))
    prob.repack()
    out = prob.outputs()
    p = vto.plan_partial(w.block_size, w.num_blocks, w.bt_offsets, w.bt_blocks, w.tt_offsets, w.tt_slots, w.keep,
                         w.free_blocks, w.select, w.thr_num, w.thr_den, util=(1, 1), theta=(1, 4))
    assert out["error_flags"] == 0 and out["num_moves"] == p.num_moves > 10000
    assert np.array_equal(out["req_status"], p.req_status)
    assert np.array_equal(out["new_bt_offsets"], p.new_bt_offsets)
    assert np.array_equal(out["new_bt_blocks"], p.new_bt_blocks)
    assert np.array_equal(out["new_tt_slots"], p.new_tt_slots)
    assert np.array_equal(out["freed_blocks"], p.freed_blocks)
    assert prob.verify_pools(origin_map(w.slots_per_layer, p.move_src, p.move_dst)) == 0
    prob.close()
    del prob
    torch.cuda.empty_cache()


@pytest.mark.parametrize("degree", [1, 2, 4, 8])
def test_shared_prefix_workload(degree):
    """Synthetic prefix-cache workload: shared blocks protected, private suffixes repacked."""
    import torch
    from harness.device import DeviceProblem
    w, protect = wl.shared_prefix(seed=degree, groups=2, degree=degree, prefix_len=256, suffix_len=320, layers=2,
                                  heads=2, head_dim=64)
    prob = DeviceProblem(w, fill_seed=FILL_SEED)
    prob.plan_partial(protect=torch.from_numpy(protect).to(prob.device))
    prob.repack()
    out = prob.outputs()
    p = vto.plan_partial(w.block_size, w.num_blocks, w.bt_offsets, w.bt_blocks, w.tt_offsets, w.tt_slots, w.keep,
                         w.free_blocks, protect=protect)
    assert out["error_flags"] == 0 and out["num_admitted"] == p.num_admitted == w.num_requests
    assert np.array_equal(out["new_bt_offsets"], p.new_bt_offsets)
    assert np.array_equal(out["new_bt_blocks"], p.new_bt_blocks)
    assert np.array_equal(out["new_tt_slots"], p.new_tt_slots)
    assert np.array_equal(out["freed_blocks"], p.freed_blocks)
    assert not (set(out["freed_blocks"].tolist()) & set(np.flatnonzero(protect).tolist()))
    k, v = host_pools(w)
    vto.apply_moves_pools(k, v, p.move_src, p.move_dst)
    assert np.array_equal(prob.k_pool.cpu().numpy().view(np.uint16), k)
    assert np.array_equal(prob.v_pool.cpu().numpy().view(np.uint16), v)
    prob.close()


@pytest.mark.parametrize("opts", [dict(util=(1, 1)), dict(util=(1, 1), theta=(1, 4), max_source_blocks=9),
                                  dict(protect="prefix", util=(3, 4))], ids=["util", "bound", "protect"])
def test_repack_host_partial_entry_point(opts):
    """Host tables in, host tables out, partial planner; the protect mask is a host array."""
    import torch
    from harness.device import DeviceProblem
    w = wl.steady_state(seed=5, requests=14, lo=100, hi=900, layers=2, heads=2, head_dim=64)
    opts = dict(opts)
    if opts.get("protect") == "prefix":
        protect = np.zeros(w.num_blocks, np.uint8)
        for r in range(w.num_requests):
            protect[w.bt_blocks[w.bt_offsets[r]:w.bt_offsets[r + 1]][:2]] = 1
        opts["protect"] = protect
    prob = DeviceProblem(w, fill_seed=FILL_SEED)
    R, T, NBT = w.num_requests, w.num_tokens, len(w.bt_blocks)
    pin = lambda a: torch.from_numpy(np.ascontiguousarray(a)).pin_memory()
    h_in = dict(bt_offsets=pin(w.bt_offsets), bt_blocks=pin(w.bt_blocks), tt_offsets=pin(w.tt_offsets),
                tt_slots=pin(w.tt_slots), keep=pin(w.keep), free_blocks=pin(w.free_blocks))
    if w.select is not None:
        h_in["select"] = pin(w.select)
    h_out = dict(new_bt_offsets=torch.zeros(R + 1, dtype=torch.int32).pin_memory(),
                 new_bt_blocks=torch.zeros(NBT, dtype=torch.int32).pin_memory(),
                 new_tt_slots=torch.zeros(T, dtype=torch.int32).pin_memory(),
                 freed_blocks=torch.zeros(NBT, dtype=torch.int32).pin_memory(),
                 req_status=torch.zeros(R, dtype=torch.int32).pin_memory())
    s = torch.cuda.Stream()
    for _ in range(2):                                   # the second call reuses the staging buffers
        prob.fill_pools()
        torch.cuda.synchronize()
        c = vt.vtoken_repack_host_partial(prob.ctx, num_requests=R, num_free=len(w.free_blocks), thr_num=w.thr_num,
                                          thr_den=w.thr_den, stream=s, **opts, **h_in, **h_out)
    p = vto.plan_partial(w.block_size, w.num_blocks, w.bt_offsets, w.bt_blocks, w.tt_offsets, w.tt_slots, w.keep,
                         w.free_blocks, w.select, w.thr_num, w.thr_den, **opts)
    assert c["num_moves"] == p.num_moves > 0 and c["error_flags"] == 0 and c["num_freed"] == p.num_freed
    assert np.array_equal(h_out["new_tt_slots"].numpy(), p.new_tt_slots)
    assert np.array_equal(h_out["new_bt_offsets"].numpy(), p.new_bt_offsets)
    assert np.array_equal(h_out["new_bt_blocks"].numpy()[:len(p.new_bt_blocks)], p.new_bt_blocks)
    assert np.array_equal(h_out["freed_blocks"].numpy()[:p.num_freed], p.freed_blocks)
    assert np.array_equal(h_out["req_status"].numpy(), p.req_status)
    k, v = host_pools(w)
    vto.apply_moves_pools(k, v, p.move_src, p.move_dst)
    assert np.array_equal(prob.k_pool.cpu().numpy().view(np.uint16), k)
    assert np.array_equal(prob.v_pool.cpu().numpy().view(np.uint16), v)
    with pytest.raises(vt.VtokenError):
        vt._check(vt.load().vtoken_repack_host_partial(prob.ctx, None, None, None), "null arguments")
    prob.close()


@pytest.mark.parametrize("detach", [(1, 1), (1, 2), (1, 4), (1, 100)], ids=lambda d: f"detach{d[0]}_{d[1]}")
@pytest.mark.parametrize("degree", [1, 2, 4, 8])
@pytest.mark.parametrize("rule", [0, 1, 2], ids=["per_request", "per_block_own", "per_block_all"])
def test_copy_on_write_detach_on_the_shared_prefix_workload(degree, detach, rule):
    """Requests leave their shared prefix when their own tokens fill too little of it -- all of it at
    once, block by block, or block by block judged by all holders' tokens: tables, the reclaimed and the
    released lists, counts and whole pools against the oracle; the shared blocks keep their bytes."""
    import torch
    from harness.device import DeviceProblem
    w, protect = wl.shared_prefix(seed=10 + degree, groups=2, degree=degree, prefix_len=256, suffix_len=320, layers=2,
                                  heads=2, head_dim=64)
    prob = DeviceProblem(w, fill_seed=FILL_SEED)
    prob.plan_partial(protect=torch.from_numpy(protect).to(prob.device), util=(1, 1), detach=detach,
                      detach_rule=rule)
    prob.repack()
    out = prob.outputs()
    p = vto.plan_partial(w.block_size, w.num_blocks, w.bt_offsets, w.bt_blocks, w.tt_offsets, w.tt_slots, w.keep,
                         w.free_blocks, protect=protect, util=(1, 1), detach=detach, detach_rule=rule)
    assert out["error_flags"] == 0
    for n in ("num_moves", "num_dst_blocks", "num_freed", "num_free_consumed", "num_admitted", "num_deferred"):
        assert out[n] == getattr(p, n), n
    assert out["num_released"] == len(p.released_blocks)
    assert np.array_equal(out["released_blocks"], p.released_blocks)
    assert np.array_equal(out["req_status"], p.req_status)
    assert np.array_equal(out["new_bt_offsets"], p.new_bt_offsets)
    assert np.array_equal(out["new_bt_blocks"], p.new_bt_blocks)
    assert np.array_equal(out["new_tt_slots"], p.new_tt_slots)
    assert np.array_equal(out["freed_blocks"], p.freed_blocks)
    if detach == (1, 1) and rule == 0:
        assert out["num_released"] == degree * 2 * w.notes["prefix_blocks"]       # every sharer left every prefix block
    if detach == (1, 100) and rule == 0:
        assert out["num_released"] == 0                                           # nobody is that sparse
    if rule == 2 and p.num_admitted == w.num_requests:
        # judged by all holders' tokens: a shared block stays in every sharer's table or in none
        shared = np.flatnonzero(protect)
        held = np.bincount(p.new_bt_blocks[np.isin(p.new_bt_blocks, shared)], minlength=w.num_blocks)[shared]
        assert set(held.tolist()) <= {0, degree}
    if rule == 1 and detach == (1, 4):
        # the block rule really splits prefixes here: some request keeps part of its shared blocks
        kept_shared = np.isin(p.new_bt_blocks, np.flatnonzero(protect)).sum()
        assert 0 < out["num_released"] and kept_shared > 0
    k, v = host_pools(w)
    k0 = k.copy()
    vto.apply_moves_pools(k, v, p.move_src, p.move_dst)
    shared_rows = np.isin(np.arange(w.slots_per_layer) // w.block_size, np.flatnonzero(protect))
    assert np.array_equal(k[:, shared_rows], k0[:, shared_rows])
    assert np.array_equal(prob.k_pool.cpu().numpy().view(np.uint16), k)
    assert np.array_equal(prob.v_pool.cpu().numpy().view(np.uint16), v)
    prob.close()


def test_detach_needs_a_released_list_everywhere():
    import torch
    from harness.device import DeviceProblem
    w, protect = wl.shared_prefix(seed=3, groups=1, degree=2, prefix_len=64, suffix_len=80, layers=1, heads=1,
                                  head_dim=8)
    prob = DeviceProblem(w, fill_seed=FILL_SEED, wave_capacity=True)
    prot = torch.from_numpy(protect).to(prob.device)
    saved = prob.released_blocks
    prob.released_blocks = None
    with pytest.raises(vt.VtokenError) as e:
        prob.plan_partial(protect=prot, detach=(1, 1))
    assert e.value.code == vt.EINVAL
    prob.released_blocks = saved
    # the wave entry point and the host front end want a list of their own
    prob.repack_waves(2, partial=dict(protect=prot, util=(1, 1)))          # allocates the wave buffers
    wv = prob._waves
    args = dict(num_requests=prob.num_requests, bt_offsets=prob.bt_offsets, bt_blocks=prob.bt_blocks,
                tt_offsets=prob.tt_offsets, tt_slots=prob.tt_slots, keep=prob.keep, free_blocks=prob.free_blocks,
                num_free=prob.num_free, num_waves=2, new_bt_offsets=prob.new_bt_offsets,
                new_bt_blocks=prob.new_bt_blocks, new_tt_slots=prob.new_tt_slots, req_status=prob.req_status,
                req_wave=wv["req_wave"], free_out=wv["free_out"], num_free_out=wv["num_free_out"],
                wave_counts=wv["counts"], free_capacity=prob.max_free, workspace=wv["workspace"],
                workspace_bytes=wv["nbytes"])
    with pytest.raises(vt.VtokenError) as e:
        vt.vtoken_repack_waves(prob.ctx, partial=dict(protect=prot, detach=(1, 1)), **args)
    assert e.value.code == vt.EINVAL
    prob.close()


@pytest.mark.parametrize("degree", [2, 4])
@pytest.mark.parametrize("detach", [(1, 1), (1, 2)], ids=lambda d: f"detach{d[0]}_{d[1]}")
@pytest.mark.parametrize("rule", [0, 1, 2], ids=["per_request", "per_block_own", "per_block_all"])
def test_detach_through_the_wave_entry_point_and_the_host_front_end(degree, detach, rule):
    """Copy-on-write detach through vtoken_repack_waves (references dropped wave after wave, in one list)
    and through vtoken_repack_host_partial (host tables in and out): tables, lists and every byte of both
    pools against the oracle."""
    import torch
    from harness.device import DeviceProblem, origin_map
    w, protect = wl.shared_prefix(seed=7, groups=2, degree=degree, prefix_len=256, suffix_len=600, layers=2, heads=1,
                                  head_dim=64)
    opts = dict(util=(1, 1), max_source_blocks=12, detach=detach, detach_rule=rule)
    # ---- waves with a short pool: the detaches are spread over several waves
    need = vto.plan_partial(w.block_size, w.num_blocks, w.bt_offsets, w.bt_blocks, w.tt_offsets, w.tt_slots, w.keep,
                            w.free_blocks, protect=protect, **opts).num_dst_blocks
    nf = max(2, need // 3)
    W = 4
    v = vto.plan_waves(w.block_size, w.num_blocks, w.bt_offsets, w.bt_blocks, w.tt_offsets, w.tt_slots, w.keep,
                       w.free_blocks[:nf], W, partial=dict(protect=protect, **opts))
    prob = DeviceProblem(w, fill_seed=FILL_SEED, wave_capacity=True)
    prot = torch.from_numpy(protect).to(prob.device)
    nf_dev = torch.tensor([nf], dtype=torch.int32, device=prob.device)
    prob.repack_waves(W, num_free=nf_dev, partial=dict(protect=prot, **opts))
    out = prob.waves_outputs(W)
    assert all(c["error_flags"] == 0 for c in out["wave_counts"])
    assert [c["num_moves"] for c in out["wave_counts"]] == [c["num_moves"] for c in v.wave_counts]
    assert np.array_equal(out["new_tt_slots"], v.new_tt_slots) and np.array_equal(out["new_bt_blocks"], v.new_bt_blocks)
    assert np.array_equal(out["new_bt_offsets"], v.new_bt_offsets) and np.array_equal(out["req_status"], v.req_status)
    assert np.array_equal(out["free_out"], v.free_out) and np.array_equal(out["req_wave"], v.req_wave)
    assert np.array_equal(out["released_blocks"], v.released_blocks)
    if detach == (1, 1):
        assert len(v.released_blocks) > 0 and sum(1 for c in v.wave_counts if c["num_released"]) >= 1
    assert prob.verify_pools(origin_map(w.slots_per_layer, v.move_src, v.move_dst, v.wave_move_offsets)) == 0
    assert (prob._waves["released"][len(v.released_blocks):].cpu().numpy() == -9).all()
    prob.close()

    # ---- the host front end
    p = vto.plan_partial(w.block_size, w.num_blocks, w.bt_offsets, w.bt_blocks, w.tt_offsets, w.tt_slots, w.keep,
                         w.free_blocks, protect=protect, **opts)
    prob = DeviceProblem(w, fill_seed=FILL_SEED)
    R, T, NBT = w.num_requests, w.num_tokens, len(w.bt_blocks)
    pin = lambda a: torch.from_numpy(np.ascontiguousarray(a)).pin_memory()
    h_in = dict(bt_offsets=pin(w.bt_offsets), bt_blocks=pin(w.bt_blocks), tt_offsets=pin(w.tt_offsets),
                tt_slots=pin(w.tt_slots), keep=pin(w.keep), free_blocks=pin(w.free_blocks))
    h_out = dict(new_bt_offsets=torch.zeros(R + 1, dtype=torch.int32).pin_memory(),
                 new_bt_blocks=torch.zeros(NBT, dtype=torch.int32).pin_memory(),
                 new_tt_slots=torch.zeros(T, dtype=torch.int32).pin_memory(),
                 freed_blocks=torch.zeros(NBT, dtype=torch.int32).pin_memory(),
                 req_status=torch.zeros(R, dtype=torch.int32).pin_memory(),
                 released_blocks=torch.full((NBT,), -9, dtype=torch.int32).pin_memory())
    with pytest.raises(vt.VtokenError) as e:                 # no released list: refused before anything is enqueued
        vt.vtoken_repack_host_partial(prob.ctx, num_requests=R, num_free=len(w.free_blocks), protect=protect, **opts,
                                      **h_in, **{k: x for k, x in h_out.items() if k != "released_blocks"})
    assert e.value.code == vt.EINVAL
    c = vt.vtoken_repack_host_partial(prob.ctx, num_requests=R, num_free=len(w.free_blocks), protect=protect, **opts,
                                      **h_in, **h_out)
    assert c["error_flags"] == 0 and c["num_moves"] == p.num_moves and c["num_released"] == len(p.released_blocks)
    assert np.array_equal(h_out["new_tt_slots"].numpy(), p.new_tt_slots)
    assert np.array_equal(h_out["new_bt_blocks"].numpy()[:len(p.new_bt_blocks)], p.new_bt_blocks)
    assert np.array_equal(h_out["freed_blocks"].numpy()[:p.num_freed], p.freed_blocks)
    assert np.array_equal(h_out["released_blocks"].numpy()[:c["num_released"]], p.released_blocks)
    assert prob.verify_pools(origin_map(w.slots_per_layer, p.move_src, p.move_dst)) == 0
    prob.close()


@pytest.mark.parametrize("seed", range(16 * max(1, int(os.environ.get("VTOKEN_FUZZ_SCALE", "1")))))
def test_fuzz_detach_on_random_shared_prefix_shapes(seed):
    """Random prefix-cache shapes (block size, sharing degree, prefix and suffix lengths, kept
    fraction), thresholds, source bounds and pool cuts, the three detach rules, some requests
    deselected: tables, lists, counts and every byte of both pools against the oracle."""
    import torch
    from harness.device import DeviceProblem, origin_map
    rng = np.random.default_rng(7000 + seed)
    S = int(rng.choice([1, 2, 4, 16, 32]))
    w, protect = wl.shared_prefix(seed=seed, groups=int(rng.integers(1, 4)), degree=int(rng.integers(1, 6)),
                                  prefix_len=S * max(1, 8 // S) * int(rng.integers(1, 40)),
                                  suffix_len=int(rng.integers(1, 30 * max(S, 8) + 2)),
                                  layers=1, heads=1, head_dim=64, block_size=S,
                                  budget_frac=float(rng.choice([0.1, 0.2, 0.5, 0.9])))
    if rng.random() < 0.5:
        w.select = rng.integers(0, 2, size=w.num_requests).astype(np.uint8)
    opts = dict(util=[(0, 0), (1, 1), (1, 2)][int(rng.integers(0, 3))],
                max_source_blocks=int(rng.choice([0, 0, 2, 9])),
                detach=[(1, 1), (1, 2), (1, 4), (3, 4), (5, 4), (1, 16)][int(rng.integers(0, 6))],
                detach_rule=(1, 2, 1, 0, 2, 2)[seed % 6])
    num_free = None if rng.random() < 0.5 else int(rng.integers(0, len(w.free_blocks) + 1))
    p = vto.plan_partial(S, w.num_blocks, w.bt_offsets, w.bt_blocks, w.tt_offsets, w.tt_slots, w.keep, w.free_blocks,
                         w.select, w.thr_num, w.thr_den, num_free=num_free, protect=protect, **opts)
    prob = DeviceProblem(w, fill_seed=FILL_SEED)
    nf_dev = None if num_free is None else torch.tensor([num_free], dtype=torch.int32, device=prob.device)
    prob.plan_partial(num_free=nf_dev, protect=torch.from_numpy(protect).to(prob.device), **opts)
    prob.repack()
    out = prob.outputs()
    assert out["error_flags"] == 0
    for n in ("num_moves", "num_dst_blocks", "num_freed", "num_free_consumed", "num_admitted", "num_deferred"):
        assert out[n] == getattr(p, n), n
    assert out["num_released"] == len(p.released_blocks)
    for n in ("released_blocks", "req_status", "new_bt_offsets", "new_bt_blocks", "new_tt_slots", "freed_blocks"):
        assert np.array_equal(out[n], getattr(p, n)), n
    assert prob.verify_pools(origin_map(w.slots_per_layer, p.move_src, p.move_dst)) == 0
    prob.close()


@pytest.mark.parametrize("degree", [1, 2, 4])
def test_caller_side_of_copy_on_write_with_reference_counts(degree):
    """The whole protocol around a copy-on-write plan, as a caller with reference counts runs it: plan with
    the all-holders rule at 1/1, repack, adopt the new tables, drop one reference per entry of the released
    list, hand the blocks whose count reached zero back to the free list together with the reclaimed ones.
    Then the library's own precondition checker must accept the new state (no block free and held, unique
    mapping outside the blocks still shared), the relocation digest of every request must be what it was,
    and the pool must have gained exactly the blocks the tables lost."""
    import torch
    from harness.device import DeviceProblem
    from test_gpu_fuzz import _digest
    w, protect = wl.shared_prefix(seed=40 + degree, groups=3, degree=degree, prefix_len=256, suffix_len=300, layers=2,
                                  heads=2, head_dim=64)
    S, R = w.block_size, w.num_requests
    # room for every private copy: the generator sizes the pool for the conservative plan
    extra = 600
    w.num_blocks += extra
    w.free_blocks = np.concatenate([w.free_blocks, np.arange(w.num_blocks - extra, w.num_blocks, dtype=np.int32)])
    protect = np.concatenate([protect, np.zeros(extra, np.uint8)])
    refcount = np.bincount(w.bt_blocks, minlength=w.num_blocks)              # holders per block, as the caller tracks them
    assert set(refcount[protect != 0].tolist()) == {degree}
    prob = DeviceProblem(w, fill_seed=FILL_SEED)
    prot = torch.from_numpy(protect).to(prob.device)
    before = _digest(prob, vt, prob.tt_slots, prob.keep)
    prob.plan_partial(protect=prot, util=(1, 1), detach=(1, 1), detach_rule=2)
    prob.repack()
    out = prob.outputs()
    p = vto.plan_partial(S, w.num_blocks, w.bt_offsets, w.bt_blocks, w.tt_offsets, w.tt_slots, w.keep, w.free_blocks,
                         protect=protect, util=(1, 1), detach=(1, 1), detach_rule=2)
    assert out["error_flags"] == 0 and out["num_admitted"] == R == p.num_admitted
    assert np.array_equal(out["released_blocks"], p.released_blocks) and out["num_released"] > 0
    # ---- the caller's bookkeeping
    refcount -= np.bincount(out["released_blocks"], minlength=w.num_blocks)
    assert (refcount >= 0).all()
    unshared = np.flatnonzero((protect != 0) & (refcount == 0))              # every holder left: free again
    still_shared = (protect != 0) & (refcount > 0)
    if degree > 1:
        assert set(refcount[still_shared].tolist()) <= {degree}              # left by all holders or by none
    new_free = np.concatenate([w.free_blocks[out["num_free_consumed"]:], out["freed_blocks"], unshared]).astype(np.int32)
    new_bt, new_off = out["new_bt_blocks"], out["new_bt_offsets"]
    blocks_before, blocks_after = len(set(w.bt_blocks.tolist())), len(set(new_bt.tolist()))
    assert len(new_free) - len(w.free_blocks) == blocks_before - blocks_after > 0
    # ---- the new state through the library's checker and the relocation digest
    i32 = dict(dtype=torch.int32, device=prob.device)
    d_bt = torch.zeros(prob.max_table_blocks, **i32)
    d_bt[:len(new_bt)] = torch.from_numpy(new_bt)
    free_cap = torch.zeros(max(len(new_free), 1), **i32)
    free_cap[:len(new_free)] = torch.from_numpy(new_free)
    ctx2 = vt.vtoken_create(w.num_layers, w.num_blocks, S, w.num_kv_heads, w.head_dim, prob.k_pool, prob.v_pool,
                            prob.max_requests, prob.max_tokens, prob.max_table_blocks, max(len(new_free), 1))
    bits = torch.full((1,), -1, **i32)
    vt.vtoken_check_tables(ctx2, num_requests=prob.num_requests, bt_offsets=torch.from_numpy(new_off).to(prob.device),
                           bt_blocks=d_bt, tt_offsets=prob.tt_offsets, tt_slots=prob.new_tt_slots, free_blocks=free_cap,
                           num_free=torch.tensor([len(new_free)], **i32), out_bits=bits,
                           protect=torch.from_numpy(still_shared.astype(np.uint8)).to(prob.device))
    torch.cuda.synchronize()
    assert int(bits.item()) == 0
    vt.vtoken_destroy(ctx2)
    assert np.array_equal(before, _digest(prob, vt, prob.new_tt_slots, None))
    prob.close()
