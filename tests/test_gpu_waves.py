"""GPU parity of the repack in waves (blocks reclaimed by one wave are the destinations of the
next) against the oracle: final tables, statuses, wave indices, the pool, per-wave counts and
whole K/V pools, bit-exact; small headroom, both buffer parities, partial plans, graph replay."""
import numpy as np
import pytest

from oracle import vto
from paper_2608_13263_b200 import binding as vt
from harness import workloads as wl

pytestmark = pytest.mark.gpu

FILL_SEED = 1
COUNT_NAMES = ("num_moves", "num_dst_blocks", "num_freed", "num_free_consumed", "num_admitted", "num_deferred")


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
        wl.mistral7b_random(seed=0, requests=17, lo=100, hi=500, layers=2),
        wl.longctx_scissor(seed=0, requests=3, lo=3000, hi=6000, layers=1),
        wl.steady_state(seed=0, requests=24, lo=100, hi=1500, layers=2),
        wl.steady_state(seed=1, requests=24, lo=100, hi=1500, layers=1, block_size=32),
        wl.streaming_window(seed=0, requests=9, lo=200, hi=1500, window=100, layers=1),
    ]


def oracle_waves(w, nf, num_waves, partial=None):
    return vto.plan_waves(w.block_size, w.num_blocks, w.bt_offsets, w.bt_blocks, w.tt_offsets, w.tt_slots, w.keep,
                          w.free_blocks[:nf], num_waves, w.select, w.thr_num, w.thr_den, partial)


def compare(out, v, num_waves):
    for k in range(num_waves):
        assert out["wave_counts"][k]["error_flags"] == 0
        for n in COUNT_NAMES:
            assert out["wave_counts"][k][n] == v.wave_counts[k][n], (k, n)
    assert np.array_equal(out["req_status"], v.req_status)
    assert np.array_equal(out["req_wave"], v.req_wave)
    assert np.array_equal(out["req_append_pos"], v.req_append_pos)
    assert np.array_equal(out["new_bt_offsets"], v.new_bt_offsets)
    assert np.array_equal(out["new_bt_blocks"], v.new_bt_blocks)
    assert np.array_equal(out["new_tt_slots"], v.new_tt_slots)
    assert np.array_equal(out["free_out"], v.free_out)


def run_waves(w, nf, num_waves, partial=None, whole_pool=True):
    import torch
    from harness.device import DeviceProblem
    prob = DeviceProblem(w, fill_seed=FILL_SEED, wave_capacity=True)
    dpart = None
    if partial is not None:
        dpart = dict(partial)
        if dpart.get("protect") is not None:
            dpart["protect"] = torch.from_numpy(dpart["protect"]).to(prob.device)
    nf_dev = torch.tensor([nf], dtype=torch.int32, device=prob.device)
    prob.repack_waves(num_waves, num_free=nf_dev, partial=dpart)
    out = prob.waves_outputs(num_waves)
    v = oracle_waves(w, nf, num_waves, partial)
    compare(out, v, num_waves)
    if whole_pool:
        k, vv = host_pools(w)
        vto.apply_moves_pools(k, vv, v.move_src, v.move_dst, threads=2)      # list order = wave order
        assert np.array_equal(prob.k_pool.cpu().numpy().view(np.uint16), k)
        assert np.array_equal(prob.v_pool.cpu().numpy().view(np.uint16), vv)
    prob.close()
    return out, v


def largest_demand(w):
    p = vto.plan_workload(w)
    need = np.diff(p.new_bt_offsets)[p.req_status == vto.REPACKED]
    return int(need.max()) if len(need) else 0, p


@pytest.mark.parametrize("num_waves", [1, 2, 3, 6])
@pytest.mark.parametrize("w", small_configs(), ids=lambda w: f"{w.name}-S{w.block_size}")
def test_waves_with_the_headroom_of_one_request(w, num_waves):
    biggest, _ = largest_demand(w)
    out, v = run_waves(w, biggest, num_waves)
    if num_waves >= 3:
        assert sum(1 for c in v.wave_counts if c["num_admitted"]) >= 2       # blocks really were reused


@pytest.mark.parametrize("frac", [0.0, 0.5, 1.0])
@pytest.mark.parametrize("w", small_configs()[:5], ids=lambda w: f"{w.name}-S{w.block_size}")
def test_waves_pool_sizes(w, frac):
    _, p = largest_demand(w)
    run_waves(w, int(frac * p.num_dst_blocks), 4, whole_pool=(frac != 0.0))


PARTIALS = [dict(util=(1, 1)), dict(util=(1, 1), max_source_blocks=6), dict(util=(3, 4), theta=(1, 4)),
            dict(protect="prefix", util=(1, 1), max_source_blocks=9)]


@pytest.mark.parametrize("opts", PARTIALS, ids=[str(i) for i in range(len(PARTIALS))])
@pytest.mark.parametrize("w", small_configs()[:5], ids=lambda w: f"{w.name}-S{w.block_size}")
def test_partial_waves(w, opts):
    opts = dict(opts)
    if opts.get("protect") == "prefix":
        protect = np.zeros(w.num_blocks, np.uint8)
        for r in range(w.num_requests):
            protect[w.bt_blocks[w.bt_offsets[r]:w.bt_offsets[r + 1]][:3]] = 1
        opts["protect"] = protect
    biggest, _ = largest_demand(w)
    run_waves(w, max(2, biggest // 2), 5, partial=opts)


def test_waves_graph_replay_after_the_pools_are_refilled():
    """The whole chain is one captured graph on a side stream; replaying it after restoring the
    pools reproduces the result (every count and pool lives on the device)."""
    import torch
    from harness.device import DeviceProblem
    w = wl.mistral7b_random(seed=4, requests=20, lo=100, hi=400, layers=2)
    biggest, _ = largest_demand(w)
    W = 5
    prob = DeviceProblem(w, fill_seed=FILL_SEED, wave_capacity=True)
    nf_dev = torch.tensor([biggest], dtype=torch.int32, device=prob.device)
    prob.repack_waves(W, num_free=nf_dev)                  # allocates the wave buffers outside the capture
    torch.cuda.synchronize()
    side = torch.cuda.Stream()
    g = torch.cuda.CUDAGraph()
    with torch.cuda.stream(side):
        g.capture_begin()
        prob.repack_waves(W, num_free=nf_dev, stream=side)
        g.capture_end()
    v = oracle_waves(w, biggest, W)
    k, vv = host_pools(w)
    vto.apply_moves_pools(k, vv, v.move_src, v.move_dst, threads=2)
    for _ in range(2):
        prob.fill_pools()
        prob.new_tt_slots.fill_(-9)
        torch.cuda.synchronize()
        g.replay()
        compare(prob.waves_outputs(W), v, W)
        assert np.array_equal(prob.k_pool.cpu().numpy().view(np.uint16), k)
        assert np.array_equal(prob.v_pool.cpu().numpy().view(np.uint16), vv)
    prob.close()


def test_waves_argument_errors():
    import torch
    from harness.device import DeviceProblem
    w = wl.tiny(seed=0)
    prob = DeviceProblem(w, fill_seed=FILL_SEED)           # max_free_blocks = len(free list): no room to grow
    i32 = dict(dtype=torch.int32, device=prob.device)
    nbytes = vt.vtoken_waves_workspace_bytes(prob.ctx, prob.max_free)
    assert nbytes > 0 and nbytes % 16 == 0
    ws = torch.empty(nbytes, dtype=torch.uint8, device=prob.device)
    args = dict(num_requests=prob.num_requests, bt_offsets=prob.bt_offsets, bt_blocks=prob.bt_blocks,
                tt_offsets=prob.tt_offsets, tt_slots=prob.tt_slots, keep=prob.keep, free_blocks=prob.free_blocks,
                num_free=prob.num_free, num_waves=2, new_bt_offsets=prob.new_bt_offsets,
                new_bt_blocks=prob.new_bt_blocks, new_tt_slots=prob.new_tt_slots, req_status=prob.req_status,
                req_wave=torch.zeros(prob.max_requests, **i32), free_out=torch.zeros(prob.max_free + 64, **i32),
                num_free_out=torch.zeros(1, **i32), wave_counts=torch.zeros((2, 8), **i32),
                free_capacity=prob.max_free, workspace=ws, workspace_bytes=nbytes)
    for bad, code in ((dict(num_waves=0), vt.EINVAL), (dict(free_capacity=prob.max_free + 1), vt.ECAPACITY),
                      (dict(workspace_bytes=nbytes - 16), vt.ECAPACITY), (dict(workspace=None), vt.EINVAL),
                      (dict(workspace=ws.data_ptr() + 4), vt.EINVAL), (dict(req_wave=None), vt.EINVAL)):
        with pytest.raises(vt.VtokenError) as e:
            vt.vtoken_repack_waves(prob.ctx, **{**args, **bad})
        assert e.value.code == code, bad
    # a pool that outgrows free_capacity is truncated and flagged, nothing is written behind it
    vt.vtoken_repack_waves(prob.ctx, **args)
    torch.cuda.synchronize()
    counts = args["wave_counts"].cpu().numpy()
    assert int(np.uint32(counts[0][6])) & vt.FLAG_CAPACITY
    assert int(args["num_free_out"].item()) == prob.max_free
    assert not args["free_out"][prob.max_free:].any()
    prob.close()


def test_waves_full_size_llama_shape_with_a_twentieth_of_the_headroom():
    """Llama-3-8B-shaped H2O workload at full size: the one-shot plan needs ~2300 destination
    blocks; a pool of the largest single demand finishes the same repack in waves.  Tables against
    the oracle, both pools through the origin map."""
    import torch
    from harness.device import DeviceProblem, origin_map
    free_bytes, _ = torch.cuda.mem_get_info()
    requests = 64
    while True:
        w = wl.llama8b_h2o(seed=0, requests=requests)
        if 2 * w.pool_bytes + (3 << 30) < free_bytes or requests == 1:
            break
        requests //= 2
    biggest, p = largest_demand(w)
    assert biggest * 10 < p.num_dst_blocks
    W = 8
    prob = DeviceProblem(w, fill_seed=FILL_SEED, wave_capacity=True)
    prob.repack_waves(W, num_free=torch.tensor([biggest], dtype=torch.int32, device=prob.device))
    out = prob.waves_outputs(W)
    v = oracle_waves(w, biggest, W)
    compare(out, v, W)
    assert (v.req_status == vto.REPACKED).sum() == p.num_admitted and len(v.move_src) == p.num_moves
    assert prob.verify_pools(origin_map(w.slots_per_layer, v.move_src, v.move_dst, v.wave_move_offsets)) == 0
    prob.close()
    del prob
    torch.cuda.empty_cache()
