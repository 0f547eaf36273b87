"""GPU parity: the CUDA path (through the C ABI) against the CPU oracle, element by element,
on the same seeded inputs.  Integer, byte and index work: the bar is bit-exact.
"""
import numpy as np
import pytest

from oracle import vto
from paper_2608_13263_b200 import binding as vt
from harness import workloads as wl

pytestmark = pytest.mark.gpu

FILL_SEED = 1


def _torch():
    import torch
    return torch


def host_pools(w):
    k = np.stack([wl.fill_slab(FILL_SEED, 0, l, w.num_layers, w.slots_per_layer, w.row_elems)
                  for l in range(w.num_layers)])
    v = np.stack([wl.fill_slab(FILL_SEED, 1, l, w.num_layers, w.slots_per_layer, w.row_elems)
                  for l in range(w.num_layers)])
    return k, v


def assert_tables_equal(out, p, w):
    assert out["error_flags"] == 0
    for name in ("num_moves", "num_dst_blocks", "num_freed", "num_free_consumed", "num_admitted", "num_deferred"):
        assert out[name] == getattr(p, name), name
    assert np.array_equal(out["req_status"], p.req_status)
    assert np.array_equal(out["new_bt_offsets"], p.new_bt_offsets)
    assert np.array_equal(out["new_bt_blocks"], p.new_bt_blocks)
    assert np.array_equal(out["new_tt_slots"], p.new_tt_slots)
    assert np.array_equal(out["freed_blocks"], p.freed_blocks)


def run_and_compare(w, copy_variant=0, num_free=None, whole_pool=True, capacity_slack=0, **ctx_options):
    """plan + repack on the GPU, oracle on the host, compare everything."""
    from harness.device import DeviceProblem
    torch = _torch()
    prob = DeviceProblem(w, fill_seed=FILL_SEED, copy_variant=copy_variant, capacity_slack=capacity_slack,
                         **ctx_options)
    nf_dev = None
    if num_free is not None:
        nf_dev = torch.tensor([num_free], dtype=torch.int32, device=prob.device)
    prob.plan(num_free=nf_dev)
    prob.repack()
    out = prob.outputs()
    p = vto.plan_workload(w, num_free=num_free)
    assert_tables_equal(out, p, w)
    counts = prob.read_counts()
    assert counts["error_flags"] == 0 and counts["num_moves"] == p.num_moves
    # nothing was written beyond the valid part of any output buffer (they were pre-filled with -9)
    R, T = w.num_requests, w.num_tokens
    for buf, valid in ((prob.new_bt_offsets, R + 1), (prob.new_bt_blocks, len(p.new_bt_blocks)),
                       (prob.new_tt_slots, T), (prob.freed_blocks, p.num_freed), (prob.req_status, R)):
        tail = buf[valid:].cpu().numpy()
        assert (tail == -9).all(), "stray write behind an output table"
    if whole_pool:
        k, v = host_pools(w)
        # the device fill and the numpy fill are the same generator
        vto.apply_moves_pools(k, v, p.move_src, p.move_dst, threads=2)
        gk = prob.k_pool.cpu().numpy().view(np.uint16)
        gv = prob.v_pool.cpu().numpy().view(np.uint16)
        assert np.array_equal(gk, k), "K pool differs from the oracle"
        assert np.array_equal(gv, v), "V pool differs from the oracle"
    prob.close()
    return out, p


def small_configs():
    """The five workload recipes at sizes the oracle finishes in seconds, each spanning many
    copy items and a ragged tail."""
    return [
        wl.tiny(seed=0),
        wl.llama8b_h2o(seed=0, requests=6, lo=300, hi=900, layers=3),
        wl.mistral7b_random(seed=0, requests=17, lo=100, hi=500, layers=2),
        wl.longctx_scissor(seed=0, requests=3, lo=3000, hi=6000, layers=2),
        wl.steady_state(seed=0, requests=24, lo=100, hi=1500, layers=2),
        wl.steady_state(seed=1, requests=24, lo=100, hi=1500, layers=2, block_size=32),
        wl.streaming_window(seed=0, requests=9, lo=200, hi=1500, window=100, layers=2),
    ]


@pytest.mark.parametrize("variant", [1, 2])
@pytest.mark.parametrize("w", small_configs(), ids=lambda w: f"{w.name}-S{w.block_size}")
def test_configs_small_whole_pool(w, variant):
    if variant == 2 and w.row_bytes < 16:
        pytest.skip("row too small")
    run_and_compare(w, copy_variant=variant)


@pytest.mark.parametrize("variant", [1, 2])
@pytest.mark.parametrize("S,heads,head_dim", [(1, 1, 8), (2, 1, 8), (3, 2, 64), (16, 4, 128), (32, 8, 128),
                                               (48, 8, 128), (16, 16, 128), (5, 3, 8), (16, 64, 256), (4, 128, 256)])
def test_block_sizes_and_row_bytes(S, heads, head_dim, variant):
    """S in {1,2,3,4,5,16,32,48}; row_bytes in {16, 48, 256, 1024, 2048, 4096, 32768, 65536} (the last
    is beyond what one bulk-copy stage holds: the library must fall back to the register path)."""
    if heads * head_dim * 2 > 32768 and variant == 2:
        variant = 0
    big = heads * head_dim * 2 >= 32768
    w = wl.mistral7b_random(seed=S, requests=3 if big else 5, lo=10, hi=(6 if big else 40) * S + 20,
                            layers=1 if big else 2, heads=heads, head_dim=head_dim, block_size=S)
    run_and_compare(w, copy_variant=variant)


@pytest.mark.parametrize("tune", ["1,2,1,0,1", "1,12,1,10,2", "8,6,2,2,2", "4,3,8,1,1", "2,3,16,1,2", "8,12,1,4,1",
                                  "3,5,4,3,2", "8,2,32,0,2"])
def test_bulk_copy_ring_shapes(tune):
    """Every ring shape the tuning fields can select (warps, stages, rows per item, loads ahead,
    plan entries ahead) must give the same bytes: whole pools against the oracle."""
    tuning = dict(zip(("warps", "stages", "rows", "depth", "ahead"), (int(x) for x in tune.split(","))))
    for w in (wl.mistral7b_random(seed=5, requests=7, lo=60, hi=700, layers=2),
              wl.longctx_scissor(seed=5, requests=2, lo=1500, hi=2500, layers=2, block_size=32),
              wl.mistral7b_random(seed=6, requests=4, lo=30, hi=300, layers=1, heads=4, head_dim=128, block_size=48)):
        run_and_compare(w, copy_variant=2, tuning=tuning)
    run_and_compare(wl.mistral7b_random(seed=5, requests=7, lo=60, hi=700, layers=2), copy_variant=2, max_ctas=37)


@pytest.mark.parametrize("dynamic,chunk", [("0", "4"), ("1", "1"), ("1", "3"), ("1", "64"), ("1", "1000")])
def test_copy_work_distribution_modes(dynamic, chunk):
    """Fixed shares per warp and ticket distribution with several chunk sizes (one item per ticket,
    an odd count, more items per ticket than a small launch has): the same bytes, whole pools
    against the oracle, also when the context is reused for a second plan (the ticket counter must
    be back at zero)."""
    tuning = dict(fixed_shares=int(dynamic == "0"), chunk=int(chunk))
    for w in (wl.mistral7b_random(seed=5, requests=7, lo=60, hi=700, layers=2),
              wl.longctx_scissor(seed=5, requests=2, lo=1500, hi=2500, layers=2, block_size=32),
              wl.tiny(seed=1)):
        run_and_compare(w, copy_variant=2, tuning=tuning)
    from harness.device import DeviceProblem
    w = wl.llama8b_h2o(seed=2, requests=5, lo=200, hi=900, layers=2)
    prob = DeviceProblem(w, fill_seed=FILL_SEED, copy_variant=2, tuning=tuning)
    p = vto.plan_workload(w)
    k, v = host_pools(w)
    vto.apply_moves_pools(k, v, p.move_src, p.move_dst)
    for _ in range(3):                                   # three launches on one context
        prob.fill_pools()
        prob.plan()
        prob.repack()
        assert prob.outputs()["error_flags"] == 0
        assert np.array_equal(prob.k_pool.cpu().numpy().view(np.uint16), k)
        assert np.array_equal(prob.v_pool.cpu().numpy().view(np.uint16), v)
    prob.close()


@pytest.mark.parametrize("pdl", ["0", "1"])
def test_launch_modes_give_the_same_result(pdl):
    """Plain stream-ordered launches and programmatic dependent launches (a kernel may become resident
    while its predecessor finishes and waits for it on the device): the same tables and bytes, for both
    copy paths, with launches issued back to back on one stream without host synchronisation between
    plan, copy and the next plan."""
    plain = int(pdl == "0")
    from harness.device import DeviceProblem
    torch = _torch()
    for variant in (1, 2):
        run_and_compare(wl.mistral7b_random(seed=9, requests=6, lo=80, hi=600, layers=2), copy_variant=variant,
                        plain_launches=plain)
        w = wl.llama8b_h2o(seed=4, requests=6, lo=200, hi=900, layers=2)
        prob = DeviceProblem(w, fill_seed=FILL_SEED, copy_variant=variant, plain_launches=plain)
        p = vto.plan_workload(w)
        k, v = host_pools(w)
        vto.apply_moves_pools(k, v, p.move_src, p.move_dst)
        st = torch.cuda.Stream()
        with torch.cuda.stream(st):
            for _ in range(5):                           # nothing but stream order between these launches
                prob.fill_pools(stream=st)
                prob.plan(stream=st)
                prob.repack(stream=st)
        st.synchronize()
        assert_tables_equal(prob.outputs(), p, w)
        assert np.array_equal(prob.k_pool.cpu().numpy().view(np.uint16), k)
        assert np.array_equal(prob.v_pool.cpu().numpy().view(np.uint16), v)
        prob.close()


def _request(n_tokens, S, first_block):
    nb = -(-n_tokens // S)
    bt = np.arange(first_block, first_block + nb, dtype=np.int32)
    tt = (bt[np.arange(n_tokens) // S] * S + np.arange(n_tokens) % S).astype(np.int32)
    return bt, tt


def _custom(S, lens, keeps, free_extra=8, layers=1, heads=1, head_dim=8, select=None, thr=(0, 0), holes=None):
    bts, tts, nxt = [], [], 0
    for n in lens:
        bt, tt = _request(n, S, nxt)
        nxt += len(bt)
        bts.append(bt), tts.append(tt)
    bt_off = np.concatenate([[0], np.cumsum([len(b) for b in bts])]).astype(np.int32)
    tt_off = np.concatenate([[0], np.cumsum(lens)]).astype(np.int32)
    tt = np.concatenate(tts + [np.zeros(0, np.int32)]).astype(np.int32)
    if holes is not None:
        tt[holes] = -1
    need = sum(-(-int(np.sum(k)) // S) for k in keeps)
    NB = nxt + need + free_extra
    free = np.arange(nxt, NB, dtype=np.int32)[::-1].copy()
    return wl.Workload(name="custom", num_layers=layers, num_kv_heads=heads, head_dim=head_dim, block_size=S,
                       num_blocks=NB, bt_offsets=bt_off,
                       bt_blocks=np.concatenate(bts + [np.zeros(0, np.int32)]).astype(np.int32),
                       tt_offsets=tt_off, tt_slots=tt,
                       keep=np.concatenate(list(keeps) + [np.zeros(0, np.uint8)]).astype(np.uint8),
                       free_blocks=free, select=select, thr_num=thr[0], thr_den=thr[1])


def test_edge_all_keep_all_evict_empty_and_boundaries():
    S = 16
    rng = np.random.default_rng(0)
    lens = [100, 0, 64, 33, 1, 16 * 7, 16 * 7 + 1, 16 * 7 - 1, 500]
    keeps = [np.ones(100, np.uint8), np.zeros(0, np.uint8), np.zeros(64, np.uint8),
             (rng.random(33) < 0.5).astype(np.uint8), np.ones(1, np.uint8)]
    for n, k in ((16 * 7, 47), (16 * 7 + 1, 48), (16 * 7 - 1, 49)):      # live = k*S-1, k*S, k*S+1
        m = np.zeros(n, np.uint8)
        m[rng.permutation(n)[:k]] = 1
        keeps.append(m)
    m = np.zeros(500, np.uint8)
    m[::S] = 1                                                           # one survivor per block
    keeps.append(m)
    w = _custom(S, lens, keeps)
    out, p = run_and_compare(w)
    assert p.req_status.tolist()[:3] == [vto.NO_GAIN, vto.NO_GAIN, vto.REPACKED]
    # everything kept: outputs equal inputs, pools untouched
    w2 = _custom(S, [100, 37], [np.ones(100, np.uint8), np.ones(37, np.uint8)])
    out, p = run_and_compare(w2)
    assert out["num_moves"] == 0 and np.array_equal(out["new_tt_slots"], w2.tt_slots)


def test_edge_free_list_cut_at_every_length():
    w = wl.mistral7b_random(seed=11, requests=6, lo=30, hi=90, layers=1, heads=1, head_dim=8, block_size=4)
    total = vto.plan_workload(w).num_free_consumed
    seen_deferred = False
    for c in range(total + 1):
        out, p = run_and_compare(w, num_free=c, whole_pool=(c % 7 == 0))
        seen_deferred |= out["num_deferred"] > 0
    assert seen_deferred


def test_edge_select_threshold_and_holes():
    rng = np.random.default_rng(5)
    S = 4
    lens = [40, 25, 64, 9, 80]
    for trial in range(6):
        keeps = [(rng.random(n) < rng.uniform(0.1, 0.9)).astype(np.uint8) for n in lens]
        holes = rng.permutation(sum(lens))[:30]
        select = None if trial == 0 else rng.integers(0, 2, len(lens)).astype(np.uint8)
        thr = [(0, 0), (1, 4), (1, 2), (3, 4), (1, 1), (1, 2)][trial]
        w = _custom(S, lens, keeps, select=select, thr=thr, holes=holes, layers=2)
        run_and_compare(w)
    # live fraction exactly at the threshold is not selected
    bt_keep = np.zeros(16, np.uint8)
    bt_keep[:8] = 1
    w = _custom(4, [16], [bt_keep], thr=(1, 2))
    out, p = run_and_compare(w)
    assert out["req_status"].tolist() == [vt.NOT_SELECTED]


def test_long_and_one_token_requests_in_one_batch():
    rng = np.random.default_rng(9)
    lens = [1, 33000, 1, 2, 5000, 1]
    keeps = [(rng.random(n) < 0.4).astype(np.uint8) for n in lens]
    w = _custom(32, lens, keeps, layers=1, heads=1, head_dim=64)
    run_and_compare(w)


def test_capacities_larger_than_the_problem():
    w = wl.mistral7b_random(seed=3, requests=9, lo=50, hi=300, layers=2, heads=1, head_dim=64)
    run_and_compare(w, capacity_slack=1000)


def test_repeated_repack_and_idempotence():
    """Adopt the new tables, evict again, repack again; then all-keep -> nothing to gain."""
    from harness.device import DeviceProblem
    torch = _torch()
    w = wl.mistral7b_random(seed=21, requests=8, lo=100, hi=400, layers=2, heads=2, head_dim=64)
    out, p = run_and_compare(w)
    rng = np.random.default_rng(2)
    # state after the first repack (from the oracle; the GPU outputs were just shown to equal it)
    keep2 = ((p.new_tt_slots >= 0) & (rng.random(w.num_tokens) < 0.5)).astype(np.uint8)
    used = set(p.new_bt_blocks.tolist())
    free2 = np.array(sorted(set(range(w.num_blocks)) - used), np.int32)
    w2 = wl.Workload(name="second_repack", num_layers=w.num_layers, num_kv_heads=w.num_kv_heads, head_dim=w.head_dim,
                     block_size=w.block_size, num_blocks=w.num_blocks, bt_offsets=p.new_bt_offsets,
                     bt_blocks=p.new_bt_blocks, tt_offsets=w.tt_offsets, tt_slots=p.new_tt_slots, keep=keep2,
                     free_blocks=free2)
    out2, p2 = run_and_compare(w2)
    assert out2["num_admitted"] > 0
    keep3 = (p2.new_tt_slots >= 0).astype(np.uint8)
    used3 = set(p2.new_bt_blocks.tolist())
    w3 = wl.Workload(name="third_repack", num_layers=w.num_layers, num_kv_heads=w.num_kv_heads, head_dim=w.head_dim,
                     block_size=w.block_size, num_blocks=w.num_blocks, bt_offsets=p2.new_bt_offsets,
                     bt_blocks=p2.new_bt_blocks, tt_offsets=w.tt_offsets, tt_slots=p2.new_tt_slots, keep=keep3,
                     free_blocks=np.array(sorted(set(range(w.num_blocks)) - used3), np.int32))
    out3, p3 = run_and_compare(w3)
    assert out3["num_moves"] == 0 and set(out3["req_status"].tolist()) <= {vt.NO_GAIN}


@pytest.mark.parametrize("heads,head_dim", [(1, 8), (4, 64)], ids=["register-path", "bulk-path"])
def test_out_of_range_ids_raise_flags_not_faults(heads, head_dim):
    """Host-fabricated bad slot / block / free ids: a flag bit, the row skipped, no fault."""
    from harness.device import DeviceProblem
    rng = np.random.default_rng(4)
    lens = [60, 60]
    keeps = [(rng.random(60) < 0.3).astype(np.uint8) for _ in lens]
    w = _custom(4, lens, keeps, heads=heads, head_dim=head_dim)
    w.tt_slots[np.flatnonzero(w.keep)[0]] = w.num_blocks * w.block_size + 5      # slot beyond the pool
    w.free_blocks[1] = w.num_blocks + 3                                          # free id beyond the pool
    w.bt_blocks[len(w.bt_blocks) - 1] = -4                                       # bad block-table id
    prob = DeviceProblem(w, fill_seed=FILL_SEED)
    prob.plan()
    prob.repack()
    out = prob.outputs()
    flags = prob.read_counts()["error_flags"]
    assert flags & vt.FLAG_BAD_SLOT and flags & vt.FLAG_BAD_FREE and flags & vt.FLAG_BAD_BLOCK
    assert not flags & vt.FLAG_TIMEOUT
    # the bad token was treated as not live
    assert out["new_tt_slots"][np.flatnonzero(w.keep)[0]] == -1
    prob.close()


def test_counts_above_capacity_are_clamped_and_flagged():
    """A device-side request count or free count above the create-time capacities: clamped,
    VTOKEN_FLAG_CAPACITY raised, the part inside the capacities still exact."""
    from harness.device import DeviceProblem
    torch = _torch()
    w = wl.mistral7b_random(seed=13, requests=8, lo=50, hi=300, layers=1, heads=1, head_dim=64)
    prob = DeviceProblem(w, fill_seed=FILL_SEED)                 # capacities == problem sizes
    prob.num_requests.fill_(w.num_requests + 5)
    prob.num_free.fill_(len(w.free_blocks) + 1000)
    prob.plan()
    prob.repack()
    out = prob.outputs()
    assert out["error_flags"] & vt.FLAG_CAPACITY
    p = vto.plan_workload(w)
    assert np.array_equal(out["new_tt_slots"], p.new_tt_slots)
    assert np.array_equal(out["new_bt_blocks"], p.new_bt_blocks)
    assert np.array_equal(out["freed_blocks"], p.freed_blocks)
    prob.close()


@pytest.mark.parametrize("planner", ["whole", "partial"])
def test_tables_beyond_the_context_capacities_are_clipped(planner):
    """Token and block tables longer than the capacities the context was created with: entries at or
    beyond a capacity do not exist for the planner (the result is the oracle's on the clipped tables),
    VTOKEN_FLAG_CAPACITY is raised, and nothing is written behind a capacity in any output buffer."""
    from harness.device import DeviceProblem
    w = wl.mistral7b_random(seed=21, requests=9, lo=60, hi=400, layers=1, heads=1, head_dim=64)
    T, NBT = w.num_tokens, len(w.bt_blocks)
    cap_t, cap_b = T - 157, NBT - 5                      # cuts into the last request (and the one before it)
    assert cap_t < w.tt_offsets[-2] + 40 and cap_b > w.bt_offsets[-2] - 3
    prob = DeviceProblem(w, fill_seed=FILL_SEED, ctx_capacity=dict(max_tokens=cap_t, max_table_blocks=cap_b))
    if planner == "whole":
        prob.plan()
    else:
        prob.plan_partial()
    prob.repack()
    out = prob.outputs()
    assert out["error_flags"] == vt.FLAG_CAPACITY
    tt_off = np.minimum(w.tt_offsets, cap_t).astype(np.int32)
    bt_off = np.minimum(w.bt_offsets, cap_b).astype(np.int32)
    p = vto.plan(w.block_size, bt_off, w.bt_blocks[:cap_b], tt_off, w.tt_slots[:cap_t], w.keep[:cap_t], w.free_blocks)
    assert p.num_admitted > 0
    assert np.array_equal(out["req_status"], p.req_status)
    assert np.array_equal(out["new_bt_offsets"], p.new_bt_offsets)
    nbt = int(p.new_bt_offsets[-1])
    assert np.array_equal(prob.new_bt_blocks[:nbt].cpu().numpy(), p.new_bt_blocks)
    assert np.array_equal(prob.new_tt_slots[:cap_t].cpu().numpy(), p.new_tt_slots)
    assert np.array_equal(prob.freed_blocks[:p.num_freed].cpu().numpy(), p.freed_blocks)
    assert (prob.new_tt_slots[cap_t:].cpu().numpy() == -9).all()
    assert (prob.new_bt_blocks[nbt:].cpu().numpy() == -9).all()
    assert (prob.freed_blocks[p.num_freed:].cpu().numpy() == -9).all()
    k, v = host_pools(w)
    vto.apply_moves_pools(k, v, p.move_src, p.move_dst)
    assert np.array_equal(prob.k_pool.cpu().numpy().view(np.uint16), k)
    assert np.array_equal(prob.v_pool.cpu().numpy().view(np.uint16), v)
    prob.close()


def _misaligned_copy(t, offset_elems):
    """A copy of tensor ``t`` whose data pointer is ``offset_elems`` elements behind an aligned allocation."""
    torch = _torch()
    buf = torch.empty(t.numel() + offset_elems, dtype=t.dtype, device=t.device)
    view = buf[offset_elems:]
    view.copy_(t)
    return view


@pytest.mark.parametrize("planner", ["whole", "partial"])
def test_tables_that_are_not_16_byte_aligned(planner):
    """The planners read four table entries per thread with 16-byte and 4-byte accesses when the caller's
    arrays allow it; arrays that start at an odd element take the scalar path and give the same result."""
    from harness.device import DeviceProblem
    w = wl.mistral7b_random(seed=23, requests=7, lo=50, hi=1400, layers=1, heads=1, head_dim=64)
    prob = DeviceProblem(w, fill_seed=FILL_SEED)
    prob.tt_slots = _misaligned_copy(prob.tt_slots, 1)
    prob.keep = _misaligned_copy(prob.keep, 3)
    prob.new_tt_slots = _misaligned_copy(prob.new_tt_slots, 1)
    assert prob.tt_slots.data_ptr() % 16 != 0 and prob.keep.data_ptr() % 4 != 0 and prob.new_tt_slots.data_ptr() % 16 != 0
    if planner == "whole":
        prob.plan()
    else:
        prob.plan_partial(util=(1, 1))
    prob.repack()
    out = prob.outputs()
    if planner == "whole":
        p = vto.plan_workload(w)
    else:
        p = vto.plan_partial(w.block_size, w.num_blocks, w.bt_offsets, w.bt_blocks, w.tt_offsets, w.tt_slots, w.keep,
                             w.free_blocks, w.select, w.thr_num, w.thr_den, util=(1, 1))
    assert_tables_equal(out, p, w)
    assert (prob.new_tt_slots[w.num_tokens:].cpu().numpy() == -9).all()
    k, v = host_pools(w)
    vto.apply_moves_pools(k, v, p.move_src, p.move_dst)
    assert np.array_equal(prob.k_pool.cpu().numpy().view(np.uint16), k)
    assert np.array_equal(prob.v_pool.cpu().numpy().view(np.uint16), v)
    prob.close()


@pytest.mark.parametrize("planner", ["whole", "partial"])
def test_token_table_that_does_not_start_at_entry_zero(planner):
    """tt_offsets[0] > 0: the entries in front of the first request belong to nobody; they are neither
    counted nor written, and every request is planned as if the table started at its first entry."""
    from harness.device import DeviceProblem
    torch = _torch()
    w = wl.mistral7b_random(seed=29, requests=6, lo=50, hi=900, layers=1, heads=1, head_dim=64)
    gap = 1029                                           # more than one tile, not a multiple of four
    prob = DeviceProblem(w, fill_seed=FILL_SEED, capacity_slack=gap)
    T = w.num_tokens
    shifted_slots = torch.zeros(T + gap, dtype=torch.int32, device=prob.device)     # slot 0 "live" in the gap
    shifted_slots[gap:] = prob.tt_slots[:T]
    shifted_keep = torch.ones(T + gap, dtype=torch.uint8, device=prob.device)
    shifted_keep[gap:] = prob.keep[:T]
    prob.tt_slots, prob.keep = shifted_slots, shifted_keep
    prob.tt_offsets = (prob.tt_offsets + gap).to(torch.int32)
    if planner == "whole":
        prob.plan()
        p = vto.plan_workload(w)
    else:
        prob.plan_partial(util=(1, 1))
        p = vto.plan_partial(w.block_size, w.num_blocks, w.bt_offsets, w.bt_blocks, w.tt_offsets, w.tt_slots, w.keep,
                             w.free_blocks, w.select, w.thr_num, w.thr_den, util=(1, 1))
    prob.repack()
    torch.cuda.synchronize()
    counts = prob.read_counts()
    assert counts["error_flags"] == 0 and counts["num_moves"] == p.num_moves
    assert np.array_equal(prob.req_status[:w.num_requests].cpu().numpy(), p.req_status)
    assert np.array_equal(prob.new_tt_slots[gap:gap + T].cpu().numpy(), p.new_tt_slots)
    assert (prob.new_tt_slots[:gap].cpu().numpy() == -9).all()          # untouched
    assert np.array_equal(prob.new_bt_blocks[:len(p.new_bt_blocks)].cpu().numpy(), p.new_bt_blocks)
    k, v = host_pools(w)
    vto.apply_moves_pools(k, v, p.move_src, p.move_dst)
    assert np.array_equal(prob.k_pool.cpu().numpy().view(np.uint16), k)
    assert np.array_equal(prob.v_pool.cpu().numpy().view(np.uint16), v)
    prob.close()


def test_argument_errors():
    from harness.device import DeviceProblem
    w = wl.tiny()
    prob = DeviceProblem(w)
    with pytest.raises(vt.VtokenError) as e:
        prob.repack()                                   # no plan yet
    assert e.value.code == vt.ESTATE
    with pytest.raises(vt.VtokenError) as e:
        prob.gather_logical(prob.tt_slots, prob.keep, 0, 2, 10)     # layer range beyond L = 1
    assert e.value.code == vt.EINVAL
    prob.close()


@pytest.mark.parametrize("heads,head_dim", [(2, 64), (4, 128), (8, 128), (3, 128)],
                         ids=["row256-register", "row1024-bulk", "row2048-bulk", "row768-bulk"])
def test_gather_logical_before_equals_after_and_matches_oracle(heads, head_dim):
    """Rows below 512 bytes go through the register kernel, the others through the bulk-copy kernel
    in gather mode; the last step replays the gather from a captured graph (its work tickets must
    be back at zero after every launch)."""
    from harness.device import DeviceProblem
    torch = _torch()
    w = wl.steady_state(seed=3, requests=10, lo=100, hi=900, layers=3, heads=heads, head_dim=head_dim)
    prob = DeviceProblem(w, fill_seed=FILL_SEED)
    cap = int(((w.tt_slots >= 0) & (w.keep != 0)).sum())
    bk, bv, boff = prob.gather_logical(prob.tt_slots, prob.keep, 0, 3, cap)
    prob.plan()
    prob.repack()
    ak, av, aoff = prob.gather_logical(prob.new_tt_slots, None, 0, 3, cap)
    torch.cuda.synchronize()
    assert torch.equal(bk, ak) and torch.equal(bv, av) and torch.equal(boff, aoff)
    # against the oracle's logical view of the untouched host pools
    k, v = host_pools(w)
    off = boff.cpu().numpy()
    R = w.num_requests
    assert off[R] == cap
    for pool, got in ((k, bk), (v, bv)):
        g = got.cpu().numpy().view(np.uint16)
        for l in range(3):
            for r in range(R):
                t0, t1 = w.tt_offsets[r], w.tt_offsets[r + 1]
                exp = vto.gather_logical(pool[l], w.tt_slots[t0:t1], w.keep[t0:t1])
                assert np.array_equal(g[l, off[r]:off[r + 1]], exp)
    # a layer sub-range and a request subset
    sel = np.zeros(R, np.uint8)
    sel[[1, 4, 7]] = 1
    sel_d = torch.from_numpy(sel).to(prob.device)
    sk, sv, soff = prob.gather_logical(prob.new_tt_slots, None, 1, 2, cap, select=sel_d)
    soff = soff.cpu().numpy()
    p = vto.plan_workload(w)
    k2, v2 = host_pools(w)
    vto.apply_moves_pools(k2, v2, p.move_src, p.move_dst)
    g = sk.cpu().numpy().view(np.uint16)
    for r in range(R):
        t0, t1 = w.tt_offsets[r], w.tt_offsets[r + 1]
        if sel[r]:
            assert np.array_equal(g[0, soff[r]:soff[r + 1]], vto.gather_logical(k2[1], p.new_tt_slots[t0:t1]))
        else:
            assert soff[r] == soff[r + 1]
    # overflow: capacity below the live count raises the flag, keeps what fits
    ok, ov, ooff = prob.gather_logical(prob.tt_slots, prob.keep, 0, 1, cap - 5)
    assert prob.read_counts()["error_flags"] & vt.FLAG_GATHER_OVERFLOW
    assert torch.equal(ok[0, :cap - 5], bk[0, :cap - 5])
    # captured once, replayed three times
    gk = torch.zeros((3, cap, w.row_elems), dtype=torch.int16, device=prob.device)
    gv = torch.zeros_like(gk)
    goff = torch.zeros(prob.max_requests + 1, dtype=torch.int32, device=prob.device)
    call = lambda st: vt.vtoken_gather_logical(prob.ctx, num_requests=prob.num_requests, tt_offsets=prob.tt_offsets,
                                               tt_slots=prob.new_tt_slots, keep=None, select=None, layer_begin=0,
                                               layer_end=3, out_k=gk, out_v=gv, out_capacity_tokens=cap,
                                               out_offsets=goff, stream=st)
    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    with torch.cuda.stream(side):
        call(side)
    side.synchronize()
    g = torch.cuda.CUDAGraph()
    with torch.cuda.graph(g, stream=side):
        call(torch.cuda.current_stream())
    for _ in range(3):
        gk.zero_()
        gv.zero_()
        torch.cuda.synchronize()
        g.replay()
        torch.cuda.synchronize()
        assert torch.equal(gk, ak) and torch.equal(gv, av) and torch.equal(goff, aoff)
    prob.close()


def test_repack_host_tables_entry_point():
    from harness.device import DeviceProblem
    torch = _torch()
    w = wl.mistral7b_random(seed=8, requests=12, lo=100, hi=400, layers=2, heads=2, head_dim=64)
    prob = DeviceProblem(w, fill_seed=FILL_SEED)
    R, T, NBT = w.num_requests, w.num_tokens, len(w.bt_blocks)
    pin = lambda a: torch.from_numpy(np.ascontiguousarray(a)).pin_memory()
    h_in = dict(bt_offsets=pin(w.bt_offsets), bt_blocks=pin(w.bt_blocks), tt_offsets=pin(w.tt_offsets),
                tt_slots=pin(w.tt_slots), keep=pin(w.keep), free_blocks=pin(w.free_blocks))
    h_out = dict(new_bt_offsets=torch.zeros(R + 1, dtype=torch.int32).pin_memory(),
                 new_bt_blocks=torch.zeros(NBT, dtype=torch.int32).pin_memory(),
                 new_tt_slots=torch.zeros(T, dtype=torch.int32).pin_memory(),
                 freed_blocks=torch.zeros(NBT, dtype=torch.int32).pin_memory(),
                 req_status=torch.zeros(R, dtype=torch.int32).pin_memory())
    s = torch.cuda.Stream()
    c = vt.vtoken_repack_host(prob.ctx, num_requests=R, num_free=len(w.free_blocks), **h_in, **h_out, stream=s)
    p = vto.plan_workload(w)
    assert c["num_moves"] == p.num_moves and c["error_flags"] == 0
    assert np.array_equal(h_out["new_tt_slots"].numpy(), p.new_tt_slots)
    assert np.array_equal(h_out["new_bt_offsets"].numpy(), p.new_bt_offsets)
    assert np.array_equal(h_out["new_bt_blocks"].numpy()[:len(p.new_bt_blocks)], p.new_bt_blocks)
    assert np.array_equal(h_out["freed_blocks"].numpy()[:p.num_freed], p.freed_blocks)
    assert np.array_equal(h_out["req_status"].numpy(), p.req_status)
    k, v = host_pools(w)
    vto.apply_moves_pools(k, v, p.move_src, p.move_dst)
    assert np.array_equal(prob.k_pool.cpu().numpy().view(np.uint16), k)
    assert np.array_equal(prob.v_pool.cpu().numpy().view(np.uint16), v)
    prob.close()


def test_graph_capture_side_stream_replay_with_new_contents():
    """plan + repack captured once on a side stream; replayed three times after rewriting the
    CONTENTS of the input buffers (same addresses, same capacities); a consumer on the main
    stream waits on the event recorded behind the replay (pre-attention visibility)."""
    from harness.device import DeviceProblem
    torch = _torch()
    base = wl.mistral7b_random(seed=30, requests=10, lo=100, hi=400, layers=2, heads=2, head_dim=64)
    prob = DeviceProblem(base, fill_seed=FILL_SEED, capacity_slack=64)
    side = torch.cuda.Stream()
    graph = torch.cuda.CUDAGraph()
    side.wait_stream(torch.cuda.current_stream())
    with torch.cuda.stream(side):
        prob.plan(stream=side)          # warm-up outside capture
        prob.repack(stream=side)
    side.synchronize()
    prob.fill_pools()
    torch.cuda.synchronize()
    with torch.cuda.graph(graph, stream=side):
        prob.plan(stream=torch.cuda.current_stream())
        prob.repack(stream=torch.cuda.current_stream())
    rng = np.random.default_rng(1)
    for it in range(3):
        keep = ((rng.random(base.num_tokens) < (0.2 + 0.25 * it))).astype(np.uint8)
        prob.keep[:len(keep)].copy_(torch.from_numpy(keep))
        prob.fill_pools()
        torch.cuda.synchronize()
        with torch.cuda.stream(side):
            graph.replay()
            done = torch.cuda.Event()
            done.record(side)
        torch.cuda.current_stream().wait_event(done)
        # consumer on the main stream: reads through the NEW tables after the event
        ak, av, aoff = prob.gather_logical(prob.new_tt_slots, None, 0, 2, base.num_tokens)
        w_it = wl.Workload(**{**base.__dict__, "keep": keep})
        p = vto.plan_workload(w_it)
        out = prob.outputs()
        assert_tables_equal(out, p, w_it)
        k, v = host_pools(base)
        k0 = k.copy()
        vto.apply_moves_pools(k, v, p.move_src, p.move_dst)
        assert np.array_equal(prob.k_pool.cpu().numpy().view(np.uint16), k)
        assert np.array_equal(prob.v_pool.cpu().numpy().view(np.uint16), v)
        # the consumer saw the logical view of the original cache
        off = aoff.cpu().numpy()
        g = ak.cpu().numpy().view(np.uint16)
        for r in range(base.num_requests):
            t0, t1 = base.tt_offsets[r], base.tt_offsets[r + 1]
            assert np.array_equal(g[1, off[r]:off[r + 1]], vto.gather_logical(k0[1], base.tt_slots[t0:t1], keep[t0:t1]))
    prob.close()


def test_decode_read_proxy_is_undisturbed_by_a_concurrent_repack():
    """A reader of every allocated block through the OLD block tables (decode-read proxy) runs on
    one stream while the captured repack runs on another: its per-request checksums must equal the
    solo values, because destinations are free blocks and sources are only read."""
    from harness import kernels as vh
    from harness.device import DeviceProblem
    torch = _torch()
    w = wl.steady_state(seed=9, requests=40, lo=300, hi=3000, layers=4)
    prob = DeviceProblem(w, fill_seed=FILL_SEED)
    owner = np.repeat(np.arange(w.num_requests, dtype=np.int32), np.diff(w.bt_offsets))
    owner_d = torch.from_numpy(owner).to(prob.device)
    nbt = len(w.bt_blocks)
    block_bytes = w.block_size * w.row_bytes

    def proxy(sums, stream):
        vh.vth_decode_read(prob.k_pool, prob.v_pool, prob.bt_offsets, prob.bt_blocks, owner_d, nbt, w.num_layers,
                           block_bytes, w.slab_bytes, sums, stream=stream)

    solo = torch.zeros(w.num_requests, dtype=torch.int64, device=prob.device)
    proxy(solo, torch.cuda.current_stream())
    torch.cuda.synchronize()
    assert int((solo != 0).sum()) == w.num_requests

    side, main = torch.cuda.Stream(), torch.cuda.Stream(priority=-1)
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.stream(side):
        prob.plan(stream=side)
        prob.repack(stream=side)
    side.synchronize()
    prob.fill_pools()
    torch.cuda.synchronize()
    with torch.cuda.graph(graph, stream=side):
        prob.plan(stream=torch.cuda.current_stream())
        prob.repack(stream=torch.cuda.current_stream())
    both = torch.zeros_like(solo)
    go = torch.cuda.Event()
    go.record()
    main.wait_event(go)
    side.wait_event(go)
    proxy(both, main)
    with torch.cuda.stream(side):
        graph.replay()
    torch.cuda.synchronize()
    assert torch.equal(both, solo)
    # and the repack that ran beside it is exact
    p = vto.plan_workload(w)
    k, v = host_pools(w)
    vto.apply_moves_pools(k, v, p.move_src, p.move_dst, threads=2)
    assert np.array_equal(prob.k_pool.cpu().numpy().view(np.uint16), k)
    assert np.array_equal(prob.v_pool.cpu().numpy().view(np.uint16), v)
    prob.close()


@pytest.mark.parametrize("tp", [2, 8])
def test_tensor_parallel_shards_repack_identically(tp):
    """Under tensor parallelism every shard holds the same blocks with its share of the KV heads
    (Sec. 6: shard-local block ids, nothing to exchange): the same tables planned on a shard's
    context give the same plan, and its pools after the repack are the head slice of the unsharded
    result -- which is the oracle's.  tp = 8 with 8 heads leaves rows of one head (256 bytes)."""
    import dataclasses
    from harness.device import DeviceProblem
    torch = _torch()
    w = wl.llama8b_h2o(seed=4, requests=5, lo=200, hi=700, layers=2, heads=8, head_dim=128)
    full = DeviceProblem(w, fill_seed=FILL_SEED)
    L, slots, H, D = w.num_layers, w.slots_per_layer, w.num_kv_heads, w.head_dim
    before_k = full.k_pool.view(L, slots, H, D).clone()
    before_v = full.v_pool.view(L, slots, H, D).clone()
    full.plan()
    full.repack()
    out = full.outputs()
    p = vto.plan_workload(w)
    assert_tables_equal(out, p, w)
    k, v = host_pools(w)
    vto.apply_moves_pools(k, v, p.move_src, p.move_dst, threads=2)
    assert np.array_equal(full.k_pool.cpu().numpy().view(np.uint16), k)
    assert np.array_equal(full.v_pool.cpu().numpy().view(np.uint16), v)
    after_k, after_v = full.k_pool.view(L, slots, H, D), full.v_pool.view(L, slots, H, D)
    per = H // tp
    ws = dataclasses.replace(w, num_kv_heads=per)
    for s in range(tp):
        heads = slice(s * per, (s + 1) * per)
        shard = DeviceProblem(ws, fill_seed=FILL_SEED)
        shard.k_pool.copy_(before_k[:, :, heads, :].reshape(L, slots, per * D))
        shard.v_pool.copy_(before_v[:, :, heads, :].reshape(L, slots, per * D))
        shard.plan()
        shard.repack()
        so = shard.outputs()
        assert so["error_flags"] == 0
        for name in ("new_bt_offsets", "new_bt_blocks", "new_tt_slots", "freed_blocks", "req_status", "num_moves"):
            assert np.array_equal(so[name], out[name]), name
        assert torch.equal(shard.k_pool.view(L, slots, per, D), after_k[:, :, heads, :])
        assert torch.equal(shard.v_pool.view(L, slots, per, D), after_v[:, :, heads, :])
        shard.close()
    full.close()
