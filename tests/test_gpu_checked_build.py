"""The checked build of the library (libvtoken_checked.so: the same sources with -DVTOKEN_CHECKED)
stands in for a memory sanitizer: every index a kernel forms into scratch, a table, a list or a pool
slab is compared with the array's size; an index outside it raises VTOKEN_FLAG_CHECK_FAILED, the access
is skipped, nothing faults.  This file runs the parity tests of the other files once more against that
build -- same oracle, same bit-exact bar -- and requires the flag to stay clear, which also covers what a
comparison of results cannot see: a read beyond an array, a stray write into the context's scratch.
(The checked build plans with the three-kernel planner unless told otherwise, the production build
uses the two-kernel one on tables this small; the two-kernel planner is run under the checker as well.)"""
import numpy as np
import pytest

from harness import workloads as wl
from oracle import vto
from paper_2608_13263_b200 import binding as vt

pytestmark = pytest.mark.gpu


@pytest.fixture
def checked(monkeypatch):
    """Every call of the binding goes to the checked build; every context is asked for its flags before
    it is destroyed, and none may have seen a failed check."""
    prev = vt.use_library("checked")
    seen = []
    destroy = vt.vtoken_destroy

    def destroy_after_reading_the_flags(ctx):
        seen.append(vt.vtoken_read_counts(ctx)["error_flags"])
        destroy(ctx)

    monkeypatch.setattr(vt, "vtoken_destroy", destroy_after_reading_the_flags)
    try:
        assert vt.vtoken_checked_build() == 1
        yield seen
        assert seen, "no context was created under the checked build"
        assert not any(f & vt.FLAG_CHECK_FAILED for f in seen), "an index left its array"
    finally:
        monkeypatch.undo()
        vt.use_library(prev)


def test_production_library_is_not_the_checked_one():
    assert vt.vtoken_checked_build() == 0


def test_the_checker_catches_an_index_outside_its_array(checked):
    """The mechanism itself: one thread reads element `index` of a scratch array of max_requests
    elements through the checked accessor.  Inside: no flag.  Outside (either side): the flag, no
    fault, and the context goes on working."""
    import torch
    from harness.device import DeviceProblem
    w = wl.tiny(seed=3)
    prob = DeviceProblem(w, fill_seed=1)
    out = torch.full((1,), -5, dtype=torch.int32, device=prob.device)
    for index in (0, prob.max_requests - 1):
        vt.vtoken_debug_probe(prob.ctx, index, out)
        assert prob.read_counts()["error_flags"] == 0
    for index in (prob.max_requests, -1, 1 << 40):
        vt.vtoken_debug_probe(prob.ctx, index, out)
        assert prob.read_counts()["error_flags"] == vt.FLAG_CHECK_FAILED
        assert prob.read_counts()["error_flags"] == 0          # reported once
    prob.plan()
    prob.repack()
    p = vto.plan_workload(w)
    outp = prob.outputs()
    assert np.array_equal(outp["new_tt_slots"], p.new_tt_slots) and prob.read_counts()["error_flags"] == 0
    prob.close()
    # the production library has no such probe
    prev = vt.use_library("production")
    try:
        prob = DeviceProblem(w, fill_seed=1)
        with pytest.raises(vt.VtokenError):
            vt.vtoken_debug_probe(prob.ctx, 0, out)
        prob.close()
    finally:
        vt.use_library(prev)


def test_small_configs_whole_pool(checked):
    import test_gpu_parity as tp
    for w in tp.small_configs():
        for variant in (1, 2):
            tp.run_and_compare(w, copy_variant=variant)      # tables, lists, counts, every byte; flags == 0
        tp.run_and_compare(w, copy_variant=2, plan_variant=2, whole_pool=False)      # the two-kernel planner's indices


def test_edges_and_shapes(checked):
    import test_gpu_parity as tp
    for S, heads, head_dim in ((1, 1, 8), (3, 2, 64), (16, 4, 128), (48, 8, 128), (5, 3, 8)):
        w = wl.mistral7b_random(seed=S, requests=5, lo=10, hi=40 * S + 20, layers=2, heads=heads, head_dim=head_dim,
                                block_size=S)
        tp.run_and_compare(w, copy_variant=2)
    # short free lists (prefix cut-off), a threshold, a request subset
    w = wl.mistral7b_random(seed=11, requests=9, lo=60, hi=400, layers=1, heads=1, head_dim=64)
    p = vto.plan_workload(w)
    for nf in (0, 1, p.num_dst_blocks // 2, p.num_dst_blocks - 1):
        tp.run_and_compare(w, num_free=nf)
    w = wl.steady_state(seed=2, requests=20, lo=100, hi=900, layers=1, heads=1, head_dim=64)
    tp.run_and_compare(w)
    # capacities larger than the problem (grids larger than the work)
    tp.run_and_compare(wl.tiny(seed=4), capacity_slack=3000)


def test_partial_planner_detach_and_waves(checked):
    import test_gpu_partial as tpp
    import test_gpu_waves as tw
    small = tpp.small_configs()
    # partial plans with every option set (the partial planner's own scratch and lists)
    for w in (small[1], small[4]):
        for opts in tpp.OPTION_SETS:
            tpp.test_partial_plans_small_whole_pool(w, opts)
    tpp.test_block_liveness_matches_oracle(small[2])
    # copy-on-write detach on the shared-prefix workload: released list, shared bytes untouched
    tpp.test_copy_on_write_detach_on_the_shared_prefix_workload(4, (1, 2), 0)
    tpp.test_copy_on_write_detach_on_the_shared_prefix_workload(4, (1, 4), 1)        # census hashes and their probes
    tpp.test_copy_on_write_detach_on_the_shared_prefix_workload(2, (1, 1), 2)
    tpp.test_detach_through_the_wave_entry_point_and_the_host_front_end(2, (1, 2), 1)
    tpp.test_shared_prefix_workload(2)
    # repack in waves, whole and partial: pool hand-over between the waves, commit kernel
    ws = tw.small_configs()
    tw.test_waves_with_the_headroom_of_one_request(ws[1], 3)
    tw.test_waves_pool_sizes(ws[2], 0.5)
    tw.test_partial_waves(ws[4], tw.PARTIALS[-1])


def test_fuzz_subset(checked):
    import test_gpu_fuzz as tf
    for seed in range(6):
        tf.test_fuzz_whole_and_partial_plans(seed)
    for seed in range(3):
        tf.test_fuzz_repack_in_waves(seed)


def test_gather_digest_slot_mapping(checked):
    import torch
    from harness.device import DeviceProblem
    w = wl.steady_state(seed=6, requests=14, lo=100, hi=1200, layers=3, heads=2, head_dim=64)
    prob = DeviceProblem(w, fill_seed=1)
    live = int(((w.tt_slots >= 0) & (w.keep != 0)).sum())
    gk, gv, goff = prob.gather_logical(prob.tt_slots, prob.keep, 0, 3, live)
    torch.cuda.synchronize()
    off = goff.cpu().numpy()
    for layer in range(3):
        ks = wl.fill_slab(1, 0, layer, w.num_layers, w.slots_per_layer, w.row_elems)
        for r in range(w.num_requests):
            t0, t1 = w.tt_offsets[r], w.tt_offsets[r + 1]
            want = vto.gather_logical(ks, w.tt_slots[t0:t1], w.keep[t0:t1])
            assert np.array_equal(gk[layer, off[r]:off[r + 1]].cpu().numpy().view(np.uint16), want)
    T, R = w.num_tokens, w.num_requests
    i32 = dict(dtype=torch.int32, device=prob.device)
    m_slots, m_ids, m_off = torch.zeros(T, **i32), torch.zeros(T, **i32), torch.zeros(prob.max_requests + 1, **i32)
    vt.vtoken_build_slot_mapping(prob.ctx, num_requests=prob.num_requests, tt_offsets=prob.tt_offsets,
                                 tt_slots=prob.tt_slots, keep=prob.keep, select=None, out_slots=m_slots,
                                 out_token_ids=m_ids, out_capacity=T, out_offsets=m_off)
    digest = torch.zeros(prob.max_requests, dtype=torch.int64, device=prob.device)
    vt.vtoken_digest_logical(prob.ctx, num_requests=prob.num_requests, tt_offsets=prob.tt_offsets,
                             tt_slots=prob.tt_slots, keep=prob.keep, select=None, layer_begin=0, layer_end=3,
                             out_digest=digest)
    torch.cuda.synchronize()
    o_slots, o_ids, o_off = vto.build_slot_mapping(w.tt_offsets, w.tt_slots, w.keep)
    assert np.array_equal(m_off.cpu().numpy()[:R + 1], o_off)
    assert np.array_equal(m_slots.cpu().numpy()[:len(o_slots)], o_slots)
    assert np.array_equal(m_ids.cpu().numpy()[:len(o_ids)], o_ids)
    k = np.stack([wl.fill_slab(1, 0, l, w.num_layers, w.slots_per_layer, w.row_elems) for l in range(3)])
    v = np.stack([wl.fill_slab(1, 1, l, w.num_layers, w.slots_per_layer, w.row_elems) for l in range(3)])
    for r in range(R):
        t0, t1 = w.tt_offsets[r], w.tt_offsets[r + 1]
        want, _ = vto.digest_logical(k, v, w.tt_slots[t0:t1], w.keep[t0:t1])
        assert int(digest[r].item()) & (2 ** 64 - 1) == want
    assert prob.read_counts()["error_flags"] == 0
    prob.close()


def test_serving_loop(checked):
    import test_gpu_runtime as tr
    # append / evict / slot mapping / repack / commit / slot cache, one configuration of each planner kind
    tr.test_serving_loop_matches_oracle_step_by_step(0, 4, (), ())
    tr.test_serving_loop_matches_oracle_step_by_step(3, 4, tr.PARTIAL_MIX, ())
    tr.test_serving_loop_matches_oracle_step_by_step(6, 4, tr.PARTIAL_MIX, (0, 2, 3, 4))


def test_address_fill_names_the_origin_of_every_row():
    """The address-encoding fill: after a repack every row of both pools must say it came from the slot
    the oracle's moves put there; a misrouted row would name the slot it really came from."""
    from harness.device import DeviceProblem, origin_map
    w = wl.llama8b_h2o(seed=1, requests=4, lo=200, hi=700, layers=2, heads=2, head_dim=64)
    prob = DeviceProblem(w, fill_mode="address")
    host = wl.fill_slab_address(1, 1, w.slots_per_layer, w.row_elems)       # the numpy twin and the kernel agree
    assert np.array_equal(prob.v_pool[1].cpu().numpy().view(np.uint16), host)
    prob.plan()
    prob.repack()
    p = vto.plan_workload(w)
    origin = origin_map(w.slots_per_layer, p.move_src, p.move_dst)
    moved = 0
    for kv, pool in ((0, prob.k_pool), (1, prob.v_pool)):
        for layer in range(w.num_layers):
            slab = pool[layer].cpu().numpy().view(np.uint16)
            for s in range(w.slots_per_layer):
                got = wl.decode_row_address(slab[s])
                assert got == (kv, layer, int(origin[s])), f"row {(kv, layer, s)} holds the bytes of {got}"
                moved += int(origin[s] != s)
    assert moved == 2 * w.num_layers * p.num_moves
    prob.close()
