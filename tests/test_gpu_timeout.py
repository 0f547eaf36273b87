"""The bounded wait of the bulk-copy kernel: when a shared-memory barrier never completes, the
waiting warp gives up after the configured limit, raises VTOKEN_FLAG_TIMEOUT, lets its copies in
flight land and returns -- the kernel ends, the context and the GPU stay usable.

The stall is produced without faulting anything: a test hook arms the barrier of ONE work item
with 16 bytes that no copy will ever deliver (every real copy still runs and completes).  The
hook exists only in the checked build of the library (vtoken_config.debug_stall_item; the
production library refuses the field), the limit is vtoken_config.wait_limit_ms."""

import numpy as np
import pytest

from oracle import vto
from paper_2608_13263_b200 import binding as vt
from harness import workloads as wl

pytestmark = pytest.mark.gpu


def test_wait_runs_out_sets_flag_and_context_survives():
    import torch
    from harness.device import DeviceProblem
    w = wl.llama8b_h2o(seed=0, requests=4, lo=200, hi=600, layers=2)
    # the production library has no such hook
    with pytest.raises(vt.VtokenError) as e:
        DeviceProblem(w, fill_seed=1, copy_variant=2, wait_limit_ms=20, debug_stall_item=6)
    assert e.value.code == vt.EINVAL
    prev = vt.use_library("checked")
    try:
        assert vt.vtoken_checked_build() == 1
        _stalled_launch_and_recovery(w)
    finally:
        vt.use_library(prev)


def _stalled_launch_and_recovery(w):
    import torch
    from harness.device import DeviceProblem
    prob = DeviceProblem(w, fill_seed=1, copy_variant=2, wait_limit_ms=20, debug_stall_item=6)   # item 5
    prob.plan()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    prob.repack()
    e1.record()
    torch.cuda.synchronize()
    ms = e0.elapsed_time(e1)
    flags = prob.read_counts()["error_flags"]
    assert flags & vt.FLAG_TIMEOUT
    assert 15.0 < ms < 2000.0                       # gave up after the 20 ms limit (plus the bounded drain)
    out = prob.outputs()
    p = vto.plan_workload(w)
    assert np.array_equal(out["new_tt_slots"], p.new_tt_slots)      # the plan itself is unaffected
    prob.close()

    # same process, same GPU, a fresh context without the hook: everything works and is exact
    prob = DeviceProblem(w, fill_seed=1, copy_variant=2)
    prob.plan()
    prob.repack()
    assert prob.read_counts()["error_flags"] == 0
    k = np.stack([wl.fill_slab(1, 0, l, w.num_layers, w.slots_per_layer, w.row_elems) for l in range(w.num_layers)])
    v = np.stack([wl.fill_slab(1, 1, l, w.num_layers, w.slots_per_layer, w.row_elems) for l in range(w.num_layers)])
    vto.apply_moves_pools(k, v, p.move_src, p.move_dst)
    assert np.array_equal(prob.k_pool.cpu().numpy().view(np.uint16), k)
    assert np.array_equal(prob.v_pool.cpu().numpy().view(np.uint16), v)
    prob.close()
