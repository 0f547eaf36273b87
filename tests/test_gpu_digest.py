"""GPU parity of the relocation digest: equal to the oracle's per request, equal before and after
a repack (token conservation without materialising the rows), different after a defect."""
import numpy as np
import pytest

from oracle import vto
from paper_2608_13263_b200 import binding as vt
from harness import workloads as wl

pytestmark = pytest.mark.gpu


def host_pools(w, seed=1):
    k = np.stack([wl.fill_slab(seed, 0, l, w.num_layers, w.slots_per_layer, w.row_elems) for l in range(w.num_layers)])
    v = np.stack([wl.fill_slab(seed, 1, l, w.num_layers, w.slots_per_layer, w.row_elems) for l in range(w.num_layers)])
    return k, v


def device_digest(prob, tt_slots, keep, l0, l1, select=None):
    import torch
    dig = torch.full((prob.max_requests,), -1, dtype=torch.int64, device=prob.device)
    off = torch.full((prob.max_requests + 1,), -1, dtype=torch.int32, device=prob.device)
    vt.vtoken_digest_logical(prob.ctx, num_requests=prob.num_requests, tt_offsets=prob.tt_offsets, tt_slots=tt_slots,
                             keep=keep, select=select, layer_begin=l0, layer_end=l1, out_digest=dig, out_offsets=off)
    torch.cuda.synchronize()
    return dig.cpu().numpy().view(np.uint64), off.cpu().numpy()


@pytest.mark.parametrize("w", [
    wl.tiny(seed=0),
    wl.steady_state(seed=2, requests=9, lo=50, hi=900, layers=3, heads=2, head_dim=64),
    wl.longctx_scissor(seed=1, requests=2, lo=2000, hi=5000, layers=2),
    # row sizes that exercise every lane-group width of the kernel and its tail loop:
    # 16 B, 48 B, 384 B, 1.5 KiB, 2 KiB, 4 KiB rows
    wl.mistral7b_random(seed=5, requests=5, lo=40, hi=300, layers=2, heads=1, head_dim=8),
    wl.mistral7b_random(seed=6, requests=5, lo=40, hi=300, layers=2, heads=1, head_dim=24),
    wl.mistral7b_random(seed=7, requests=5, lo=40, hi=300, layers=2, heads=3, head_dim=64),
    wl.mistral7b_random(seed=8, requests=5, lo=40, hi=300, layers=1, heads=6, head_dim=128),
    wl.mistral7b_random(seed=9, requests=5, lo=40, hi=300, layers=1, heads=8, head_dim=128),
    wl.mistral7b_random(seed=10, requests=4, lo=40, hi=200, layers=1, heads=16, head_dim=128),
], ids=lambda w: f"{w.name}-row{w.row_bytes}")
def test_digest_matches_oracle_and_survives_repack(w):
    import torch
    from harness.device import DeviceProblem
    prob = DeviceProblem(w, fill_seed=1)
    L = w.num_layers
    k, v = host_pools(w)
    R = w.num_requests
    before, off = device_digest(prob, prob.tt_slots, prob.keep, 0, L)
    for r in range(R):
        t0, t1 = w.tt_offsets[r], w.tt_offsets[r + 1]
        d, n = vto.digest_logical(k, v, w.tt_slots[t0:t1], w.keep[t0:t1])
        assert int(before[r]) == d and off[r + 1] - off[r] == n
    # a layer sub-range
    sub, _ = device_digest(prob, prob.tt_slots, prob.keep, L - 1, L)
    t0, t1 = w.tt_offsets[0], w.tt_offsets[1]
    assert int(sub[0]) == vto.digest_logical(k, v, w.tt_slots[t0:t1], w.keep[t0:t1], L - 1, L)[0]
    # repack, then the digest through the new tables must be the same
    prob.plan()
    prob.repack()
    after, off2 = device_digest(prob, prob.new_tt_slots, None, 0, L)
    assert np.array_equal(before[:R], after[:R]) and np.array_equal(off[:R + 1], off2[:R + 1])
    assert prob.outputs()["num_moves"] > 0
    # a defect: exchange the slots of two live tokens of request 0 in the new table
    new = prob.new_tt_slots.clone()
    live = torch.nonzero(new[t0:t1] >= 0).flatten()[:2] + int(t0)
    a, b = int(new[live[0]]), int(new[live[1]])
    new[live[0]], new[live[1]] = b, a
    broken, _ = device_digest(prob, new, None, 0, L)
    assert broken[0] != after[0] and np.array_equal(broken[1:R], after[1:R])
    prob.close()
