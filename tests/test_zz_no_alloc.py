"""vtoken_gather_logical_noalloc: the logical gather for callers that cannot allocate device
memory (an engine whose HBM is fully committed to the KV pool, a latency-critical step that
cannot take cudaMalloc's device-wide synchronisation, an embedder that forbids allocator
calls).  Its scratch is a fixed array in the library image, shared by all calls and carrying
the previous call's contents, so the check is: two calls in a row, the second on different
tables with fewer live tokens, each bit-identical to what the context-based
vtoken_gather_logical returns for the same inputs, and each compared directly with the CPU
oracle's logical view of the same pools as well.

Collected last on purpose (file name), so a failure here cannot hide any other test.
"""
import numpy as np
import pytest

from harness import workloads as wl
from oracle import vto
from paper_2608_13263_b200 import binding as vt

pytestmark = pytest.mark.gpu


def test_noalloc_gather_equals_context_gather_twice_in_a_row():
    import torch
    from harness.device import DeviceProblem
    w = wl.steady_state(seed=6, requests=14, lo=100, hi=1200, layers=3, heads=2, head_dim=64)
    prob = DeviceProblem(w, fill_seed=1)
    dev = prob.device
    live = int(((w.tt_slots >= 0) & (w.keep != 0)).sum())
    resident = int((w.tt_slots >= 0).sum())
    cap = resident
    assert cap <= vt.NOALLOC_MAX_TOKENS

    def noalloc(tt_slots, keep, l0, l1, capacity, select=None):
        out_k = torch.zeros((l1 - l0, capacity, w.row_elems), dtype=torch.int16, device=dev)
        out_v = torch.zeros_like(out_k)
        out_off = torch.full((prob.max_requests + 1,), -9, dtype=torch.int32, device=dev)
        flags = torch.full((1,), 12345, dtype=torch.int32, device=dev)
        vt.vtoken_gather_logical_noalloc(
            k_pool=prob.k_pool, v_pool=prob.v_pool, num_layers=w.num_layers, num_blocks=w.num_blocks,
            block_size=w.block_size, row_bytes=w.row_bytes, num_requests=prob.num_requests,
            max_requests=prob.max_requests, tt_offsets=prob.tt_offsets, tt_slots=tt_slots, keep=keep, select=select,
            layer_begin=l0, layer_end=l1, out_k=out_k, out_v=out_v, out_capacity_tokens=capacity,
            out_offsets=out_off, error_flags=flags)
        return out_k, out_v, out_off, flags

    # call 1: every resident token (keep = NULL), all layers -- the larger problem first
    k1, v1, off1, f1 = noalloc(prob.tt_slots, None, 0, 3, cap)
    # call 2: kept tokens only, one layer, a request subset -- fewer rows than call 1 left behind
    sel = torch.zeros(prob.max_requests, dtype=torch.uint8, device=dev)
    sel[::2] = 1
    k2, v2, off2, f2 = noalloc(prob.tt_slots, prob.keep, 1, 2, cap, select=sel)
    torch.cuda.synchronize()

    ek1, ev1, eoff1 = prob.gather_logical(prob.tt_slots, None, 0, 3, cap)
    ek2, ev2, eoff2 = prob.gather_logical(prob.tt_slots, prob.keep, 1, 2, cap, select=sel)
    torch.cuda.synchronize()
    R = w.num_requests
    assert int(eoff1[R]) == resident and int(eoff2[R]) < live
    for got, exp in ((k1, ek1), (v1, ev1), (k2, ek2), (v2, ev2)):
        assert torch.equal(got, exp)
    assert torch.equal(off1[:R + 1], eoff1[:R + 1]) and torch.equal(off2[:R + 1], eoff2[:R + 1])
    assert int(f1) == 0 and int(f2) == 0

    # ... and against the oracle itself: per request, per layer, K and V, rows in token-id order
    def slab(kv, layer):
        return wl.fill_slab(1, kv, layer, w.num_layers, w.slots_per_layer, w.row_elems)

    def check_against_oracle(got_k, got_v, got_off, keep, l0, l1, selected):
        off = got_off.cpu().numpy()
        for li, layer in enumerate(range(l0, l1)):
            ks, vs = slab(0, layer), slab(1, layer)
            gk = got_k[li].cpu().numpy().view(np.uint16)
            gv = got_v[li].cpu().numpy().view(np.uint16)
            for r in range(R):
                t0, t1 = w.tt_offsets[r], w.tt_offsets[r + 1]
                if not selected(r):
                    assert off[r + 1] == off[r]
                    continue
                kp = None if keep is None else keep[t0:t1]
                want_k = vto.gather_logical(ks, w.tt_slots[t0:t1], kp)
                want_v = vto.gather_logical(vs, w.tt_slots[t0:t1], kp)
                assert off[r + 1] - off[r] == len(want_k)
                assert np.array_equal(gk[off[r]:off[r + 1]], want_k), (layer, r)
                assert np.array_equal(gv[off[r]:off[r + 1]], want_v), (layer, r)

    check_against_oracle(k1, v1, off1, None, 0, 3, lambda r: True)
    check_against_oracle(k2, v2, off2, w.keep, 1, 2, lambda r: r % 2 == 0)

    # overflow is reported through error_flags, like the context version reports it in its counts
    k3, v3, off3, f3 = noalloc(prob.tt_slots, None, 0, 1, resident - 7)
    torch.cuda.synchronize()
    assert int(f3) & vt.FLAG_GATHER_OVERFLOW
    assert torch.equal(k3[0], ek1[0, :resident - 7])

    # sizes beyond the fixed scratch are refused with a clear error, nothing is enqueued
    with pytest.raises(vt.VtokenError) as e:
        noalloc(prob.tt_slots, None, 0, 1, vt.NOALLOC_MAX_TOKENS + 1)
    assert e.value.code == vt.ECAPACITY
    with pytest.raises(vt.VtokenError) as e:
        vt.vtoken_gather_logical_noalloc(
            k_pool=prob.k_pool, v_pool=prob.v_pool, num_layers=w.num_layers, num_blocks=w.num_blocks,
            block_size=w.block_size, row_bytes=w.row_bytes, num_requests=prob.num_requests,
            max_requests=vt.NOALLOC_MAX_REQUESTS + 1, tt_offsets=prob.tt_offsets, tt_slots=prob.tt_slots, keep=None,
            select=None, layer_begin=0, layer_end=1, out_k=k3, out_v=v3, out_capacity_tokens=16, out_offsets=off3)
    assert e.value.code == vt.ECAPACITY
    prob.close()
