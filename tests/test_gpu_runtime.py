"""GPU parity of the device-side token-table runtime (evict, append, slot mapping, commit) and of
the whole serving loop around the repack: the same seeded step sequence runs on the oracle and
through the C ABI; after every step all table state, the slot mapping and the logical K/V view
must be identical."""
import numpy as np
import pytest

from oracle import vto
from paper_2608_13263_b200 import binding as vt

from runtime_sim import Append, DictCache, Evict, Repack, ServingState, random_serving_steps

pytestmark = pytest.mark.gpu


class DeviceServing:
    """Device copy of a ServingState plus small K/V pools whose rows carry (request, token)."""

    def __init__(self, st, layers=2, row_elems=8, max_victims=64):
        import torch
        self.torch = torch
        dev = torch.device("cuda:0")
        self.dev = dev
        self.S, self.NB, self.R = st.S, st.num_blocks, st.R
        self.row_elems = row_elems
        self.layers = layers
        i32 = dict(dtype=torch.int32, device=dev)
        self.num_requests = torch.tensor([st.R], **i32)
        self.tt_offsets = torch.from_numpy(st.tt_offsets).to(dev)
        cap = int(st.tt_offsets[-1])
        self.cap = cap
        self.tt_slots = torch.from_numpy(st.tt_slots.copy()).to(dev)
        self.keep = torch.from_numpy(st.keep.copy()).to(dev)
        self.tt_len = torch.from_numpy(st.tt_len.copy()).to(dev)
        self.phys_len = torch.from_numpy(st.phys_len.copy()).to(dev)
        self.bt_offsets = torch.zeros(st.R + 1, **i32)
        self.bt_blocks = torch.zeros(self.NB, **i32)
        self.free_blocks = torch.zeros(self.NB, **i32)
        self.num_free = torch.zeros(1, **i32)
        self.new_len = torch.zeros(st.R, **i32)
        self.max_victims = max_victims
        self.victim_req = torch.zeros(max_victims, **i32)
        self.victim_tok = torch.zeros(max_victims, **i32)
        self.num_victims = torch.zeros(1, **i32)
        self.new_bt_offsets = torch.zeros(st.R + 1, **i32)
        self.new_bt_blocks = torch.zeros(self.NB, **i32)
        self.new_tt_slots = torch.zeros(cap, **i32)
        self.freed_blocks = torch.zeros(self.NB, **i32)
        self.req_status = torch.zeros(st.R, **i32)
        self.counts = torch.zeros(8, **i32)
        self.map_slots = torch.zeros(cap, **i32)
        self.map_ids = torch.zeros(cap, **i32)
        self.map_offsets = torch.zeros(st.R + 1, **i32)
        # cached slot-translation arrays (poisoned so that untouched entries are recognisable)
        self.dirty = torch.zeros(st.R, dtype=torch.uint8, device=dev)
        self.cache_slots = torch.full((cap,), -77, **i32)
        self.cache_ids = torch.full((cap,), -77, **i32)
        self.cache_len = torch.zeros(st.R, **i32)
        self.cache_seen = torch.zeros(st.R, **i32)
        self.cache_stats = torch.zeros(2, **i32)
        # per-block liveness kept current by the counted interfaces (None: plain interfaces)
        self.n_b = self.live_total = None
        self.k_pool = torch.zeros((layers, self.NB * self.S, row_elems), dtype=torch.int16, device=dev)
        self.v_pool = torch.zeros_like(self.k_pool)
        self.ctx = vt.vtoken_create(layers, self.NB, self.S, 1, row_elems, self.k_pool, self.v_pool, st.R, cap,
                                    self.NB, self.NB)

    def enable_counters(self):
        t = self.torch
        self.n_b = t.zeros(self.NB, dtype=t.int32, device=self.dev)
        self.live_total = t.zeros(1, dtype=t.int64, device=self.dev)

    def recount(self, st):
        """After a repack: per-block liveness recomputed on the device."""
        t = self.torch
        self.upload_blocks(st)
        summary = t.zeros(2, dtype=t.int64, device=self.dev)
        vt.vtoken_block_liveness(self.ctx, num_requests=self.num_requests, bt_offsets=self.bt_offsets,
                                 bt_blocks=self.bt_blocks, tt_offsets=self.tt_offsets, tt_slots=self.tt_slots,
                                 keep=self.keep, n_b=self.n_b, summary=summary)
        self.live_total.copy_(summary[:1])

    def upload_blocks(self, st):
        t = self.torch
        self.bt_offsets.copy_(t.from_numpy(st.bt_offsets))
        b = st.bt_blocks
        self.bt_blocks[:len(b)].copy_(t.from_numpy(b))

    @staticmethod
    def payload(r, t, layer, kv, row_elems):
        base = np.array([r, t & 0x7FFF, t >> 15, layer, kv, r ^ t & 0xFF, 7, -3], np.int16)
        return np.resize(base, row_elems)

    # ---- the three steps through the C ABI ------------------------------------------------
    def append(self, st_before_len, st, new_len):
        t = self.torch
        self.upload_blocks(st)                                  # scheduler grew the block lists on the host
        self.new_len.copy_(t.from_numpy(np.asarray(new_len, np.int32)))
        args = dict(num_requests=self.num_requests, tt_offsets=self.tt_offsets, tt_slots=self.tt_slots,
                    keep=self.keep, tt_len=self.tt_len, phys_len=self.phys_len, bt_offsets=self.bt_offsets,
                    bt_blocks=self.bt_blocks, new_len=self.new_len)
        if self.n_b is None:
            vt.vtoken_sync_new_tokens(self.ctx, **args)
        else:
            vt.vtoken_sync_new_tokens_counted(self.ctx, n_b=self.n_b, live_total=self.live_total, **args)
        # "the model" writes the K/V of the new tokens at the slots the runtime assigned
        slots = self.tt_slots.cpu().numpy()
        lens = self.tt_len.cpu().numpy()
        for r in range(self.R):
            for tok in range(int(st_before_len[r]), int(lens[r])):
                s = int(slots[st.tt_offsets[r] + tok])
                for l in range(self.layers):
                    self.k_pool[l, s] = t.from_numpy(self.payload(r, tok, l, 0, self.row_elems)).to(self.dev)
                    self.v_pool[l, s] = t.from_numpy(self.payload(r, tok, l, 1, self.row_elems)).to(self.dev)

    def evict(self, victim_req, victim_tok):
        t = self.torch
        n = len(victim_req)
        assert n <= self.max_victims
        self.victim_req[:n].copy_(t.from_numpy(victim_req))
        self.victim_tok[:n].copy_(t.from_numpy(victim_tok))
        self.num_victims.fill_(n)
        args = dict(num_victims=self.num_victims, max_victims=self.max_victims, victim_req=self.victim_req,
                    victim_tok=self.victim_tok, num_requests=self.num_requests, tt_offsets=self.tt_offsets,
                    tt_len=self.tt_len, keep=self.keep)
        if self.n_b is None:
            vt.vtoken_evict_tokens(self.ctx, **args)
        else:
            vt.vtoken_evict_tokens_counted(self.ctx, tt_slots=self.tt_slots, n_b=self.n_b,
                                           live_total=self.live_total, **args)

    def repack(self, st, free, nf, thr, partial=None):
        t = self.torch
        self.upload_blocks(st)
        self.free_blocks[:len(free)].copy_(t.from_numpy(np.asarray(free, np.int32)))
        self.num_free.fill_(nf)
        side = t.cuda.Stream()
        side.wait_stream(t.cuda.current_stream())
        args = dict(num_requests=self.num_requests, bt_offsets=self.bt_offsets, bt_blocks=self.bt_blocks,
                    tt_offsets=self.tt_offsets, tt_slots=self.tt_slots, keep=self.keep,
                    free_blocks=self.free_blocks, num_free=self.num_free, new_bt_offsets=self.new_bt_offsets,
                    new_bt_blocks=self.new_bt_blocks, new_tt_slots=self.new_tt_slots,
                    freed_blocks=self.freed_blocks, req_status=self.req_status, counts=self.counts,
                    thr_num=thr[0], thr_den=thr[1], stream=side)
        if partial is None:
            vt.vtoken_plan(self.ctx, **args)
        else:
            vt.vtoken_plan_partial(self.ctx, **args, **partial)
        vt.vtoken_repack(self.ctx, stream=side)
        done = t.cuda.Event()
        done.record(side)
        t.cuda.current_stream().wait_event(done)                # commit only behind the repack event
        vt.vtoken_apply_moves(self.ctx, num_requests=self.num_requests, tt_offsets=self.tt_offsets,
                              tt_slots=self.tt_slots, keep=self.keep, phys_len=self.phys_len,
                              new_tt_slots=self.new_tt_slots, req_status=self.req_status,
                              new_bt_offsets=self.new_bt_offsets)

    def repack_waves(self, st, free, nf, thr, partial, waves):
        """Plan + copy + commit in waves on a side stream, then the table commit with the append
        positions the waves report."""
        t = self.torch
        i32 = dict(dtype=t.int32, device=self.dev)
        self.upload_blocks(st)
        self.free_blocks[:len(free)].copy_(t.from_numpy(np.asarray(free, np.int32)))
        self.num_free.fill_(nf)
        nbytes = vt.vtoken_waves_workspace_bytes(self.ctx, self.NB)
        wv = dict(req_wave=t.full((self.R,), -9, **i32), req_append_pos=t.full((self.R,), -9, **i32),
                  free_out=t.full((self.NB,), -9, **i32), num_free_out=t.zeros(1, **i32),
                  wave_counts=t.zeros((waves, 8), **i32), workspace=t.empty(nbytes, dtype=t.uint8, device=self.dev))
        side = t.cuda.Stream()
        side.wait_stream(t.cuda.current_stream())
        vt.vtoken_repack_waves(self.ctx, num_requests=self.num_requests, bt_offsets=self.bt_offsets,
                               bt_blocks=self.bt_blocks, tt_offsets=self.tt_offsets, tt_slots=self.tt_slots,
                               keep=self.keep, free_blocks=self.free_blocks, num_free=self.num_free, num_waves=waves,
                               new_bt_offsets=self.new_bt_offsets, new_bt_blocks=self.new_bt_blocks,
                               new_tt_slots=self.new_tt_slots, req_status=self.req_status, free_capacity=self.NB,
                               workspace_bytes=nbytes, thr_num=thr[0], thr_den=thr[1], partial=partial, stream=side,
                               **wv)
        done = t.cuda.Event()
        done.record(side)
        t.cuda.current_stream().wait_event(done)
        vt.vtoken_apply_moves(self.ctx, num_requests=self.num_requests, tt_offsets=self.tt_offsets,
                              tt_slots=self.tt_slots, keep=self.keep, phys_len=self.phys_len,
                              new_tt_slots=self.new_tt_slots, req_status=self.req_status,
                              append_pos=wv["req_append_pos"])
        t.cuda.synchronize()
        return wv

    def slot_mapping(self):
        vt.vtoken_build_slot_mapping(self.ctx, num_requests=self.num_requests, tt_offsets=self.tt_offsets,
                                     tt_slots=self.tt_slots, keep=self.keep, select=None, out_slots=self.map_slots,
                                     out_token_ids=self.map_ids, out_capacity=self.cap, out_offsets=self.map_offsets)
        off = self.map_offsets.cpu().numpy()
        n = int(off[self.R])
        return self.map_slots.cpu().numpy()[:n], self.map_ids.cpu().numpy()[:n], off

    def cache_mark(self, victims=False, status=False):
        vt.vtoken_slot_cache_mark(self.ctx, dirty=self.dirty, num_requests=self.num_requests,
                                  num_victims=self.num_victims if victims else None,
                                  max_victims=self.max_victims if victims else 0,
                                  victim_req=self.victim_req if victims else None,
                                  req_status=self.req_status if status else None)

    def cache_update(self):
        vt.vtoken_slot_cache_update(self.ctx, num_requests=self.num_requests, tt_offsets=self.tt_offsets,
                                    tt_slots=self.tt_slots, keep=self.keep, tt_len=self.tt_len, dirty=self.dirty,
                                    cache_slots=self.cache_slots, cache_ids=self.cache_ids, cache_len=self.cache_len,
                                    cache_seen=self.cache_seen, stats=self.cache_stats)
        return tuple(self.cache_stats.cpu().numpy().tolist())

    def close(self):
        self.torch.cuda.synchronize()
        vt.vtoken_destroy(self.ctx)


PARTIAL_MIX = (None, dict(util=(1, 1)), dict(util=(1, 2)), dict(util=(3, 4), max_source_blocks=3), dict())


@pytest.mark.parametrize("seed,S,partial_options,wave_options", [
    (0, 4, (), ()), (1, 16, (), ()), (2, 3, (), ()), (3, 4, PARTIAL_MIX, ()), (4, 16, PARTIAL_MIX, ()),
    (5, 3, PARTIAL_MIX, ()), (6, 4, PARTIAL_MIX, (0, 2, 3, 4)), (7, 8, PARTIAL_MIX, (2, 3, 5)),
    (8, 3, PARTIAL_MIX, (0, 3, 4))])
def test_serving_loop_matches_oracle_step_by_step(seed, S, partial_options, wave_options):
    import torch
    rng = np.random.default_rng(seed)
    R = 5
    st = ServingState.random(rng, S, R, capacity=260 if partial_options else 200,
                             num_blocks=600 if partial_options else 400)
    truth = DictCache()
    dev = DeviceServing(st)
    n_cap = int(st.tt_offsets[-1])
    oc = dict(dirty=np.zeros(R, np.uint8), slots=np.full(n_cap, -77, np.int32), ids=np.full(n_cap, -77, np.int32),
              len=np.zeros(R, np.int32), seen=np.zeros(R, np.int32))      # the oracle's cached arrays
    repacked_something = False
    for step in random_serving_steps(rng, st, steps=36 if partial_options else 25, partial_options=partial_options,
                                     wave_options=wave_options):
        if isinstance(step, Append):
            before = st.tt_len.copy()
            step.run_on_oracle(st, None, truth)
            dev.append(before, st, step.new_len)
        elif isinstance(step, Evict):
            step.run_on_oracle(st, None, truth)
            dev.evict(step.victim_req, step.victim_tok)
            vto.slot_cache_mark(oc["dirty"], victim_req=step.victim_req)
            dev.cache_mark(victims=True)
        else:
            free = list(st.free)
            nf = len(free) if step.num_free_limit < 0 else min(len(free), step.num_free_limit)
            blocks_before = st.bt_blocks.copy()
            st_before = ServingState(st.S, st.num_blocks, st.tt_offsets, st.tt_slots.copy(), st.keep.copy(),
                                     st.tt_len.copy(), st.phys_len.copy(), [b.copy() for b in st.block_lists], free)
            step.run_on_oracle(st, None, truth)
            p = step.last_plan
            if step.waves:
                wv = dev.repack_waves(st_before, free, nf, step.thr, step.partial, step.waves)
                repacked_something |= len(p.move_src) > 0
                for k in range(step.waves):
                    c = wv["wave_counts"][k].cpu().numpy()
                    assert c[:6].tolist() == [p.wave_counts[k][n] for n in
                                              ("num_moves", "num_dst_blocks", "num_freed", "num_free_consumed",
                                               "num_admitted", "num_deferred")] and c[6] == 0
                assert np.array_equal(dev.req_status.cpu().numpy(), p.req_status)
                assert np.array_equal(wv["req_wave"].cpu().numpy(), p.req_wave)
                assert np.array_equal(wv["req_append_pos"].cpu().numpy(), p.req_append_pos)
                assert np.array_equal(dev.new_bt_offsets.cpu().numpy(), p.new_bt_offsets)
                assert np.array_equal(dev.new_bt_blocks.cpu().numpy()[:len(p.new_bt_blocks)], p.new_bt_blocks)
                assert np.array_equal(wv["free_out"].cpu().numpy()[:int(wv["num_free_out"].item())], p.free_out)
            else:
                dev.repack(st_before, free, nf, step.thr, step.partial)
                repacked_something |= p.num_moves > 0
                c = dev.counts.cpu().numpy()
                assert c[:6].tolist() == [p.num_moves, p.num_dst_blocks, p.num_freed, p.num_free_consumed,
                                          p.num_admitted, p.num_deferred] and c[6] == 0
                assert np.array_equal(dev.req_status.cpu().numpy(), p.req_status)
                assert np.array_equal(dev.new_bt_offsets.cpu().numpy(), p.new_bt_offsets)
                assert np.array_equal(dev.new_bt_blocks.cpu().numpy()[:len(p.new_bt_blocks)], p.new_bt_blocks)
                assert np.array_equal(dev.freed_blocks.cpu().numpy()[:p.num_freed], p.freed_blocks)
            assert len(blocks_before) >= len(p.new_bt_blocks)
            vto.slot_cache_mark(oc["dirty"], req_status=p.req_status)
            dev.cache_mark(status=True)
        torch.cuda.synchronize()
        # cached slot-translation arrays: marks, then one update per step, everything bit for bit
        assert np.array_equal(dev.dirty.cpu().numpy(), oc["dirty"])
        want_stats = vto.slot_cache_update(st.tt_offsets, st.tt_slots, st.keep, st.tt_len, oc["dirty"], oc["slots"],
                                           oc["ids"], oc["len"], oc["seen"])
        assert dev.cache_update() == want_stats
        assert np.array_equal(dev.cache_slots.cpu().numpy(), oc["slots"])
        assert np.array_equal(dev.cache_ids.cpu().numpy(), oc["ids"])
        assert np.array_equal(dev.cache_len.cpu().numpy(), oc["len"])
        assert np.array_equal(dev.cache_seen.cpu().numpy(), oc["seen"])
        assert not dev.dirty.cpu().numpy().any()
        # the device tables still satisfy every input precondition (unique mapping among them)
        dev.upload_blocks(st)
        dev.free_blocks[:len(st.free)].copy_(torch.from_numpy(np.asarray(st.free, np.int32)))
        dev.num_free.fill_(len(st.free))
        bits = torch.full((1,), -1, dtype=torch.int32, device=dev.dev)
        vt.vtoken_check_tables(dev.ctx, num_requests=dev.num_requests, bt_offsets=dev.bt_offsets,
                               bt_blocks=dev.bt_blocks, tt_offsets=dev.tt_offsets, tt_slots=dev.tt_slots,
                               free_blocks=dev.free_blocks, num_free=dev.num_free, out_bits=bits)
        assert int(bits.item()) == 0
        # table state
        assert np.array_equal(dev.tt_slots.cpu().numpy(), st.tt_slots)
        assert np.array_equal(dev.keep.cpu().numpy(), st.keep)
        assert np.array_equal(dev.tt_len.cpu().numpy(), st.tt_len)
        assert np.array_equal(dev.phys_len.cpu().numpy(), st.phys_len)
        # slot mapping
        g_slots, g_ids, g_off = dev.slot_mapping()
        o_slots, o_ids, o_off = vto.build_slot_mapping(st.tt_offsets, st.tt_slots, st.keep)
        assert np.array_equal(g_slots, o_slots) and np.array_equal(g_ids, o_ids) and np.array_equal(g_off, o_off)
        # logical K/V view == what the dictionary cache holds, in token order
        k = dev.k_pool.cpu().numpy()
        v = dev.v_pool.cpu().numpy()
        for r in range(R):
            want = truth.live_tokens(r)
            assert g_ids[g_off[r]:g_off[r + 1]].tolist() == want
            for l in range(dev.layers):
                rows_k = k[l][g_slots[g_off[r]:g_off[r + 1]]]
                rows_v = v[l][g_slots[g_off[r]:g_off[r + 1]]]
                for i, tok in enumerate(want):
                    assert np.array_equal(rows_k[i], dev.payload(r, tok, l, 0, dev.row_elems))
                    assert np.array_equal(rows_v[i], dev.payload(r, tok, l, 1, dev.row_elems))
    assert repacked_something
    # random victim lists name tokens outside the registered range now and then (skipped, flagged); the flags
    # of the calls outside plan / repack stay up until they are read
    assert vt.vtoken_read_counts(dev.ctx)["error_flags"] & ~vt.FLAG_BAD_VICTIM == 0
    dev.close()


def test_runtime_flags_and_edges():
    import torch
    S = 4
    st = ServingState.empty(S, capacities=[10, 6], block_lists=[np.array([2, 9], np.int32), np.array([5], np.int32)],
                            num_blocks=12)
    dev = DeviceServing(st)
    # growth beyond the block list / the table capacity stops early and raises the flag
    ref = ServingState.empty(S, capacities=[10, 6], block_lists=[np.array([2, 9], np.int32), np.array([5], np.int32)],
                             num_blocks=12)
    for new_len in ([3, 2], [7, 2], [12, 6]):
        vto.sync_new_tokens(S, ref.tt_offsets, ref.tt_slots, ref.keep, ref.tt_len, ref.phys_len, ref.bt_offsets,
                            ref.bt_blocks, new_len)
        dev.upload_blocks(ref)
        dev.new_len.copy_(torch.tensor(new_len, dtype=torch.int32))
        vt.vtoken_sync_new_tokens(dev.ctx, num_requests=dev.num_requests, tt_offsets=dev.tt_offsets,
                                  tt_slots=dev.tt_slots, keep=dev.keep, tt_len=dev.tt_len, phys_len=dev.phys_len,
                                  bt_offsets=dev.bt_offsets, bt_blocks=dev.bt_blocks, new_len=dev.new_len)
        torch.cuda.synchronize()
        assert np.array_equal(dev.tt_slots.cpu().numpy(), ref.tt_slots)
        assert np.array_equal(dev.tt_len.cpu().numpy(), ref.tt_len)
        assert np.array_equal(dev.phys_len.cpu().numpy(), ref.phys_len)
    assert vt.vtoken_read_counts(dev.ctx)["error_flags"] & vt.FLAG_APPEND_STOPPED
    # victims outside the registered tokens are skipped and flagged
    vr = np.array([0, 1, 1, 0, 2, -1], np.int32)
    vtok = np.array([3, 0, 11, 10, 0, 0], np.int32)
    bad = vto.evict_tokens(ref.tt_offsets, ref.tt_len, ref.keep, vr, vtok)
    assert bad == 4
    dev.evict(vr, vtok)
    torch.cuda.synchronize()
    assert np.array_equal(dev.keep.cpu().numpy(), ref.keep)
    assert vt.vtoken_read_counts(dev.ctx)["error_flags"] & vt.FLAG_BAD_VICTIM
    # slot mapping into a buffer that is too small: what fits is kept, the flag is raised
    o_slots, o_ids, o_off = vto.build_slot_mapping(ref.tt_offsets, ref.tt_slots, ref.keep)
    small = torch.full((4,), -1, dtype=torch.int32, device=dev.dev)
    vt.vtoken_build_slot_mapping(dev.ctx, num_requests=dev.num_requests, tt_offsets=dev.tt_offsets,
                                 tt_slots=dev.tt_slots, keep=dev.keep, select=None, out_slots=small,
                                 out_token_ids=None, out_capacity=4, out_offsets=dev.map_offsets)
    torch.cuda.synchronize()
    assert np.array_equal(small.cpu().numpy(), o_slots[:4])
    assert np.array_equal(dev.map_offsets.cpu().numpy(), o_off)
    assert vt.vtoken_read_counts(dev.ctx)["error_flags"] & vt.FLAG_GATHER_OVERFLOW
    # flags of these calls are reported once
    assert vt.vtoken_read_counts(dev.ctx)["error_flags"] == 0
    dev.close()


def test_append_into_a_block_list_with_a_bad_id():
    """A block id outside [0, num_blocks), fabricated on the host: the tokens that would land in it are
    registered without a physical copy (slot -1, not kept), the flag is raised, everything else is as
    the oracle computes it for the valid part, and nothing faults."""
    import torch
    S = 4
    blocks = [np.array([2, 99, 7], np.int32), np.array([5, -3], np.int32)]        # 99 and -3 do not exist
    st = ServingState.empty(S, capacities=[12, 8], block_lists=blocks, num_blocks=12)
    dev = DeviceServing(st)
    dev.upload_blocks(st)
    dev.new_len.copy_(torch.tensor([11, 6], dtype=torch.int32))
    vt.vtoken_sync_new_tokens(dev.ctx, num_requests=dev.num_requests, tt_offsets=dev.tt_offsets,
                              tt_slots=dev.tt_slots, keep=dev.keep, tt_len=dev.tt_len, phys_len=dev.phys_len,
                              bt_offsets=dev.bt_offsets, bt_blocks=dev.bt_blocks, new_len=dev.new_len)
    torch.cuda.synchronize()
    slots, keep = dev.tt_slots.cpu().numpy(), dev.keep.cpu().numpy()
    assert slots[:11].tolist() == [8, 9, 10, 11, -1, -1, -1, -1, 28, 29, 30] and slots[11] == -1
    assert keep[:12].tolist() == [1, 1, 1, 1, 0, 0, 0, 0, 1, 1, 1, 0]
    assert slots[12:18].tolist() == [20, 21, 22, 23, -1, -1] and keep[12:18].tolist() == [1, 1, 1, 1, 0, 0]
    assert dev.tt_len.cpu().numpy().tolist() == [11, 6] and dev.phys_len.cpu().numpy().tolist() == [11, 6]
    assert vt.vtoken_read_counts(dev.ctx)["error_flags"] == vt.FLAG_BAD_BLOCK
    # the unmapped tokens are invisible to the slot mapping, like every token without a physical copy
    g_slots, g_ids, g_off = dev.slot_mapping()
    o_slots, o_ids, o_off = vto.build_slot_mapping(st.tt_offsets, slots, keep)
    assert np.array_equal(g_slots, o_slots) and np.array_equal(g_ids, o_ids) and np.array_equal(g_off, o_off)
    assert (g_slots >= 0).all()
    dev.close()


def test_slot_mapping_overlaps_plan_and_repack_on_another_stream():
    """The slot mapping is built every decode step on the compute stream while a plan and its copy run
    on a side stream (Sec. 3.3.4).  The two use separate scratch: replayed against each other many
    times without any ordering between the streams, both must still equal the oracle."""
    import torch
    from harness import workloads as wl
    from harness.device import DeviceProblem
    w = wl.steady_state(seed=3, requests=96, lo=200, hi=3000, layers=2, heads=2, head_dim=64)
    prob = DeviceProblem(w, fill_seed=1)
    dev = prob.device
    T, R = w.num_tokens, w.num_requests
    i32 = dict(dtype=torch.int32, device=dev)
    m_slots, m_ids, m_off = torch.full((T,), -5, **i32), torch.full((T,), -5, **i32), torch.full((R + 1,), -5, **i32)
    digest = torch.zeros(prob.max_requests, dtype=torch.int64, device=dev)
    main, side = torch.cuda.Stream(), torch.cuda.Stream()

    def mapping(st):
        vt.vtoken_build_slot_mapping(prob.ctx, num_requests=prob.num_requests, tt_offsets=prob.tt_offsets,
                                     tt_slots=prob.tt_slots, keep=prob.keep, select=None, out_slots=m_slots,
                                     out_token_ids=m_ids, out_capacity=T, out_offsets=m_off, stream=st)
        vt.vtoken_digest_logical(prob.ctx, num_requests=prob.num_requests, tt_offsets=prob.tt_offsets,
                                 tt_slots=prob.tt_slots, keep=prob.keep, select=None, layer_begin=0,
                                 layer_end=w.num_layers, out_digest=digest, stream=st)

    def relocation(st):
        prob.plan(stream=st)
        prob.repack(stream=st)

    for fn, st in ((mapping, main), (relocation, side)):     # warm-up outside the captures
        with torch.cuda.stream(st):
            fn(st)
    torch.cuda.synchronize()
    g_map, g_rel = torch.cuda.CUDAGraph(), torch.cuda.CUDAGraph()
    with torch.cuda.graph(g_map, stream=main):
        mapping(torch.cuda.current_stream())
    with torch.cuda.graph(g_rel, stream=side):
        relocation(torch.cuda.current_stream())
    torch.cuda.synchronize()
    m_slots.fill_(-5)
    prob.new_tt_slots.fill_(-9)
    torch.cuda.synchronize()
    for _ in range(40):                                       # no event between the two streams
        with torch.cuda.stream(main):
            g_map.replay()
        with torch.cuda.stream(side):
            g_rel.replay()
    torch.cuda.synchronize()

    o_slots, o_ids, o_off = vto.build_slot_mapping(w.tt_offsets, w.tt_slots, w.keep)
    n = len(o_slots)
    assert np.array_equal(m_off.cpu().numpy(), o_off)
    assert np.array_equal(m_slots.cpu().numpy()[:n], o_slots) and np.array_equal(m_ids.cpu().numpy()[:n], o_ids)
    out = prob.outputs()
    p = vto.plan_workload(w)
    assert out["error_flags"] == 0 and out["num_moves"] == p.num_moves
    assert np.array_equal(out["new_tt_slots"], p.new_tt_slots) and np.array_equal(out["new_bt_blocks"], p.new_bt_blocks)
    assert np.array_equal(out["freed_blocks"], p.freed_blocks) and np.array_equal(out["req_status"], p.req_status)
    k = np.stack([wl.fill_slab(1, 0, l, w.num_layers, w.slots_per_layer, w.row_elems) for l in range(w.num_layers)])
    v = np.stack([wl.fill_slab(1, 1, l, w.num_layers, w.slots_per_layer, w.row_elems) for l in range(w.num_layers)])
    want, _ = vto.digest_logical(k, v, w.tt_slots[w.tt_offsets[0]:w.tt_offsets[1]],
                                 w.keep[w.tt_offsets[0]:w.tt_offsets[1]])
    assert int(digest[0].item()) & (2 ** 64 - 1) == int(want) & (2 ** 64 - 1)
    vto.apply_moves_pools(k, v, p.move_src, p.move_dst, threads=2)
    assert np.array_equal(prob.k_pool.cpu().numpy().view(np.uint16), k)
    assert np.array_equal(prob.v_pool.cpu().numpy().view(np.uint16), v)
    assert prob.read_counts()["error_flags"] == 0
    prob.close()


def test_slot_mapping_full_size_tables_match_oracle():
    """Slot mapping over the steady-state workload's token tables (2.2 M logical entries)."""
    import torch
    from harness import workloads as wl
    from harness.device import DeviceProblem
    w = wl.steady_state(seed=0)
    prob = DeviceProblem(w, allocate_pools=False)
    # the context wants pools: a one-layer pool of 16-byte rows is enough for table-only calls
    pool = torch.zeros((1, w.slots_per_layer, 8), dtype=torch.int16, device=prob.device)
    ctx = vt.vtoken_create(1, w.num_blocks, w.block_size, 1, 8, pool, pool, prob.max_requests, prob.max_tokens,
                           prob.max_table_blocks, prob.max_free)
    T = w.num_tokens
    out_slots = torch.full((T,), -1, dtype=torch.int32, device=prob.device)
    out_ids = torch.full((T,), -1, dtype=torch.int32, device=prob.device)
    out_off = torch.zeros(w.num_requests + 1, dtype=torch.int32, device=prob.device)
    vt.vtoken_build_slot_mapping(ctx, num_requests=prob.num_requests, tt_offsets=prob.tt_offsets,
                                 tt_slots=prob.tt_slots, keep=prob.keep, select=None, out_slots=out_slots,
                                 out_token_ids=out_ids, out_capacity=T, out_offsets=out_off)
    torch.cuda.synchronize()
    o_slots, o_ids, o_off = vto.build_slot_mapping(w.tt_offsets, w.tt_slots, w.keep)
    n = len(o_slots)
    assert np.array_equal(out_off.cpu().numpy(), o_off)
    assert np.array_equal(out_slots.cpu().numpy()[:n], o_slots)
    assert np.array_equal(out_ids.cpu().numpy()[:n], o_ids)
    vt.vtoken_destroy(ctx)


def test_slot_cache_full_size_rebuild_then_append_only():
    """Steady-state tables (2.2 M entries, 512 requests) with one spare entry per request: a fresh
    cache is rebuilt for every request and equals the slot mapping; a decode step that appends one
    token per request then only appends; an eviction in three requests rebuilds exactly those."""
    import torch
    from harness import workloads as wl
    w = wl.steady_state(seed=0)
    R = w.num_requests
    dev = torch.device("cuda:0")
    lens = np.diff(w.tt_offsets).astype(np.int32)
    cap_off = (w.tt_offsets.astype(np.int64) + np.arange(R + 1)).astype(np.int32)
    n = int(cap_off[-1])
    tt = np.full(n, -1, np.int32)
    keep = np.zeros(n, np.uint8)
    for r in range(R):
        tt[cap_off[r]:cap_off[r] + lens[r]] = w.tt_slots[w.tt_offsets[r]:w.tt_offsets[r + 1]]
        keep[cap_off[r]:cap_off[r] + lens[r]] = w.keep[w.tt_offsets[r]:w.tt_offsets[r + 1]]
    tt_len = lens.copy()
    pool = torch.zeros((1, w.slots_per_layer, 8), dtype=torch.int16, device=dev)
    ctx = vt.vtoken_create(1, w.num_blocks, w.block_size, 1, 8, pool, pool, R, n, len(w.bt_blocks), 1)
    d = lambda a: torch.from_numpy(np.ascontiguousarray(a)).to(dev)
    g = dict(num_requests=d(np.array([R], np.int32)), tt_offsets=d(cap_off), tt_slots=d(tt), keep=d(keep),
             tt_len=d(tt_len), dirty=d(np.ones(R, np.uint8)), cache_slots=d(np.full(n, -77, np.int32)),
             cache_ids=d(np.full(n, -77, np.int32)), cache_len=d(np.zeros(R, np.int32)),
             cache_seen=d(np.zeros(R, np.int32)), stats=d(np.zeros(2, np.int32)))
    o = dict(dirty=np.ones(R, np.uint8), slots=np.full(n, -77, np.int32), ids=np.full(n, -77, np.int32),
             len=np.zeros(R, np.int32), seen=np.zeros(R, np.int32))

    def both(expect):
        got = vto.slot_cache_update(cap_off, tt, keep, tt_len, o["dirty"], o["slots"], o["ids"], o["len"], o["seen"])
        assert got == expect
        vt.vtoken_slot_cache_update(ctx, **g)
        torch.cuda.synchronize()
        assert tuple(g["stats"].cpu().numpy().tolist()) == expect
        for a, b in (("cache_slots", "slots"), ("cache_ids", "ids"), ("cache_len", "len"), ("cache_seen", "seen"),
                     ("dirty", "dirty")):
            assert np.array_equal(g[a].cpu().numpy(), o[b]), a

    both((R, 0))
    slots, ids, off = vto.build_slot_mapping(cap_off, tt, keep)
    for r in (0, 1, R // 2, R - 1):
        assert np.array_equal(o["slots"][cap_off[r]:cap_off[r] + o["len"][r]], slots[off[r]:off[r + 1]])
    # one decode step: every request registers one token at a slot of its own
    for r in range(R):
        tt[cap_off[r] + tt_len[r]] = w.num_blocks * w.block_size - 1 - r
        keep[cap_off[r] + tt_len[r]] = 1
    tt_len += 1
    g["tt_slots"].copy_(d(tt)); g["keep"].copy_(d(keep)); g["tt_len"].copy_(d(tt_len))
    both((0, R))
    both((0, 0))
    # evictions in three requests, marked through the library
    vr = np.array([3, 3, 100, R - 1], np.int32)
    for r, t in zip(vr.tolist(), (0, 5, 7, 2)):
        keep[cap_off[r] + t] = 0
    g["keep"].copy_(d(keep))
    vto.slot_cache_mark(o["dirty"], victim_req=vr)
    vt.vtoken_slot_cache_mark(ctx, dirty=g["dirty"], num_requests=g["num_requests"],
                              num_victims=d(np.array([4], np.int32)), max_victims=4, victim_req=d(vr))
    both((3, 0))
    assert vt.vtoken_read_counts(ctx)["error_flags"] == 0
    vt.vtoken_destroy(ctx)


@pytest.mark.parametrize("seed,S", [(10, 4), (11, 16), (12, 3)])
def test_incremental_block_liveness_on_the_device(seed, S):
    """The counted evict / append interfaces keep n_b and the live total current on the device
    (recounted only after repacks); after every step they equal the oracle's counters, which the
    CPU tests pin against a recount.  Victim batches contain repeats and already evicted tokens."""
    import torch
    rng = np.random.default_rng(seed)
    R = 5
    st = ServingState.random(rng, S, R, capacity=260, num_blocks=600)
    st.enable_counters()
    dev = DeviceServing(st)
    dev.enable_counters()
    for step in random_serving_steps(rng, st, steps=30, partial_options=PARTIAL_MIX):
        if isinstance(step, Append):
            before = st.tt_len.copy()
            step.run_on_oracle(st, None, None)
            dev.append(before, st, step.new_len)
        elif isinstance(step, Evict):
            step.run_on_oracle(st, None, None)
            dev.evict(step.victim_req, step.victim_tok)
        else:
            free = list(st.free)
            nf = len(free) if step.num_free_limit < 0 else min(len(free), step.num_free_limit)
            st_before = ServingState(st.S, st.num_blocks, st.tt_offsets, st.tt_slots.copy(), st.keep.copy(),
                                     st.tt_len.copy(), st.phys_len.copy(), [b.copy() for b in st.block_lists], free)
            step.run_on_oracle(st, None, None)
            dev.repack(st_before, free, nf, step.thr, step.partial)
            dev.recount(st)
        torch.cuda.synchronize()
        assert np.array_equal(dev.keep.cpu().numpy(), st.keep)
        assert np.array_equal(dev.tt_slots.cpu().numpy(), st.tt_slots)
        assert np.array_equal(dev.n_b.cpu().numpy(), st.counters["n_b"])
        assert int(dev.live_total.item()) == int(st.counters["live"][0])
    assert vt.vtoken_read_counts(dev.ctx)["error_flags"] & ~vt.FLAG_BAD_VICTIM == 0
    dev.close()
