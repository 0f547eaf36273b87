"""Device-resident repack problem: torch is used for device memory and streams only; every
step of the path runs in the CUDA library through the C-ABI binding.

``DeviceProblem`` uploads a ``workloads.Workload`` (tables, masks, free list), allocates and
fills the K/V pools with the harness fill kernel, creates a library context and exposes
``plan()``, ``repack()``, ``gather_logical()`` plus host copies of the outputs.
"""
from __future__ import annotations

import numpy as np
import torch

from paper_2608_13263_b200 import binding as vt

from . import kernels as vh
from .workloads import Workload


class DeviceProblem:
    def __init__(self, w: Workload, device="cuda:0", fill_seed: int = 1, copy_variant: int = 0, max_ctas: int = 0,
                 capacity_slack: int = 0, allocate_pools: bool = True, wave_capacity: bool = False,
                 ctx_capacity: dict = None, fill_mode: str = "random", **ctx_options):
        """``ctx_options``: further keyword arguments of ``vtoken_create`` (wait_limit_ms,
        plain_launches, tuning, debug_stall_item).  ``fill_mode``: "random" (the seeded pool fill) or
        "address" (every row says where it was filled: a debugging aid)."""
        self.fill_mode = fill_mode
        self.w = w
        self.device = torch.device(device)
        self.fill_seed = fill_seed
        dev = self.device
        R, T, NBT = w.num_requests, w.num_tokens, len(w.bt_blocks)
        self.max_requests = max(1, R + capacity_slack)
        self.max_tokens = max(1, T + capacity_slack)
        self.max_table_blocks = max(1, NBT + capacity_slack)
        self.max_free = max(1, len(w.free_blocks) + capacity_slack)
        if wave_capacity:       # a pool that takes back every reclaimed block (repack in waves)
            self.max_free += self.max_table_blocks
        self._waves = None

        def up(a, dtype):
            t = torch.from_numpy(np.ascontiguousarray(a, dtype=dtype))
            out = torch.empty(max(1, t.numel()), dtype=t.dtype, device=dev)
            out[:t.numel()].copy_(t)
            return out

        self.num_requests = up([R], np.int32)
        self.num_free = up([len(w.free_blocks)], np.int32)
        self.bt_offsets = up(w.bt_offsets, np.int32)
        self.bt_blocks = self._padded(w.bt_blocks, np.int32, self.max_table_blocks)
        self.tt_offsets = up(w.tt_offsets, np.int32)
        self.tt_slots = self._padded(w.tt_slots, np.int32, self.max_tokens)
        self.keep = self._padded(w.keep, np.uint8, self.max_tokens)
        self.select = None if w.select is None else self._padded(w.select, np.uint8, self.max_requests)
        self.free_blocks = self._padded(w.free_blocks, np.int32, self.max_free)

        i32 = dict(dtype=torch.int32, device=dev)
        self.new_bt_offsets = torch.full((self.max_requests + 1,), -9, **i32)
        self.new_bt_blocks = torch.full((self.max_table_blocks,), -9, **i32)
        self.new_tt_slots = torch.full((self.max_tokens,), -9, **i32)
        self.freed_blocks = torch.full((self.max_table_blocks,), -9, **i32)
        self.released_blocks = torch.full((self.max_table_blocks,), -9, **i32)
        self.req_status = torch.full((self.max_requests,), -9, **i32)
        self.counts = torch.zeros(8, **i32)

        self.k_pool = self.v_pool = None
        self.ctx = None
        if allocate_pools:
            shape = (w.num_layers, w.slots_per_layer, w.row_elems)
            self.k_pool = torch.empty(shape, dtype=torch.int16, device=dev)
            self.v_pool = torch.empty(shape, dtype=torch.int16, device=dev)
            self.fill_pools()
            self._caps = dict(max_requests=self.max_requests, max_tokens=self.max_tokens,
                              max_table_blocks=self.max_table_blocks, max_free=self.max_free)
            self._caps.update(ctx_capacity or {})     # a context smaller than the buffers (capacity tests)
            self.ctx = self.make_ctx(max_ctas=max_ctas, copy_variant=copy_variant, **ctx_options)

    def make_ctx(self, **options):
        """A (further) library context over this problem's pools; the caller destroys it."""
        w, caps = self.w, self._caps
        return vt.vtoken_create(w.num_layers, w.num_blocks, w.block_size, w.num_kv_heads, w.head_dim,
                                self.k_pool, self.v_pool, caps["max_requests"], caps["max_tokens"],
                                caps["max_table_blocks"], caps["max_free"], elem_bytes=w.elem_bytes, **options)

    def _padded(self, a, dtype, n):
        out = torch.zeros(max(1, n), dtype=torch.from_numpy(np.zeros(1, dtype)).dtype, device=self.device)
        a = np.ascontiguousarray(a, dtype=dtype)
        if a.size:
            out[:a.size].copy_(torch.from_numpy(a))
        return out

    # ---- pools --------------------------------------------------------------------------
    def fill_pools(self, stream=None):
        w = self.w
        for kv, pool in ((0, self.k_pool), (1, self.v_pool)):
            if self.fill_mode == "address":
                vh.vth_fill_address(pool, kv, w.num_layers, 0, w.num_layers, w.slots_per_layer, w.row_elems,
                                    stream=stream)
            else:
                vh.vth_fill(pool, kv, w.num_layers, 0, w.num_layers, w.slots_per_layer, w.row_elems, self.fill_seed,
                            stream=stream)

    def fresh_slab(self, kv: int, layer: int) -> torch.Tensor:
        """Pre-repack content of one (K|V, layer) slab, regenerated on the device."""
        w = self.w
        out = torch.empty((w.slots_per_layer, w.row_elems), dtype=torch.int16, device=self.device)
        vh.vth_fill(out, kv, w.num_layers, layer, layer + 1, w.slots_per_layer, w.row_elems, self.fill_seed)
        return out

    def verify_pools(self, origin: np.ndarray) -> int:
        """Number of 32-bit words of K and V, all layers, that differ from fill(origin[slot])."""
        w = self.w
        org = torch.from_numpy(np.ascontiguousarray(origin, dtype=np.int32)).to(self.device)
        bad = torch.zeros(1, dtype=torch.int64, device=self.device)
        for kv, pool in ((0, self.k_pool), (1, self.v_pool)):
            vh.vth_verify(pool, kv, w.num_layers, w.slots_per_layer, w.row_elems, self.fill_seed, org, bad)
        return int(bad.item())

    # ---- the path -----------------------------------------------------------------------
    def plan(self, stream=None, num_free=None, ctx=None):
        vt.vtoken_plan(ctx or self.ctx, num_requests=self.num_requests, bt_offsets=self.bt_offsets,
                       bt_blocks=self.bt_blocks, tt_offsets=self.tt_offsets, tt_slots=self.tt_slots, keep=self.keep,
                       free_blocks=self.free_blocks, num_free=self.num_free if num_free is None else num_free,
                       new_bt_offsets=self.new_bt_offsets, new_bt_blocks=self.new_bt_blocks,
                       new_tt_slots=self.new_tt_slots, freed_blocks=self.freed_blocks, req_status=self.req_status,
                       counts=self.counts, select=self.select, thr_num=self.w.thr_num, thr_den=self.w.thr_den,
                       stream=stream)

    def plan_partial(self, stream=None, num_free=None, protect=None, util=(0, 0), max_source_blocks=0, theta=(0, 0),
                     detach=(0, 0), detach_rule=0, ctx=None):
        vt.vtoken_plan_partial(ctx or self.ctx, num_requests=self.num_requests, bt_offsets=self.bt_offsets,
                               bt_blocks=self.bt_blocks, tt_offsets=self.tt_offsets, tt_slots=self.tt_slots,
                               keep=self.keep, free_blocks=self.free_blocks,
                               num_free=self.num_free if num_free is None else num_free,
                               new_bt_offsets=self.new_bt_offsets, new_bt_blocks=self.new_bt_blocks,
                               new_tt_slots=self.new_tt_slots, freed_blocks=self.freed_blocks,
                               req_status=self.req_status, counts=self.counts, select=self.select,
                               thr_num=self.w.thr_num, thr_den=self.w.thr_den, protect=protect, util=util,
                               max_source_blocks=max_source_blocks, theta=theta, detach=detach,
                               detach_rule=detach_rule, released_blocks=self.released_blocks,
                               stream=stream)

    def repack(self, stream=None, ctx=None):
        vt.vtoken_repack(ctx or self.ctx, stream=stream)

    def repack_waves(self, num_waves: int, num_free=None, partial=None, stream=None):
        """Plan + copy + commit, ``num_waves`` times, reclaimed blocks feeding the next wave.  Needs
        ``wave_capacity=True`` at construction.  Results: ``waves_outputs()``."""
        dev = self.device
        if self._waves is None or self._waves["counts"].shape[0] < num_waves:
            i32 = dict(dtype=torch.int32, device=dev)
            nbytes = vt.vtoken_waves_workspace_bytes(self.ctx, self.max_free)
            self._waves = dict(req_wave=torch.full((self.max_requests,), -9, **i32),
                               req_append_pos=torch.full((self.max_requests,), -9, **i32),
                               free_out=torch.full((self.max_free,), -9, **i32),
                               num_free_out=torch.full((1,), -9, **i32),
                               released=torch.full((self.max_table_blocks,), -9, **i32),
                               num_released=torch.full((1,), -9, **i32),
                               counts=torch.zeros((num_waves, 8), **i32),
                               workspace=torch.empty(max(16, nbytes), dtype=torch.uint8, device=dev), nbytes=nbytes)
        wv = self._waves
        vt.vtoken_repack_waves(self.ctx, num_requests=self.num_requests, bt_offsets=self.bt_offsets,
                               bt_blocks=self.bt_blocks, tt_offsets=self.tt_offsets, tt_slots=self.tt_slots,
                               keep=self.keep, free_blocks=self.free_blocks,
                               num_free=self.num_free if num_free is None else num_free, num_waves=num_waves,
                               new_bt_offsets=self.new_bt_offsets, new_bt_blocks=self.new_bt_blocks,
                               new_tt_slots=self.new_tt_slots, req_status=self.req_status, req_wave=wv["req_wave"],
                               free_out=wv["free_out"], num_free_out=wv["num_free_out"], wave_counts=wv["counts"],
                               free_capacity=self.max_free, workspace=wv["workspace"], workspace_bytes=wv["nbytes"],
                               select=self.select, thr_num=self.w.thr_num, thr_den=self.w.thr_den, partial=partial,
                               req_append_pos=wv["req_append_pos"], released_blocks=wv["released"],
                               num_released=wv["num_released"], stream=stream)

    def waves_outputs(self, num_waves: int) -> dict:
        """Host copies of the outputs of ``repack_waves``."""
        torch.cuda.synchronize(self.device)
        R, T = self.w.num_requests, self.w.num_tokens
        wv = self._waves
        names = ["num_moves", "num_dst_blocks", "num_freed", "num_free_consumed", "num_admitted", "num_deferred"]
        c = wv["counts"].cpu().numpy()[:num_waves]
        out = dict(wave_counts=[dict({n: int(row[i]) for i, n in enumerate(names)}, error_flags=int(np.uint32(row[6])))
                                for row in c])
        nbo = self.new_bt_offsets.cpu().numpy()[:R + 1]
        out["new_bt_offsets"] = nbo
        out["new_bt_blocks"] = self.new_bt_blocks.cpu().numpy()[:int(nbo[R])]
        out["new_tt_slots"] = self.new_tt_slots.cpu().numpy()[:T]
        out["req_status"] = self.req_status.cpu().numpy()[:R]
        out["req_wave"] = wv["req_wave"].cpu().numpy()[:R]
        out["req_append_pos"] = wv["req_append_pos"].cpu().numpy()[:R]
        nfo = int(wv["num_free_out"].item())
        out["free_out"] = wv["free_out"].cpu().numpy()[:nfo]
        out["released_blocks"] = wv["released"].cpu().numpy()[:int(wv["num_released"].item())]
        return out

    def read_counts(self, stream=None) -> dict:
        return vt.vtoken_read_counts(self.ctx, stream=stream)

    def outputs(self) -> dict:
        """Host copies of every planner output, trimmed by the counts the device wrote."""
        torch.cuda.synchronize(self.device)
        R, T = self.w.num_requests, self.w.num_tokens
        c = self.counts.cpu().numpy()
        names = ["num_moves", "num_dst_blocks", "num_freed", "num_free_consumed", "num_admitted", "num_deferred"]
        out = {n: int(c[i]) for i, n in enumerate(names)}
        out["error_flags"] = int(np.uint32(c[6]))
        out["num_released"] = int(c[7])
        out["released_blocks"] = self.released_blocks.cpu().numpy()[:out["num_released"]]
        nbo = self.new_bt_offsets.cpu().numpy()[:R + 1]
        out["new_bt_offsets"] = nbo
        out["new_bt_blocks"] = self.new_bt_blocks.cpu().numpy()[:int(nbo[R]) if R >= 0 else 0]
        out["new_tt_slots"] = self.new_tt_slots.cpu().numpy()[:T]
        out["freed_blocks"] = self.freed_blocks.cpu().numpy()[:out["num_freed"]]
        out["req_status"] = self.req_status.cpu().numpy()[:R]
        return out

    def gather_logical(self, tt_slots, keep, layer_begin, layer_end, capacity, select=None, stream=None):
        """Returns (out_k, out_v, out_offsets) device tensors; out_* are [layers, capacity, row_elems]."""
        w = self.w
        nl = layer_end - layer_begin
        out_k = torch.zeros((nl, max(1, capacity), w.row_elems), dtype=torch.int16, device=self.device)
        out_v = torch.zeros_like(out_k)
        out_off = torch.full((self.max_requests + 1,), -9, dtype=torch.int32, device=self.device)
        vt.vtoken_gather_logical(self.ctx, num_requests=self.num_requests, tt_offsets=self.tt_offsets,
                                 tt_slots=tt_slots, keep=keep, select=select, layer_begin=layer_begin,
                                 layer_end=layer_end, out_k=out_k, out_v=out_v, out_capacity_tokens=capacity,
                                 out_offsets=out_off, stream=stream)
        return out_k, out_v, out_off

    def close(self):
        if self.ctx:
            torch.cuda.synchronize(self.device)
            vt.vtoken_destroy(self.ctx)
            self.ctx = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass


def origin_map(slots_per_layer: int, move_src: np.ndarray, move_dst: np.ndarray, wave_offsets=None) -> np.ndarray:
    """origin[s] = the slot whose pre-repack bytes slot s must hold after the moves.  With
    ``wave_offsets`` the list holds several waves back to back, applied in order (a later wave may
    copy from, or overwrite, rows an earlier wave has written or read)."""
    origin = np.arange(slots_per_layer, dtype=np.int32)
    if wave_offsets is None:
        wave_offsets = [0, len(move_src)]
    for a, b in zip(wave_offsets[:-1], wave_offsets[1:]):
        origin[move_dst[a:b]] = origin[move_src[a:b]]      # within a wave sources and destinations are disjoint
    return origin
