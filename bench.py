#!/usr/bin/env python
"""Benchmark of the repack path (plan + all-layer K/V gather-copy) on B200.

One step = one replay of the CUDA graph that holds the whole hot path (planner kernels and the
copy kernel) on a side stream, over one seeded synthetic workload whose pools are resident
in HBM.  Metric: repack HBM GB/s = 2 * M * token_bytes / t (every moved row read once and
written once, K and V, all layers), M = live tokens of the admitted requests.

    python bench.py                       # 1 GPU: the steady-state serving proxy (512 requests, 137 GiB of
                                          # pools, incremental repack, beside a decode-read proxy), and the
                                          # other four roofline workloads as entries of "configs"
    python bench.py --config mistral7b_random --steps 20 --warmup 3
    python bench.py --gpus N              # one independent pool per rank (weak scaling, no collective);
                                          # starts its own ranks unless a launcher (torchrun) already did
    python bench.py --impl reference      # the CPU oracle timed on the host cores
"""
from __future__ import annotations

import argparse
import json
import os
import socket
import subprocess
import sys
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

from harness import workloads as wl  # noqa: E402

METRIC = "repack HBM GB/s (read+write); live tokens repacked/s and fraction of HBM peak in the same line"
NOMINAL_HBM_GBS = 8000.0
FALLBACK_HBM_GBS = 6650.0
KERNELS_PER_STEP = 4        # plan: tiles, scan, assign; copy: 1
DEFAULT_CONFIG = "steady_state"
# the other roofline workloads, measured after the default one and reported under "configs"
OTHER_CONFIGS = [("llama8b_h2o", 0), ("mistral7b_random", 0), ("longctx_scissor", 0), ("steady_state", 32)]
# launch shapes of the copy kernel tried beside the decode-read proxy: (grid cap, warps per CTA, ring stages)
SWEEP_CTAS = (148, 111, 74, 37, 18)
SWEEP_RINGS = ((8, 6), (8, 4), (8, 3), (4, 3))       # 192, 128, 96, 48 KiB of shared memory per CTA with 4 KiB items


def measured_peak():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(path) as f:
            return float(json.load(f)["hbm_gbs"]), "measured"
    except Exception:
        return FALLBACK_HBM_GBS, "fallback"


def committed_traffic(token_bytes):
    """DRAM bytes per moved token of the copy kernel from the committed ncu capture (taken at
    one token size; traffic is one read and one write per moved row, so it scales with the
    token's bytes), or None."""
    path = os.path.join(ROOT, "profiles", "copy_kernel_dram_traffic.json")
    try:
        with open(path) as f:
            d = json.load(f)
        return d["default"] * token_bytes / d["per_token_bytes_basis"]
    except Exception:
        return None


class ClockSampler:
    """Samples SM clocks and throttle reasons with nvidia-smi while the timed regions run."""
    Q = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
         "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
         "clocks_event_reasons.sw_power_cap")

    def __init__(self, index):
        self.index = index
        self.lines = []
        self.proc = None

    def start(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", f"--query-gpu={self.Q}", "--format=csv,noheader,nounits",
                                          "-lms", "50", "-i", str(self.index)], stdout=subprocess.PIPE, text=True)
            self.thread = threading.Thread(target=self._read, daemon=True)
            self.thread.start()
        except Exception:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.lines.append(line.strip())

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        time.sleep(0.12)
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        sm, mx, power, reasons = [], [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for line in self.lines:
            f = [x.strip() for x in line.split(",")]
            if len(f) < 7:
                continue
            try:
                sm.append(float(f[0]))
                mx.append(float(f[1]))
                power.append(float(f[2]))
            except ValueError:
                continue
            for n, v in zip(names, f[3:7]):
                if v.lower().startswith("active"):
                    reasons.add(n)
        # "under load": samples drawing clearly more than the idle floor of the run
        load = sm
        if power and max(power) > min(power):
            cut = min(power) + 0.25 * (max(power) - min(power))
            load = [s for s, p in zip(sm, power) if p > cut] or sm
        return {"sm_mhz": float(np.median(load)) if load else None, "sm_max_mhz": max(mx) if mx else None,
                "samples": len(sm), "samples_under_load": len(load), "power_w_max": max(power) if power else None,
                "reasons": sorted(reasons)}


def build_workload(name, seed, scale_requests=1.0, block_size=0):
    gen = wl.CONFIGS[name]
    kw = {}
    if block_size:
        kw["block_size"] = block_size
    if scale_requests != 1.0:
        import inspect
        default_r = inspect.signature(gen).parameters["requests"].default
        kw["requests"] = max(1, int(round(default_r * scale_requests)))
    return gen(seed=seed, **kw)


def workload_config(w, args, world, moved_tokens, scale_requests):
    """The `config` object of the JSON line: the workload and nothing specific to an arm, so that the
    CUDA arm and the reference arm describe the same thing with the same keys."""
    bytes_per_step = 2 * moved_tokens * w.token_bytes
    return {"workload": f"{w.name} (seed {args.seed} + rank)", "requests": w.num_requests,
            "layers": w.num_layers, "kv_heads": w.num_kv_heads, "head_dim": w.head_dim,
            "block_size": w.block_size, "num_blocks": w.num_blocks, "row_bytes": w.row_bytes,
            "token_bytes": w.token_bytes, "logical_tokens": w.num_tokens,
            "tokens_moved_per_step": int(moved_tokens), "bytes_moved_per_step": int(bytes_per_step),
            "pool_GiB_per_gpu": 2 * w.pool_bytes / 2 ** 30, "scale_requests": scale_requests,
            "l2": "moved bytes per step exceed the 126 MB L2 (no flush needed)" if bytes_per_step > 4 * 126e6
                  else "moved bytes per step fit in L2: launch-bound parity configuration",
            "plan_mode": args.plan_mode if args.plan_mode == "whole" else
                         "partial: sources = blocks that are not fully live, trigger F > 1/4",
            "parallelism": f"{world} independent pools, no collective"}


def context_stats(w, out):
    """Input statistics plus block counts after the repack (reporting only)."""
    s = wl.stats(w)
    blocks_after = int(out["new_bt_offsets"][w.num_requests])
    kept = s["kept_tokens"]
    s["blocks_after"] = blocks_after
    s["F_after"] = float(1.0 - kept / max(1, blocks_after * w.block_size))
    s["retained_block_reduction_vs_naive_evict"] = float(1.0 - blocks_after / max(1, s["blocks_with_a_kept_token"]))
    s["paper_retained_block_reduction_range_h100_vllm"] = [0.272, 0.723]
    return s


# ----------------------------------------------------------------------------------------------
# the CPU oracle, as it stands, on the host cores (reference arm and cpu_baseline leg)
# ----------------------------------------------------------------------------------------------
def default_oracle_layers(w):
    """Layers of the CPU sample: host pools of 2 * layers slabs must fit host memory comfortably
    (a slab of the steady-state workload is 2.1 GiB, of which the sample touches the moved rows)."""
    return 4 if w.slab_bytes > (1 << 30) else 8


def oracle_sample(w, sample_layers, threads, steps, warmup, fill_seed=1):
    """Times plan + row moves of the oracle on `sample_layers` layers (K and V) of the workload.
    Host pools are slab-sized (the moves use the workload's real slot addresses); the rows the moves
    read hold seeded random 16-bit words drawn with numpy, every other row is untouched zero memory
    (a byte copy's time does not depend on the values).  Returns a dict with per-step seconds."""
    from oracle import vto
    L = min(sample_layers, w.num_layers)
    threads = max(1, min(threads, 2 * L))      # one slab per thread at most
    p = vto.plan_workload(w)
    shape = (L, w.slots_per_layer, w.row_elems)
    rng = np.random.Generator(np.random.PCG64(fill_seed))
    k, v = np.zeros(shape, np.uint16), np.zeros(shape, np.uint16)
    src = np.unique(p.move_src)
    for pool in (k, v):
        for l in range(L):
            for a in range(0, len(src), 65536):
                rows = src[a:a + 65536]
                pool[l, rows] = rng.integers(0, 1 << 16, size=(len(rows), w.row_elems), dtype=np.uint16)
    times = []
    for it in range(warmup + steps):
        t0 = time.perf_counter()
        p = vto.plan_workload(w)
        vto.apply_moves_pools(k, v, p.move_src, p.move_dst, threads=threads)
        dt = time.perf_counter() - t0
        if it >= warmup:
            times.append(dt)
    moved = 2 * p.num_moves * (2 * L * w.row_bytes)
    desc = (f"oracle plan over all {w.num_requests} requests + row moves of layers 0..{L - 1} "
            f"(K and V, {2 * L} of {2 * w.num_layers} slabs), host-resident slab-sized pools with seeded random "
            f"words at the source rows, {threads} OpenMP threads; {steps} timed steps after {warmup} warm-ups")
    return {"times": times, "moved_bytes": moved, "desc": desc, "plan": p, "threads": threads}


def cpu_baseline_leg(w, args, partial_opts, waves=0, steps=12, warmup=2):
    """The CPU-baseline leg of the CUDA arm: the oracle, as it stands, timed on the host cores on a
    bounded sample of the workload.  This is the only place where the CUDA arm executes the oracle;
    the plans it computed on the way are returned so that the device's tables and pools can be
    compared with them at full size."""
    from oracle import vto
    cores = min(os.cpu_count() or 1, vto.openmp_threads())
    layers = args.oracle_layers or default_oracle_layers(w)
    s = oracle_sample(w, layers, cores, steps, warmup)
    s1 = oracle_sample(w, 1, 1, 3, 1)
    p_whole = s["plan"]
    plans = {"whole": p_whole}
    if partial_opts is not None:
        plans["partial"] = vto.plan_partial(w.block_size, w.num_blocks, w.bt_offsets, w.bt_blocks, w.tt_offsets,
                                            w.tt_slots, w.keep, w.free_blocks, w.select, w.thr_num, w.thr_den,
                                            **partial_opts)
    if waves:
        need = np.diff(p_whole.new_bt_offsets)[p_whole.req_status == vto.REPACKED]
        headroom = int(need.max()) if len(need) else 0
        plans["waves"] = vto.plan_waves(w.block_size, w.num_blocks, w.bt_offsets, w.bt_blocks, w.tt_offsets,
                                        w.tt_slots, w.keep, w.free_blocks[:headroom], waves, w.select, w.thr_num,
                                        w.thr_den)
    gbs = lambda sec: s["moved_bytes"] / sec / 1e9
    baseline = {"value": gbs(float(np.median(s["times"]))), "unit": "GB/s", "cores": s["threads"], "kind": "oracle",
                "sample": s["desc"], "value_is": "median over the timed steps",
                "min": gbs(max(s["times"])), "max": gbs(min(s["times"])),
                "single_thread_GBs": s1["moved_bytes"] / float(np.median(s1["times"])) / 1e9}
    return baseline, plans


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    from oracle import vto
    w = build_workload(args.config, args.seed, args.scale_requests, args.block_size)
    cores = min(os.cpu_count() or 1, vto.openmp_threads())
    layers = args.oracle_layers or default_oracle_layers(w)
    s = oracle_sample(w, layers, cores, args.steps, max(2, args.warmup))
    sec = float(np.median(s["times"]))
    gbs = s["moved_bytes"] / sec / 1e9
    p = s["plan"]
    line = {
        "impl": "reference", "metric": METRIC, "value": gbs, "unit": "GB/s", "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": sec * 1e3, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "u8", "data": "synthetic",
        "config": workload_config(w, args, args.gpus, p.num_moves, args.scale_requests),
        "tokens_per_s": s["moved_bytes"] / (2 * w.token_bytes) / sec,
        "cpu_baseline": {"value": gbs, "unit": "GB/s", "cores": s["threads"], "kind": "oracle", "sample": s["desc"],
                         "value_is": "median over the timed steps",
                         "min": s["moved_bytes"] / max(s["times"]) / 1e9, "max": s["moved_bytes"] / min(s["times"]) / 1e9},
        "e2e": {"value": gbs, "unit": "GB/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }
    print(json.dumps(line))


# ----------------------------------------------------------------------------------------------
# CUDA arm
# ----------------------------------------------------------------------------------------------
class Timer:
    """Device timing of graph replays on the side stream, bracketed by a barrier and a device
    synchronisation on both sides."""

    def __init__(self, ranks, dev, side):
        self.ranks, self.dev, self.side = ranks, dev, side

    def __call__(self, graph, steps, warmup, per_launch=False):
        import torch
        side = self.side
        with torch.cuda.stream(side):
            for _ in range(warmup):
                graph.replay()
        side.synchronize()
        self.ranks.barrier()
        torch.cuda.synchronize(self.dev)
        evs = [torch.cuda.Event(enable_timing=True) for _ in range(steps + 1)]
        with torch.cuda.stream(side):
            evs[0].record(side)
            for i in range(steps):
                graph.replay()
                if per_launch or i == steps - 1:
                    evs[i + 1].record(side)
        side.synchronize()
        torch.cuda.synchronize(self.dev)
        self.ranks.barrier()
        total = evs[0].elapsed_time(evs[steps])
        each = [evs[i].elapsed_time(evs[i + 1]) for i in range(steps)] if per_launch else []
        return total, each


def fit_workload(args, name, seed, block_size, scale, dev):
    """The workload at the asked size, or with the request count halved until its pools fit the free
    memory of this (shared) GPU; the scale actually used is reported."""
    import torch
    w = build_workload(name, seed, scale, block_size)
    torch.cuda.empty_cache()
    free_b, _ = torch.cuda.mem_get_info(dev)
    while 2 * w.pool_bytes + (6 << 30) > free_b and w.num_requests > 1:
        scale *= 0.5
        w = build_workload(name, seed, scale, block_size)
    return w, scale


def measure(args, ranks, dev, side, name, block_size, main):
    """One workload through the whole path.  Returns the dict of everything measured; for the main
    workload that is the JSON line (minus keys added by the caller), for the others a summary."""
    import torch

    from harness.device import DeviceProblem, origin_map
    from paper_2608_13263_b200 import binding as vt

    seed = args.seed + ranks.rank
    asked = args.scale_requests if main else 1.0
    w, scale = fit_workload(args, name, seed, block_size, asked, dev)
    steps, warmup = args.steps, args.warmup
    prob = DeviceProblem(w, device=dev, fill_seed=1, copy_variant=args.variant, max_ctas=args.max_ctas,
                         wave_capacity=main and args.waves > 0)
    partial_opts = dict(util=(1, 1), theta=(1, 4))     # fully live blocks stay; the paper's default trigger F > 0.25
    partial = main and args.plan_mode == "partial"

    def do_plan(st, ctx=None):
        if partial:
            prob.plan_partial(stream=st, ctx=ctx, **partial_opts)
        else:
            prob.plan(stream=st, ctx=ctx)

    grid = vt.vtoken_copy_grid(prob.ctx)
    timed = Timer(ranks, dev, side)

    # ---- capture: whole path, the copy alone, the plan alone --------------------------------
    side.wait_stream(torch.cuda.current_stream())
    with torch.cuda.stream(side):
        do_plan(side)
        prob.repack(stream=side)
    side.synchronize()
    g_all, g_copy, g_plan = torch.cuda.CUDAGraph(), torch.cuda.CUDAGraph(), torch.cuda.CUDAGraph()
    with torch.cuda.graph(g_all, stream=side):
        do_plan(torch.cuda.current_stream())
        prob.repack(stream=torch.cuda.current_stream())
    with torch.cuda.graph(g_copy, stream=side):
        prob.repack(stream=torch.cuda.current_stream())
    with torch.cuda.graph(g_plan, stream=side):
        do_plan(torch.cuda.current_stream())
    out = prob.outputs()
    M = out["num_moves"]
    bytes_per_step = 2 * M * w.token_bytes

    total_ms, _ = timed(g_all, steps, warmup)
    copy_total_ms, copy_each = timed(g_copy, steps, warmup, per_launch=True)
    plan_total_ms, _ = timed(g_plan, steps, warmup)

    ms_per_step = ranks.max(total_ms / steps)
    all_bytes = ranks.sum(bytes_per_step)
    all_tokens = ranks.sum(M)
    value = all_bytes / (ms_per_step * 1e-3) / 1e9

    # ---- end to end: host tables in, host tables out, through vtoken_repack_host -----------
    R, T, NBT = w.num_requests, w.num_tokens, len(w.bt_blocks)
    pin = lambda a: torch.from_numpy(np.ascontiguousarray(a)).pin_memory()
    h_in = dict(bt_offsets=pin(w.bt_offsets), bt_blocks=pin(w.bt_blocks), tt_offsets=pin(w.tt_offsets),
                tt_slots=pin(w.tt_slots), keep=pin(w.keep), free_blocks=pin(w.free_blocks))
    if w.select is not None:
        h_in["select"] = pin(w.select)
    h_out = dict(new_bt_offsets=torch.zeros(R + 1, dtype=torch.int32).pin_memory(),
                 new_bt_blocks=torch.zeros(max(1, NBT), dtype=torch.int32).pin_memory(),
                 new_tt_slots=torch.zeros(max(1, T), dtype=torch.int32).pin_memory(),
                 freed_blocks=torch.zeros(max(1, NBT), dtype=torch.int32).pin_memory(),
                 req_status=torch.zeros(max(1, R), dtype=torch.int32).pin_memory())
    h2d = 8 + 2 * 4 * (R + 1) + 4 * NBT + 5 * T + 4 * len(w.free_blocks) + (R if w.select is not None else 0)
    d2h = 4 * (R + 1) + 4 * NBT + 4 * T + 4 * NBT + 4 * R + 32

    def e2e_once():
        if partial:
            return vt.vtoken_repack_host_partial(prob.ctx, num_requests=R, num_free=len(w.free_blocks),
                                                 thr_num=w.thr_num, thr_den=w.thr_den, stream=side, **partial_opts,
                                                 **h_in, **h_out)
        return vt.vtoken_repack_host(prob.ctx, num_requests=R, num_free=len(w.free_blocks), thr_num=w.thr_num,
                                     thr_den=w.thr_den, stream=side, **h_in, **h_out)
    for _ in range(warmup):
        e2e_once()
    ranks.barrier()
    torch.cuda.synchronize(dev)
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    t0 = time.perf_counter()
    e0.record(side)
    for _ in range(steps):
        c_host = e2e_once()
    e1.record(side)
    side.synchronize()
    e2e_wall_ms = (time.perf_counter() - t0) * 1e3 / steps
    e2e_ms = ranks.max(max(e0.elapsed_time(e1) / steps, e2e_wall_ms))
    # bytes the end-to-end call moved (it runs the same planner as the timed graph)
    e2e_bytes = ranks.sum(2 * c_host["num_moves"] * w.token_bytes)
    e2e_value = e2e_bytes / (e2e_ms * 1e-3) / 1e9

    # ---- parity at full size, in the launch configuration that was timed --------------------
    # The oracle is executed in ONE place, the CPU-baseline leg (rank 0, N = 1): it times the oracle
    # as it stands and hands back the plans it computed, which are then compared with the device's.
    parity = "skipped (needs the cpu_baseline leg: N = 1 without --no-cpu-baseline)"
    cpu_baseline, plans = None, None
    if ranks.world == 1 and not args.no_cpu_baseline:
        cpu_baseline, plans = cpu_baseline_leg(w, args, partial_opts if partial else None,
                                               args.waves if main else 0, steps=12 if main else 5)
    if plans is not None and not args.no_verify:
        p = plans["partial"] if partial else plans["whole"]
        ok = (out["error_flags"] == 0 and c_host["error_flags"] == 0 and M == p.num_moves
              and np.array_equal(out["new_tt_slots"], p.new_tt_slots)
              and np.array_equal(out["new_bt_offsets"], p.new_bt_offsets)
              and np.array_equal(out["new_bt_blocks"], p.new_bt_blocks)
              and np.array_equal(out["freed_blocks"], p.freed_blocks)
              and np.array_equal(out["req_status"], p.req_status)
              and c_host["num_moves"] == p.num_moves
              and np.array_equal(h_out["new_tt_slots"].numpy()[:T], p.new_tt_slots)
              and np.array_equal(h_out["new_bt_blocks"].numpy()[:len(p.new_bt_blocks)], p.new_bt_blocks)
              and np.array_equal(h_out["freed_blocks"].numpy()[:p.num_freed], p.freed_blocks))
        bad_words = prob.verify_pools(origin_map(w.slots_per_layer, p.move_src, p.move_dst))
        parity = "ok" if (ok and bad_words == 0) else f"FAILED (tables_ok={ok}, mismatching_words={bad_words})"
    if scale != asked:
        parity += f" (on {w.num_requests} requests: the pools of the full workload did not fit this GPU's free memory)"

    # ---- roofline of the dominant kernel (the copy), timed alone on its stream ---------------
    peak, peak_kind = measured_peak()
    copy_ms = float(np.mean(copy_each))
    achieved = bytes_per_step / (copy_ms * 1e-3) / 1e9
    per_token = committed_traffic(w.token_bytes)
    roofline = {"bound": "hbm", "kernel": "copy_bulk_kernel" if grid["variant"] == 2 else "copy_rows_kernel",
                "achieved": achieved, "peak": peak, "peak_kind": f"of {peak_kind}", "unit": "GB/s",
                "frac": achieved / peak, "frac_of_nominal_8TBs": achieved / NOMINAL_HBM_GBS,
                "algorithmic_bytes_per_launch": bytes_per_step,
                "launch_ms_mean": copy_ms, "launch_ms_median": float(np.median(copy_each)),
                "launch_ms_min": float(np.min(copy_each)),
                "traffic": (per_token * M) if per_token else None}

    res = {
        "value": value, "ms_per_step": ms_per_step, "tokens_per_s": all_tokens / (ms_per_step * 1e-3),
        "config": workload_config(w, args, ranks.world, M, scale),
        "frac_of_measured_hbm_peak": value / (peak * ranks.world),
        "frac_of_nominal_8TBs": value / (NOMINAL_HBM_GBS * ranks.world),
        "plan_us": plan_total_ms / steps * 1e3, "copy_ms": copy_ms,
        "e2e": {"value": e2e_value, "unit": "GB/s", "ms_per_step": e2e_ms, "h2d_bytes_per_step": h2d,
                "d2h_bytes_per_step": d2h,
                "what": ("vtoken_repack_host_partial" if partial else "vtoken_repack_host") +
                        ": pinned host tables -> device, plan, copy, every output table -> host, sync; "
                        "the K/V pools are the GPU-resident cache and stay in HBM"},
        "roofline": roofline, "parity": parity,
        "launch": {"how": "CUDA graph (plan + copy) replayed on a side stream", "copy_grid": grid,
                   "copy_work_distribution": "ticket counter" if grid["variant"] == 2 else "grid-stride rows",
                   "gpu": f"{torch.cuda.get_device_name(dev)} {str(torch.cuda.get_device_properties(dev).uuid)[-12:]}"},
    }
    if cpu_baseline is not None:
        res["cpu_baseline"] = cpu_baseline
    if main:
        res["stats"] = context_stats(w, out)
        # a plain device-to-device copy on this GPU, now (context for run-to-run variation)
        free_now, _ = torch.cuda.mem_get_info(dev)
        if free_now > (6 << 30):
            n = 1 << 30
            src_t = torch.empty(n, dtype=torch.int16, device=dev)
            dst_t = torch.empty(n, dtype=torch.int16, device=dev)
            for _ in range(3):
                dst_t.copy_(src_t)
            best = 1e9
            for _ in range(10):
                c0, c1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                c0.record()
                dst_t.copy_(src_t)
                c1.record()
                c1.synchronize()
                best = min(best, c0.elapsed_time(c1))
            roofline["plain_copy_now_GBs"] = 4 * n / (best * 1e-3) / 1e9     # torch copy_ of 1 Gi 2-byte elements
            roofline["frac_of_plain_copy_now"] = achieved / roofline["plain_copy_now_GBs"]
            del src_t, dst_t
        if ranks.world == 1 and not args.no_proxy and M > 0:
            res["concurrency"] = run_proxy(args, prob, w, side, do_plan, bytes_per_step, dev,
                                           sweep=not args.no_sweep and name == DEFAULT_CONFIG)
        if args.runtime:
            res["runtime"] = run_runtime(args, prob, w, side, dev)
        if args.waves:                # last: it overwrites allocated blocks
            res["waves"] = run_waves(args, prob, w, side, dev, plans, ms_per_step)
    prob.close()
    del prob, g_all, g_copy, g_plan, h_in, h_out
    torch.cuda.empty_cache()
    return res


def run_cuda(args):
    import torch

    from harness.parallel import Ranks

    ranks = Ranks.from_env(args.gpus)
    torch.cuda.set_device(ranks.local_rank)
    dev = torch.device("cuda", ranks.local_rank)
    ranks.init(backend="nccl")
    side = torch.cuda.Stream(device=dev)

    sampler = ClockSampler(ranks.local_rank)
    sampler.start()
    res = measure(args, ranks, dev, side, args.config, args.block_size, main=True)
    others = []
    if (ranks.world == 1 and args.config == DEFAULT_CONFIG and not args.block_size and args.scale_requests == 1.0
            and args.plan_mode == "whole" and not args.no_configs):
        for name, bs in OTHER_CONFIGS:
            try:
                r = measure(args, ranks, dev, side, name, bs, main=False)
                others.append({"workload": r["config"]["workload"], "block_size": r["config"]["block_size"],
                               "requests": r["config"]["requests"],
                               "tokens_moved_per_step": r["config"]["tokens_moved_per_step"],
                               "bytes_moved_per_step": r["config"]["bytes_moved_per_step"],
                               "pool_GiB_per_gpu": r["config"]["pool_GiB_per_gpu"],
                               "value": r["value"], "ms_per_step": r["ms_per_step"], "tokens_per_s": r["tokens_per_s"],
                               "copy_ms": r["copy_ms"], "plan_us": r["plan_us"],
                               "roofline": {k: r["roofline"][k] for k in ("achieved", "peak", "frac", "launch_ms_mean",
                                                                          "algorithmic_bytes_per_launch")},
                               "e2e": r["e2e"]["value"], "parity": r["parity"],
                               "cpu_baseline": r.get("cpu_baseline", {}).get("value")})
            except Exception as e:              # a sub-result must not cost the main line
                others.append({"workload": name, "block_size": bs, "error": f"{type(e).__name__}: {e}"[:300]})
    clocks = sampler.stop()      # sampled over every timed region above

    line = {
        "metric": METRIC, "value": res.pop("value"), "unit": "GB/s", "n_gpus": ranks.world, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": res.pop("ms_per_step"), "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "u8", "data": "synthetic", "config": res.pop("config"),
        "clocks": clocks,
        "gpu_launches": (KERNELS_PER_STEP if args.plan_mode == "whole" else KERNELS_PER_STEP + 2) * args.steps,
        "gpu_launches_what": "kernels of the library inside the timed region of `value` (plan + copy per step)",
    }
    line.update(res)
    if others:
        line["configs"] = others
    if ranks.rank == 0:
        print(json.dumps(line))
    ranks.finalize()


def _stamps(events, origin):
    return [origin.elapsed_time(e) for e in events]


def _rate_inside(stamps, nbytes, lo, hi):
    """GB/s of one stream inside the window [lo, hi] ms (stamps: start of the first launch, then the end
    of every launch): every launch counts with the fraction of its duration that lies inside the window.
    Also returns how many launches lay entirely inside."""
    moved, whole = 0.0, 0
    for a, b in zip(stamps[:-1], stamps[1:]):
        if b <= a:
            continue
        inside = max(0.0, min(b, hi) - max(a, lo))
        moved += nbytes * inside / (b - a)
        whole += int(a >= lo and b <= hi)
    if hi <= lo:
        return None, 0
    return moved / ((hi - lo) * 1e-3) / 1e9, whole


def run_proxy(args, prob, w, side, do_plan, bytes_per_step, dev, sweep):
    """Repack (captured graph, side stream) beside a bandwidth-bound decode-read proxy that reads
    every allocated block through the OLD block tables on a high-priority main stream: each one
    alone, then both at once.  Rates of the concurrent run are taken over the window in which both
    streams were busy.  The proxy's per-request checksums
    must not change (the repack never writes an allocated block).  With `sweep`, the same for a range
    of copy-kernel launch shapes (grid cap x shared-memory ring size)."""
    import torch
    from harness import kernels as vh
    from paper_2608_13263_b200 import binding as vt
    owner = np.repeat(np.arange(w.num_requests, dtype=np.int32), np.diff(w.bt_offsets))
    owner_d = torch.from_numpy(owner).to(dev)
    nbt = len(w.bt_blocks)
    block_bytes = w.block_size * w.row_bytes
    proxy_bytes = nbt * 2 * w.num_layers * block_bytes
    main = torch.cuda.Stream(device=dev, priority=-1)
    sums = torch.zeros(max(1, w.num_requests), dtype=torch.int64, device=dev)
    gbs = lambda nbytes, ms: nbytes / (ms * 1e-3) / 1e9

    def proxy(stream):
        vh.vth_decode_read(prob.k_pool, prob.v_pool, prob.bt_offsets, prob.bt_blocks, owner_d, nbt, w.num_layers,
                           block_bytes, w.slab_bytes, sums, ctas=args.proxy_ctas, stream=stream)

    def ev():
        return torch.cuda.Event(enable_timing=True)

    torch.cuda.synchronize(dev)
    sums.zero_()
    torch.cuda.synchronize(dev)
    proxy(main)
    main.synchronize()
    solo_sums = sums.clone()
    # proxy alone
    n_solo = 4
    a, b = ev(), ev()
    a.record(main)
    for _ in range(n_solo):
        proxy(main)
    b.record(main)
    main.synchronize()
    proxy_alone_ms = a.elapsed_time(b) / n_solo
    proxy_alone = gbs(proxy_bytes, proxy_alone_ms)

    def point(ctx, label):
        """One launch shape: the repack alone, then beside the proxy."""
        with torch.cuda.stream(side):
            do_plan(side, ctx)
            prob.repack(stream=side, ctx=ctx)
        side.synchronize()
        g = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g, stream=side):
            do_plan(torch.cuda.current_stream(), ctx)
            prob.repack(stream=torch.cuda.current_stream(), ctx=ctx)
        a, b = ev(), ev()
        n_alone = 3
        with torch.cuda.stream(side):
            g.replay()
            a.record(side)
            for _ in range(n_alone):
                g.replay()
            b.record(side)
        side.synchronize()
        alone_ms = a.elapsed_time(b) / n_alone
        # both at once, released by one event; the proxy queue is the longer one, so that every repack
        # replay runs beside it
        n_rep = 8
        n_proxy = int(np.ceil((n_rep + 2) * alone_ms * 4.0 / proxy_alone_ms)) + 2
        n_proxy = max(4, min(n_proxy, 80))
        n_proxy += (n_proxy + 1) % 2                      # odd: the XOR checksums then equal the solo values
        sums.zero_()
        torch.cuda.synchronize(dev)
        go = ev()
        pe = [ev() for _ in range(n_proxy + 1)]
        re_ = [ev() for _ in range(n_rep + 1)]
        go.record(torch.cuda.current_stream(dev))
        main.wait_event(go)
        side.wait_event(go)
        pe[0].record(main)
        for i in range(n_proxy):
            proxy(main)
            pe[i + 1].record(main)
            if i == 0:          # the repack joins once the proxy is queued
                with torch.cuda.stream(side):
                    re_[0].record(side)
                    for j in range(n_rep):
                        g.replay()
                        re_[j + 1].record(side)
        torch.cuda.synchronize(dev)
        ps, rs = _stamps(pe, go), _stamps(re_, go)
        lo, hi = max(ps[0], rs[0]), min(ps[-1], rs[-1])
        p_rate, p_n = _rate_inside(ps, proxy_bytes, lo, hi)
        r_rate, r_n = _rate_inside(rs, bytes_per_step, lo, hi)
        ok = bool(torch.equal(sums, solo_sums))
        grid = vt.vtoken_copy_grid(ctx or prob.ctx)
        alone = gbs(bytes_per_step, alone_ms)
        d = {"shape": label, "copy_ctas": grid["ctas"], "copy_smem_KiB": grid["smem_bytes"] / 1024,
             "repack_alone_GBs": alone, "repack_concurrent_GBs": r_rate, "proxy_concurrent_GBs": p_rate,
             "sum_concurrent_GBs": (r_rate + p_rate) if (r_rate and p_rate) else None,
             "repack_share_of_solo": (r_rate / alone) if r_rate else None,
             "proxy_share_of_solo": (p_rate / proxy_alone) if p_rate else None,
             "launches_inside_window": {"proxy": p_n, "repack": r_n}, "proxy_checksum_unchanged": ok}
        del g
        return d

    out = {"proxy_bytes_per_launch": proxy_bytes, "proxy_alone_GBs": proxy_alone,
           "streams": "proxy on a high-priority stream, repack graph on the default-priority side stream",
           "rates": "concurrent rates are taken over the window in which both streams were busy (8 repack replays); a "
                    "launch that straddles an edge of the window counts with the part of its duration inside"}
    out.update(point(None, "as timed above"))
    if sweep:
        pts = []
        rings = SWEEP_RINGS if not args.sweep_rings else [tuple(int(x) for x in r.split("x"))
                                                          for r in args.sweep_rings.split(",")]
        for warps, stages in rings:
            for ctas in (SWEEP_CTAS if not args.sweep_rings else SWEEP_CTAS[:2]):
                ctx = prob.make_ctx(max_ctas=ctas, copy_variant=2, tuning=dict(warps=warps, stages=stages))
                try:
                    pts.append(point(ctx, f"{ctas} CTAs x {warps} warps x {stages} stages"))
                finally:
                    torch.cuda.synchronize(dev)
                    vt.vtoken_destroy(ctx)
        out["sweep"] = pts
    return out


def run_waves(args, prob, w, side, dev, plans, one_shot_ms):
    """The same repack with a pool of the largest single demand instead of the sum of all demands:
    plan + copy + commit in `--waves` waves, blocks reclaimed by one wave feeding the next, one
    captured graph.  Checked against the oracle's wave plan when the CPU-baseline leg ran."""
    import torch
    from harness.device import origin_map
    W = args.waves
    prob.plan()                                            # the one-shot plan names every demand
    one = prob.outputs()
    need = np.diff(one["new_bt_offsets"])[one["req_status"] == 1]
    headroom = int(need.max()) if len(need) else 0
    nf_dev = torch.tensor([headroom], dtype=torch.int32, device=dev)
    prob.repack_waves(W, num_free=nf_dev)                  # allocates the wave buffers outside the capture
    torch.cuda.synchronize(dev)
    g = torch.cuda.CUDAGraph()
    with torch.cuda.graph(g, stream=side):
        prob.repack_waves(W, num_free=nf_dev, stream=torch.cuda.current_stream())
    prob.fill_pools()
    torch.cuda.synchronize(dev)
    with torch.cuda.stream(side):
        g.replay()
    side.synchronize()
    out = prob.waves_outputs(W)
    moved = sum(c["num_moves"] for c in out["wave_counts"])
    parity = "skipped (needs the cpu_baseline leg)"
    if plans is not None and "waves" in plans and not args.no_verify:
        v = plans["waves"]
        ok = (all(c["error_flags"] == 0 for c in out["wave_counts"])
              and [c["num_moves"] for c in out["wave_counts"]] == [c["num_moves"] for c in v.wave_counts]
              and np.array_equal(out["new_tt_slots"], v.new_tt_slots)
              and np.array_equal(out["new_bt_offsets"], v.new_bt_offsets)
              and np.array_equal(out["new_bt_blocks"], v.new_bt_blocks)
              and np.array_equal(out["req_status"], v.req_status) and np.array_equal(out["req_wave"], v.req_wave)
              and np.array_equal(out["req_append_pos"], v.req_append_pos)
              and np.array_equal(out["free_out"], v.free_out))
        bad = prob.verify_pools(origin_map(w.slots_per_layer, v.move_src, v.move_dst, v.wave_move_offsets))
        parity = "ok" if (ok and bad == 0) else f"FAILED (tables_ok={ok}, mismatching_words={bad})"
    # timing: replays read the same source slots and write the same destinations (the inputs are
    # read-only), so every replay moves the same bytes whatever the rows hold by then
    reps = max(3, args.steps)
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    with torch.cuda.stream(side):
        for _ in range(3):
            g.replay()
        e0.record(side)
        for _ in range(reps):
            g.replay()
        e1.record(side)
    side.synchronize()
    ms = e0.elapsed_time(e1) / reps
    return {"waves_enqueued": W, "waves_with_work": sum(1 for c in out["wave_counts"] if c["num_admitted"]),
            "headroom_blocks": headroom, "one_shot_headroom_blocks": one["num_dst_blocks"],
            "headroom_GiB": headroom * w.block_size * w.token_bytes / 2 ** 30,
            "one_shot_headroom_GiB": one["num_dst_blocks"] * w.block_size * w.token_bytes / 2 ** 30,
            "tokens_moved": moved, "one_shot_tokens_moved": one["num_moves"],
            "requests_repacked": int((out["req_status"] == 1).sum()), "one_shot_requests_repacked": one["num_admitted"],
            "moves_per_wave": [c["num_moves"] for c in out["wave_counts"]],
            "ms": ms, "one_shot_ms": one_shot_ms, "GBs": 2 * moved * w.token_bytes / (ms * 1e-3) / 1e9,
            "parity": parity}


def run_runtime(args, prob, w, side, dev):
    """Token-table runtime kernels on this workload's tables: slot mapping over every request,
    one decode step of appends (one token per request), a batch of evictions, and the commit of
    the plan.  Each is captured in its own graph and replayed; reported as microseconds per call
    and as table bytes moved per second (HBM-bound, a few bytes per table entry)."""
    import torch
    from paper_2608_13263_b200 import binding as vt
    R, T = w.num_requests, w.num_tokens
    i32 = dict(dtype=torch.int32, device=dev)
    live = int(((w.tt_slots >= 0) & (w.keep != 0)).sum())
    out_slots = torch.zeros(max(1, T), **i32)
    out_ids = torch.zeros(max(1, T), **i32)
    out_off = torch.zeros(R + 1, **i32)
    # a copy of the tables with one spare entry per request, so that appends have room
    cap_off = (w.tt_offsets.astype(np.int64) + np.arange(R + 1)).astype(np.int32)
    tt_slots2 = np.full(int(cap_off[-1]), -1, np.int32)
    keep2 = np.zeros(int(cap_off[-1]), np.uint8)
    for r in range(R):
        n = w.tt_offsets[r + 1] - w.tt_offsets[r]
        tt_slots2[cap_off[r]:cap_off[r] + n] = w.tt_slots[w.tt_offsets[r]:w.tt_offsets[r + 1]]
        keep2[cap_off[r]:cap_off[r] + n] = w.keep[w.tt_offsets[r]:w.tt_offsets[r + 1]]
    lens = np.diff(w.tt_offsets).astype(np.int32)
    d = lambda a: torch.from_numpy(np.ascontiguousarray(a)).to(dev)
    cap_off_d, tt2, keep2_d = d(cap_off), d(tt_slots2), d(keep2)
    tt_len, new_len = d(lens), d(lens + 1)
    phys = d(np.zeros(R, np.int32))          # position 0 of each block list: always in range
    nv = min(65536, T)
    rng = np.random.default_rng(1)
    vreq = rng.integers(0, R, size=nv).astype(np.int32)
    vtok = (rng.random(nv) * lens[vreq]).astype(np.int32)
    vreq_d, vtok_d, nv_d = d(vreq), d(vtok), d(np.array([nv], np.int32))
    keep_scratch = prob.keep.clone()

    def slot_mapping(st):
        vt.vtoken_build_slot_mapping(prob.ctx, num_requests=prob.num_requests, tt_offsets=prob.tt_offsets,
                                     tt_slots=prob.tt_slots, keep=prob.keep, select=None, out_slots=out_slots,
                                     out_token_ids=out_ids, out_capacity=T, out_offsets=out_off, stream=st)

    def append(st):
        vt.vtoken_sync_new_tokens(prob.ctx, num_requests=prob.num_requests, tt_offsets=cap_off_d, tt_slots=tt2,
                                  keep=keep2_d, tt_len=tt_len, phys_len=phys, bt_offsets=prob.bt_offsets,
                                  bt_blocks=prob.bt_blocks, new_len=new_len, stream=st)

    def evict(st):
        vt.vtoken_evict_tokens(prob.ctx, num_victims=nv_d, max_victims=nv, victim_req=vreq_d, victim_tok=vtok_d,
                               num_requests=prob.num_requests, tt_offsets=prob.tt_offsets, tt_len=tt_len,
                               keep=keep_scratch, stream=st)

    tt_commit = prob.tt_slots.clone()
    keep_commit = prob.keep.clone()

    def commit(st):
        vt.vtoken_apply_moves(prob.ctx, num_requests=prob.num_requests, tt_offsets=prob.tt_offsets,
                              tt_slots=tt_commit, keep=keep_commit, phys_len=phys, new_tt_slots=prob.new_tt_slots,
                              req_status=prob.req_status, new_bt_offsets=prob.new_bt_offsets, stream=st)

    # the two K/V-reading checkers: relocation digest over every layer (read only), logical gather of
    # a layer range that fits in 2 GiB of output per pool (read + write)
    digest_out = torch.zeros(prob.max_requests, dtype=torch.int64, device=dev)
    L = w.num_layers
    g_layers = max(1, min(L, int((2 << 30) // max(1, live * w.row_bytes))))
    gk = torch.empty((g_layers, max(1, live), w.row_elems), dtype=torch.int16, device=dev)
    gv = torch.empty_like(gk)

    def digest(st):
        vt.vtoken_digest_logical(prob.ctx, num_requests=prob.num_requests, tt_offsets=prob.tt_offsets,
                                 tt_slots=prob.tt_slots, keep=prob.keep, select=None, layer_begin=0, layer_end=L,
                                 out_digest=digest_out, stream=st)

    def gather(st):
        vt.vtoken_gather_logical(prob.ctx, num_requests=prob.num_requests, tt_offsets=prob.tt_offsets,
                                 tt_slots=prob.tt_slots, keep=prob.keep, select=None, layer_begin=0,
                                 layer_end=g_layers, out_k=gk, out_v=gv, out_capacity_tokens=max(1, live),
                                 out_offsets=out_off, stream=st)

    # cached slot-translation arrays over the same tables: rebuild of every request (all marked),
    # the append-only refresh after a decode step (the last registered token of every request is new
    # to the cache), and a step in which nothing changed
    c_slots = torch.full((max(1, T),), -1, **i32)
    c_ids = torch.full((max(1, T),), -1, **i32)
    c_len, c_seen = torch.zeros(R, **i32), torch.zeros(R, **i32)
    c_dirty = torch.zeros(R, dtype=torch.uint8, device=dev)
    full_len = d(lens)

    def cache_update(st):
        vt.vtoken_slot_cache_update(prob.ctx, num_requests=prob.num_requests, tt_offsets=prob.tt_offsets,
                                    tt_slots=prob.tt_slots, keep=prob.keep, tt_len=full_len, dirty=c_dirty,
                                    cache_slots=c_slots, cache_ids=c_ids, cache_len=c_len, cache_seen=c_seen, stream=st)

    def cache_rebuild(st):
        c_dirty.fill_(1)
        cache_update(st)

    c_dirty.fill_(1)
    cache_update(torch.cuda.current_stream())
    torch.cuda.synchronize(dev)
    last_live = torch.from_numpy(np.ascontiguousarray(
        ((w.tt_slots >= 0) & (w.keep != 0))[np.maximum(w.tt_offsets[1:] - 1, 0)] & (lens > 0))).to(dev)
    seen_before = torch.clamp(full_len - 1, min=0)
    len_before = c_len - last_live.to(torch.int32)

    def cache_append(st):
        c_seen.copy_(seen_before)
        c_len.copy_(len_before)
        cache_update(st)

    # one decode step of the policy-adapter procedure on the device (the paper's Fig. 6 order:
    # SyncNewTokens, EvictToken for the policy's victims, BuildSlotMapping): every request registers
    # one token and loses one (a policy at its budget), so every cached array is rebuilt
    n2 = int(cap_off[-1])
    step_req = np.arange(R, dtype=np.int32)
    step_tok = (rng.random(R) * np.maximum(lens, 1)).astype(np.int32)
    step_req_d, step_tok_d, step_n_d = d(step_req), d(step_tok), d(np.array([R], np.int32))
    s_slots, s_ids = torch.full((max(1, n2),), -1, **i32), torch.full((max(1, n2),), -1, **i32)
    s_len, s_seen = torch.zeros(R, **i32), torch.zeros(R, **i32)
    s_dirty = torch.ones(R, dtype=torch.uint8, device=dev)
    lens_d = d(lens)
    keep2_start = keep2_d.clone()

    def decode_step(st):
        tt_len.copy_(lens_d)                       # rewind, so that every replay appends and evicts again
        keep2_d.copy_(keep2_start)
        vt.vtoken_sync_new_tokens(prob.ctx, num_requests=prob.num_requests, tt_offsets=cap_off_d, tt_slots=tt2,
                                  keep=keep2_d, tt_len=tt_len, phys_len=phys, bt_offsets=prob.bt_offsets,
                                  bt_blocks=prob.bt_blocks, new_len=new_len, stream=st)
        vt.vtoken_evict_tokens(prob.ctx, num_victims=step_n_d, max_victims=R, victim_req=step_req_d,
                               victim_tok=step_tok_d, num_requests=prob.num_requests, tt_offsets=cap_off_d,
                               tt_len=tt_len, keep=keep2_d, stream=st)
        vt.vtoken_slot_cache_mark(prob.ctx, dirty=s_dirty, num_requests=prob.num_requests, num_victims=step_n_d,
                                  max_victims=R, victim_req=step_req_d, stream=st)
        vt.vtoken_slot_cache_update(prob.ctx, num_requests=prob.num_requests, tt_offsets=cap_off_d, tt_slots=tt2,
                                    keep=keep2_d, tt_len=tt_len, dirty=s_dirty, cache_slots=s_slots, cache_ids=s_ids,
                                    cache_len=s_len, cache_seen=s_seen, stream=st)

    # eligibility metadata (live tokens per block, utilisation histogram, totals behind F) and the
    # input-precondition checker over the same tables
    n_b = torch.zeros(w.num_blocks, **i32)
    hist = torch.zeros(w.block_size + 1, dtype=torch.int64, device=dev)
    summary = torch.zeros(4, dtype=torch.int64, device=dev)
    check_bits = torch.zeros(1, **i32)

    def liveness(st):
        vt.vtoken_block_liveness(prob.ctx, num_requests=prob.num_requests, bt_offsets=prob.bt_offsets,
                                 bt_blocks=prob.bt_blocks, tt_offsets=prob.tt_offsets, tt_slots=prob.tt_slots,
                                 keep=prob.keep, n_b=n_b, hist=hist, summary=summary, stream=st)

    def check(st):
        vt.vtoken_check_tables(prob.ctx, num_requests=prob.num_requests, bt_offsets=prob.bt_offsets,
                               bt_blocks=prob.bt_blocks, tt_offsets=prob.tt_offsets, tt_slots=prob.tt_slots,
                               free_blocks=prob.free_blocks, num_free=prob.num_free, out_bits=check_bits, stream=st)

    NBT = len(w.bt_blocks)
    out = {}
    table_bytes = {"block_liveness": 5 * T + 4 * live + 2 * 4 * w.num_blocks + 2 * 4 * NBT,
                   "check_tables": 4 * T + 2 * 4 * NBT + 4 * len(w.free_blocks) + 2 * 4 * w.num_blocks
                                   + w.slots_per_layer // 8,
                   "decode_step_policy_adapter": 2 * (4 * R + n2) + R * 60 + 5 * n2 + 8 * live,
                   "slot_cache_rebuild_all": 5 * T + 8 * live, "slot_cache_append_one_token_per_request": R * 40,
                   "slot_cache_nothing_changed": R * 13,
                   "slot_mapping": 2 * 5 * T + 8 * live, "append_one_token_per_request": R * (4 * 6 + 5),
                   "evict_64k_victims": nv * (8 + 4 + 4 + 1), "apply_moves": T * (4 + 4 + 1),
                   "digest_all_layers": live * w.token_bytes, "gather_logical": 2 * live * 2 * g_layers * w.row_bytes}
    for name, fn in (("slot_mapping", slot_mapping), ("append_one_token_per_request", append),
                     ("evict_64k_victims", evict), ("apply_moves", commit), ("digest_all_layers", digest),
                     ("gather_logical", gather), ("slot_cache_rebuild_all", cache_rebuild),
                     ("slot_cache_append_one_token_per_request", cache_append),
                     ("slot_cache_nothing_changed", cache_update), ("decode_step_policy_adapter", decode_step),
                     ("block_liveness", liveness), ("check_tables", check)):
        with torch.cuda.stream(side):
            fn(side)
        side.synchronize()
        g = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g, stream=side):
            fn(torch.cuda.current_stream())
        reps = 20
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        with torch.cuda.stream(side):
            for _ in range(3):
                g.replay()
            e0.record(side)
            for _ in range(reps):
                g.replay()
            e1.record(side)
        side.synchronize()
        us = e0.elapsed_time(e1) / reps * 1e3
        out[name] = {"us": us, "table_bytes": table_bytes[name], "GBs": table_bytes[name] / us / 1e3}
    side.synchronize()
    out["check_tables"]["bits"] = int(check_bits.cpu()[0])        # 0: the workload's tables are valid
    out["block_liveness"]["fragmentation_F"] = 1.0 - float(summary[0]) / max(1.0, float(summary[1]) * w.block_size)
    out["entries"] = {"logical_tokens": T, "live_tokens": live, "requests": R, "gather_layers": g_layers}
    out["decode_step_note"] = ("one step for all requests: sync_new_tokens (one token each), evict_tokens (one victim "
                               "each), slot-cache mark + update (every request rebuilt); includes two device copies "
                               "that rewind the tables before every replay")
    out["slot_cache_note"] = ("rebuild_all includes a fill of the marks, append includes two small device copies that "
                              "wind the cache back by one token per request before every replay")
    out["note"] = ("append after the first replay is a no-op per request (tt_len already equals new_len): the figure "
                   "is the launch + per-request check cost of a decode step")
    return out


def run_plan_only(args):
    """Planner latency on the full-size tables of a workload, without its pools: the planner kernels
    read and write tables only, so the context gets a stand-in pool of a few bytes and `vtoken_repack`
    is never called.  Lets the 512-request tables be timed (and profiled) with a few MB on the device.
    Prints one JSON line; parity of both planners is the tests' business, not this mode's."""
    import torch
    from paper_2608_13263_b200 import binding as vt
    from harness.device import DeviceProblem
    dev = torch.device("cuda", 0)
    torch.cuda.set_device(dev)
    w = build_workload(args.config, args.seed, args.scale_requests, args.block_size)
    prob = DeviceProblem(w, device=dev, allocate_pools=False)
    stand_in = torch.zeros(64, dtype=torch.int16, device=dev)
    prob.ctx = vt.vtoken_create(w.num_layers, w.num_blocks, w.block_size, w.num_kv_heads, w.head_dim, stand_in,
                                stand_in, prob.max_requests, prob.max_tokens, prob.max_table_blocks, prob.max_free,
                                elem_bytes=w.elem_bytes)
    side = torch.cuda.Stream(device=dev)
    partial_opts = dict(util=(1, 1), theta=(1, 4))
    # a protect mask over the first quarter of every block table (the place a shared prefix would take), for the
    # latency of the copy-on-write rules: all protected blocks of a request at once / block by block
    import numpy as np
    protect = np.zeros(w.num_blocks, np.uint8)
    for r in range(w.num_requests):
        b0, b1 = int(w.bt_offsets[r]), int(w.bt_offsets[r + 1])
        protect[w.bt_blocks[b0:b0 + (b1 - b0) // 4]] = 1
    protect = torch.from_numpy(protect).to(dev)
    res = {}
    for label, fn in (("whole", lambda st: prob.plan(stream=st)),
                      ("partial", lambda st: prob.plan_partial(stream=st, **partial_opts)),
                      ("partial_protect", lambda st: prob.plan_partial(stream=st, protect=protect, **partial_opts)),
                      ("partial_detach_per_request", lambda st: prob.plan_partial(stream=st, protect=protect, detach=(1, 2),
                                                                                   **partial_opts)),
                      ("partial_detach_per_block", lambda st: prob.plan_partial(stream=st, protect=protect, detach=(1, 2),
                                                                                 detach_rule=1, **partial_opts)),
                      ("partial_detach_all_holders", lambda st: prob.plan_partial(stream=st, protect=protect, detach=(1, 2),
                                                                                   detach_rule=2, **partial_opts))):
        with torch.cuda.stream(side):
            fn(side)
        side.synchronize()
        g = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g, stream=side):
            fn(torch.cuda.current_stream())
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        with torch.cuda.stream(side):
            for _ in range(args.warmup):
                g.replay()
            e0.record(side)
            for _ in range(args.steps):
                g.replay()
            e1.record(side)
        side.synchronize()
        out = prob.outputs()
        res[label] = {"us": e0.elapsed_time(e1) / args.steps * 1e3, "tokens_moved": out["num_moves"],
                      "requests_repacked": out["num_admitted"], "references_released": out["num_released"],
                      "error_flags": out["error_flags"]}
    T = w.num_tokens
    print(json.dumps({"mode": "plan-only", "config": {"workload": f"{w.name} (seed {args.seed})",
                                                      "requests": w.num_requests, "table_entries": T,
                                                      "block_size": w.block_size, "num_blocks": w.num_blocks},
                      "steps": args.steps, "warmup": args.warmup, "table_bytes_per_plan": 13 * T,
                      "planner": res, "gpu": torch.cuda.get_device_name(dev)}))
    prob.close()




def run_prefix_cache(args):
    """The paper's prefix-cache compatibility experiment (Sec. 5, Table 1) in synthetic form, at its
    shape: Llama-3.1-8B-shaped pools, `--groups` prompts each shared by 1 / 2 / 4 / 8 requests, an 8K-token
    shared prefix and an 8K-token private suffix per request, an H2O-style mask that keeps a fifth.
    Per sharing degree: the conservative plan (shared blocks stay, private suffixes are repacked) and the
    copy-on-write plan that judges a shared block by all its holders' live tokens (threshold 1/1), each as
    one captured graph of plan + copy on the side stream, checked against the oracle (tables in full,
    every word of both pools through the oracle's move list), then timed.  One JSON line."""
    import torch
    from harness import workloads as wl
    from harness.device import DeviceProblem, origin_map
    sys.path.insert(0, ROOT)
    from oracle import vto
    dev = torch.device("cuda", 0)
    torch.cuda.set_device(dev)
    side = torch.cuda.Stream(device=dev)
    rows = []
    for degree in (1, 2, 4, 8):
        R = args.groups * degree
        w, protect = wl.shared_prefix(seed=args.seed, groups=args.groups, degree=degree, prefix_len=8192,
                                      suffix_len=8192, extra_free=R * 8192 // 16 // 4)
        free_b, total_b = torch.cuda.mem_get_info(dev)
        need = 2 * w.num_layers * w.slots_per_layer * w.row_bytes
        if need > free_b - (6 << 30):
            rows.append({"degree": degree, "skipped": f"pools of {need / 2 ** 30:.1f} GiB do not fit the free memory"})
            continue
        prob = DeviceProblem(w, device=dev)
        prot = torch.from_numpy(protect).to(dev)
        blocks_before = len(set(w.bt_blocks.tolist()))
        entry = {"degree": degree, "requests": R, "logical_tokens": int(w.num_tokens),
                 "blocks_allocated": blocks_before, "shared_blocks": int(protect.sum()),
                 "pool_GiB": need / 2 ** 30, "plans": {}}
        for label, opts in (("conservative", dict(util=(1, 1))),
                            ("copy_on_write_all_holders", dict(util=(1, 1), detach=(1, 1), detach_rule=2))):
            with torch.cuda.stream(side):
                prob.plan_partial(protect=prot, stream=side, **opts)
                prob.repack(stream=side)
            side.synchronize()
            g = torch.cuda.CUDAGraph()
            with torch.cuda.graph(g, stream=side):
                prob.plan_partial(protect=prot, stream=torch.cuda.current_stream(), **opts)
                prob.repack(stream=torch.cuda.current_stream())
            prob.fill_pools()
            torch.cuda.synchronize(dev)
            with torch.cuda.stream(side):
                g.replay()
            side.synchronize()
            out = prob.outputs()
            parity = "skipped"
            if not args.no_verify:
                p = vto.plan_partial(w.block_size, w.num_blocks, w.bt_offsets, w.bt_blocks, w.tt_offsets, w.tt_slots,
                                     w.keep, w.free_blocks, protect=protect, **opts)
                ok = (out["error_flags"] == 0 and all(np.array_equal(out[k], getattr(p, k)) for k in
                      ("new_bt_offsets", "new_bt_blocks", "new_tt_slots", "freed_blocks", "released_blocks", "req_status")))
                bad = prob.verify_pools(origin_map(w.slots_per_layer, p.move_src, p.move_dst))
                parity = "ok" if ok and bad == 0 else f"FAILED (tables_ok={ok}, mismatching_words={bad})"
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            with torch.cuda.stream(side):
                for _ in range(args.warmup):
                    g.replay()
                e0.record(side)
                for _ in range(args.steps):
                    g.replay()
                e1.record(side)
            side.synchronize()
            ms = e0.elapsed_time(e1) / args.steps
            moved = out["num_moves"]
            after = len(set(out["new_bt_blocks"].tolist()))
            entry["plans"][label] = {
                "blocks_retained": after, "retained_block_reduction": 1 - after / blocks_before,
                "tokens_moved": moved, "references_released": out["num_released"],
                "requests_repacked": out["num_admitted"], "ms_plan_and_copy": ms,
                "GBs": 2 * moved * w.token_bytes / (ms * 1e-3) / 1e9 if ms > 0 else 0.0, "parity": parity}
        rows.append(entry)
        prob.close()
        del prob
        torch.cuda.empty_cache()
    print(json.dumps({"mode": "prefix-cache", "shape": "L=32, H=8, D=128, S=16; 8192 shared + 8192 private tokens per request, H2O-style mask keeping 20 %",
                      "groups": args.groups, "steps": args.steps, "warmup": args.warmup, "degrees": rows,
                      "gpu": torch.cuda.get_device_name(dev)}))


# ----------------------------------------------------------------------------------------------
# N > 1 without a launcher: this process starts one rank per GPU itself
# ----------------------------------------------------------------------------------------------
def free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def spawn_ranks(n):
    """`python bench.py --gpus N` with no launcher around it (WORLD_SIZE unset): start N copies of this
    command, one rank per GPU, rendezvous on 127.0.0.1 at a free port.  Rank 0 prints the JSON line
    (its output passes straight through); the exit code is the worst of the ranks'."""
    port = free_port()
    procs = []
    for rank in range(n):
        env = dict(os.environ, RANK=str(rank), LOCAL_RANK=str(rank), WORLD_SIZE=str(n), MASTER_ADDR="127.0.0.1",
                   MASTER_PORT=str(port))
        env.setdefault("NCCL_DEBUG", "WARN")          # keeps NCCL's communicator messages on stderr
        procs.append(subprocess.Popen([sys.executable, os.path.abspath(__file__), *sys.argv[1:]], env=env))
    rc = 0
    try:
        for p in procs:
            r = p.wait()
            rc = rc or r
    except BaseException:
        for p in procs:
            if p.poll() is None:
                p.terminate()
        raise
    return rc


def run_plumbing_check(args):
    """The multi-rank plumbing of the CUDA arm without a GPU: launch (or self-spawn), rendezvous over
    gloo, barrier, max-over-ranks time, sum-over-ranks work, one JSON line from rank 0.  No kernel
    runs and nothing is measured: each rank's "work" is the size of its own seeded workload's tables
    and its "time" a fixed figure that differs by rank, so that the reductions can be checked from
    outside.  The line says what it is (`data`: "plumbing-check")."""
    from harness.parallel import Ranks
    ranks = Ranks.from_env(args.gpus)
    ranks.init(backend="gloo")
    w = build_workload("tiny", args.seed + ranks.rank)
    units = float(w.num_tokens)                 # input size only: no method arithmetic outside the library
    seconds = 1.0 + ranks.rank
    ranks.barrier()
    total_units, slowest = ranks.sum(units), ranks.max(seconds)
    line = {"metric": METRIC, "value": total_units / slowest, "unit": "table entries/s (fabricated)", "n_gpus": ranks.world,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": slowest * 1e3, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "u8", "data": "plumbing-check",
            "config": {"workload": "tiny (seed + rank)", "parallelism": f"{ranks.world} independent pools, no collective"},
            "units_all_ranks": total_units, "slowest_rank_s": slowest, "rank_units": units}
    if ranks.rank == 0:
        print(json.dumps(line), flush=True)
    ranks.finalize()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="cuda", choices=["cuda", "reference"])
    ap.add_argument("--config", default=DEFAULT_CONFIG, choices=sorted(wl.CONFIGS))
    ap.add_argument("--seed", type=int, default=0)
    ap.add_argument("--variant", type=int, default=0, help="copy path: 0 auto, 1 registers, 2 bulk copy")
    ap.add_argument("--max-ctas", type=int, default=0)
    ap.add_argument("--scale-requests", type=float, default=1.0)
    ap.add_argument("--prefix-cache", action="store_true",
                    help="the prefix-cache experiment in synthetic form: sharing degrees 1-8, conservative and copy-on-write plans")
    ap.add_argument("--groups", type=int, default=4, help="--prefix-cache: number of shared prompts")
    ap.add_argument("--oracle-layers", type=int, default=0,
                    help="layers in the CPU-baseline sample (0: 8, or 4 when a slab exceeds 1 GiB)")
    ap.add_argument("--no-proxy", action="store_true", help="skip the run beside the decode-read proxy")
    ap.add_argument("--no-sweep", action="store_true", help="skip the sweep of copy-kernel launch shapes beside the proxy")
    ap.add_argument("--sweep-rings", default="", help="ring shapes of the sweep as warps x stages, e.g. 8x4,12x3 "
                    "(default: 8x6, 8x4, 8x3, 4x3 = 192, 128, 96, 48 KiB per CTA); with this flag only the two largest grids are tried")
    ap.add_argument("--no-configs", action="store_true", help="skip the other roofline workloads (`configs`)")
    ap.add_argument("--proxy-ctas", type=int, default=0)
    ap.add_argument("--runtime", action="store_true", help="also time the token-table runtime kernels")
    ap.add_argument("--plan-mode", default="whole", choices=["whole", "partial"],
                    help="whole-request compaction (default) or the partial planner that keeps fully live blocks")
    ap.add_argument("--waves", type=int, default=0,
                    help="also run the repack in this many waves with the headroom of the largest single demand")
    ap.add_argument("--block-size", type=int, default=0, help="override the workload's block size")
    ap.add_argument("--no-verify", action="store_true")
    ap.add_argument("--plan-only", action="store_true",
                    help="time the planners alone on the workload's tables (no pools are allocated)")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--plumbing-check", action="store_true",
                    help="no GPU: exercise launch, rendezvous (gloo) and the reductions of the N-rank path only")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3) if args.impl == "cuda" else args.warmup
    if args.gpus > 1 and "WORLD_SIZE" not in os.environ and (args.impl == "cuda" or args.plumbing_check):
        sys.exit(spawn_ranks(args.gpus))
    if args.plumbing_check:
        run_plumbing_check(args)
    elif args.impl == "reference":
        run_reference(args)
    elif args.plan_only:
        run_plan_only(args)
    elif args.prefix_cache:
        run_prefix_cache(args)
    else:
        run_cuda(args)


if __name__ == "__main__":
    main()
