"""The N > 1 plumbing of the benchmark on CPU: two gloo ranks, one independent problem per
rank, timing reduced by max and work by sum; both ranks plan with the oracle standing in for
the device (host logic only) and must report the same whole-job figure."""
import os
import socket
import sys

import numpy as np
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _worker(rank, world, port, q):
    sys.path.insert(0, ROOT)
    os.environ.update(RANK=str(rank), LOCAL_RANK=str(rank), WORLD_SIZE=str(world), MASTER_ADDR="127.0.0.1",
                      MASTER_PORT=str(port))
    from oracle import vto
    from harness import workloads as wl
    from harness.parallel import Ranks, job_throughput
    ranks = Ranks.from_env(world)
    ranks.init(backend="gloo")
    # per-rank seed -> different problems, as in the benchmark
    w = wl.mistral7b_random(seed=rank, requests=6, lo=50, hi=200, layers=1, heads=1, head_dim=8)
    p = vto.plan_workload(w)
    units = 2 * p.num_moves * w.token_bytes
    seconds = 0.5 + rank            # rank 1 is the slow one
    ranks.barrier()
    thr = job_throughput(ranks, units, seconds)
    q.put((rank, units, thr, ranks.max(seconds), ranks.sum(1)))
    ranks.finalize()


def test_two_rank_weak_scaling_aggregation():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        port = s.getsockname()[1]
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    procs = [ctx.Process(target=_worker, args=(r, 2, port, q)) for r in range(2)]
    for p in procs:
        p.start()
    res = sorted(q.get(timeout=120) for _ in range(2))
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    (r0, u0, t0, m0, s0), (r1, u1, t1, m1, s1) = res
    assert u0 != u1                               # independent problems
    assert m0 == m1 == 1.5 and s0 == s1 == 2      # max over ranks, sum over ranks
    assert np.isclose(t0, (u0 + u1) / 1.5) and np.isclose(t1, t0)


def test_world_size_mismatch_is_an_error():
    sys.path.insert(0, ROOT)
    from harness.parallel import Ranks
    os.environ.pop("WORLD_SIZE", None)
    os.environ.pop("RANK", None)
    try:
        Ranks.from_env(2)
    except RuntimeError as e:
        assert "torchrun" in str(e)
    else:
        raise AssertionError("expected an error")
    r = Ranks.from_env(1)
    assert r.world == 1 and r.max(3.0) == 3.0 and r.sum(2) == 2.0


def test_bench_starts_its_own_ranks_and_prints_one_line():
    """`python bench.py --gpus 2` without a launcher: the command starts two ranks itself (free port on
    127.0.0.1), they meet over gloo, and rank 0 prints ONE line with n_gpus 2, weak scaling, the sum of
    the ranks' work divided by the slowest rank's time.  (The plumbing check runs no kernel; its
    per-rank figures are fabricated so that the reductions can be verified here.)"""
    import json
    import subprocess
    from harness import workloads as wl
    env = {k: v for k, v in os.environ.items() if k not in ("RANK", "LOCAL_RANK", "WORLD_SIZE", "MASTER_PORT")}
    out = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--gpus", "2", "--plumbing-check",
                          "--steps", "4", "--warmup", "3"], cwd=ROOT, env=env, capture_output=True, text=True,
                         timeout=300)
    assert out.returncode == 0, out.stderr[-2000:]
    lines = [l for l in out.stdout.splitlines() if l.startswith("{")]
    assert len(lines) == 1
    d = json.loads(lines[0])
    assert d["n_gpus"] == 2 and d["scaling"] == "weak" and d["steps"] == 4 and d["data"] == "plumbing-check"
    units = [float(wl.tiny(seed=r).num_tokens) for r in range(2)]
    assert units[0] != units[1]
    assert d["units_all_ranks"] == sum(units) and d["slowest_rank_s"] == 2.0
    assert np.isclose(d["value"], sum(units) / 2.0) and d["ms_per_step"] == 2000.0


def test_bench_under_a_launcher_does_not_spawn():
    """With WORLD_SIZE set (torchrun did the launch) every rank runs in place: rank 1 prints nothing."""
    import subprocess
    import socket as sk
    with sk.socket() as s:
        s.bind(("127.0.0.1", 0))
        port = s.getsockname()[1]
    procs = []
    for rank in range(2):
        env = dict(os.environ, RANK=str(rank), LOCAL_RANK=str(rank), WORLD_SIZE="2", MASTER_ADDR="127.0.0.1",
                   MASTER_PORT=str(port))
        procs.append(subprocess.Popen([sys.executable, os.path.join(ROOT, "bench.py"), "--gpus", "2",
                                       "--plumbing-check"], cwd=ROOT, env=env, stdout=subprocess.PIPE,
                                      stderr=subprocess.PIPE, text=True))
    outs = [p.communicate(timeout=300) for p in procs]
    assert all(p.returncode == 0 for p in procs), outs
    assert len([l for l in outs[0][0].splitlines() if l.startswith("{")]) == 1
    assert [l for l in outs[1][0].splitlines() if l.startswith("{")] == []
