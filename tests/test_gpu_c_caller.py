"""The C ABI driven from plain C: ``tests/c_abi_driver.c`` is compiled with gcc against
``include/vtoken.h`` and the built library (no Python, no ctypes on that side), runs one repack on the
GPU from a problem file and writes its outputs to a second file, which is compared with the CPU
oracle bit for bit."""
import os
import subprocess

import numpy as np
import pytest

from oracle import vto
from paper_2608_13263_b200 import binding as vt
from harness import workloads as wl

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
CUDA_HOME = os.environ.get("CUDA_HOME", "/usr/local/cuda")
FILL_SEED = 3


def build_driver(tmp_path):
    exe = tmp_path / "c_abi_driver"
    libdir = os.path.dirname(vt.LIB_PATH)
    subprocess.check_call(["gcc", "-std=c99", "-Wall", "-Werror", "-O1", "-I", os.path.join(ROOT, "include"),
                           "-I", os.path.join(CUDA_HOME, "include"), "-o", str(exe),
                           os.path.join(ROOT, "tests", "c_abi_driver.c"),
                           "-L", libdir, "-lvtoken", "-L", os.path.join(CUDA_HOME, "lib64"), "-lcudart",
                           f"-Wl,-rpath,{libdir}", f"-Wl,-rpath,{os.path.join(CUDA_HOME, 'lib64')}"])
    return exe


def write_problem(path, w, k, v, num_free):
    with open(path, "wb") as f:
        np.array([w.num_layers, w.num_blocks, w.block_size, w.num_kv_heads, w.head_dim, w.num_requests, w.num_tokens,
                  len(w.bt_blocks), num_free, w.thr_num, w.thr_den], np.int64).tofile(f)
        w.bt_offsets.astype(np.int32).tofile(f)
        w.bt_blocks.astype(np.int32).tofile(f)
        w.tt_offsets.astype(np.int32).tofile(f)
        w.tt_slots.astype(np.int32).tofile(f)
        keep = np.zeros((w.num_tokens + 3) // 4 * 4, np.uint8)
        keep[:w.num_tokens] = w.keep
        keep.tofile(f)
        w.free_blocks[:num_free].astype(np.int32).tofile(f)
        k.tofile(f)
        v.tofile(f)


def read_result(path, w, k_shape):
    R, T, NBT = w.num_requests, w.num_tokens, len(w.bt_blocks)
    raw = np.fromfile(path, np.uint8)
    pos = 0

    def take(n, dtype):
        nonlocal pos
        nbytes = n * np.dtype(dtype).itemsize
        out = raw[pos:pos + nbytes].view(dtype)
        pos += nbytes
        return out

    counts = take(8, np.int32)
    res = dict(counts=counts, new_bt_offsets=take(R + 1, np.int32), new_bt_blocks=take(NBT, np.int32),
               new_tt_slots=take(T, np.int32), freed_blocks=take(NBT, np.int32), req_status=take(R, np.int32))
    n = int(np.prod(k_shape))
    res["k"] = take(n, np.uint16).reshape(k_shape)
    res["v"] = take(n, np.uint16).reshape(k_shape)
    assert pos == len(raw)
    return res


@pytest.mark.gpu
@pytest.mark.parametrize("recipe,short_pool", [("tiny", False), ("llama_small", False), ("llama_small", True)])
def test_repack_from_a_c_program(tmp_path, recipe, short_pool):
    if recipe == "tiny":
        w = wl.tiny(seed=5)
    else:
        w = wl.llama8b_h2o(seed=2, requests=5, lo=150, hi=500, layers=2, heads=2)
    p_full = vto.plan_workload(w)
    num_free = len(w.free_blocks)
    if short_pool:
        num_free = max(1, int(p_full.num_free_consumed) // 2)        # some requests are deferred
    p = vto.plan_workload(w, num_free=num_free)
    k = np.stack([wl.fill_slab(FILL_SEED, 0, l, w.num_layers, w.slots_per_layer, w.row_elems) for l in range(w.num_layers)])
    v = np.stack([wl.fill_slab(FILL_SEED, 1, l, w.num_layers, w.slots_per_layer, w.row_elems) for l in range(w.num_layers)])
    exe = build_driver(tmp_path)
    src, dst = tmp_path / "problem.bin", tmp_path / "result.bin"
    write_problem(src, w, k, v, num_free)
    done = subprocess.run([str(exe), str(src), str(dst)], capture_output=True, text=True, timeout=300)
    assert done.returncode == 0, done.stderr
    res = read_result(dst, w, k.shape)
    c = res["counts"]
    assert (int(c[0]), int(c[1]), int(c[2]), int(c[3]), int(c[4]), int(c[5])) == (
        p.num_moves, p.num_dst_blocks, p.num_freed, p.num_free_consumed, p.num_admitted, p.num_deferred)
    assert c[6] == 0 and c[7] == 0
    if short_pool:
        assert p.num_deferred > 0
    assert np.array_equal(res["req_status"], p.req_status)
    assert np.array_equal(res["new_bt_offsets"], p.new_bt_offsets)
    assert np.array_equal(res["new_bt_blocks"][:len(p.new_bt_blocks)], p.new_bt_blocks)
    assert (res["new_bt_blocks"][len(p.new_bt_blocks):] == -1).all()          # pre-filled, never written
    assert np.array_equal(res["new_tt_slots"], p.new_tt_slots)
    assert np.array_equal(res["freed_blocks"][:p.num_freed], p.freed_blocks)
    assert (res["freed_blocks"][p.num_freed:] == -1).all()
    vto.apply_moves_pools(k, v, p.move_src, p.move_dst)
    assert np.array_equal(res["k"], k)
    assert np.array_equal(res["v"], v)


def test_c_driver_compiles_and_links_without_a_gpu(tmp_path):
    """The driver builds against the header and the library here too; without arguments it only
    prints its usage (no CUDA call is made)."""
    exe = build_driver(tmp_path)
    done = subprocess.run([str(exe)], capture_output=True, text=True, timeout=60)
    assert done.returncode == 2 and "usage" in done.stderr
