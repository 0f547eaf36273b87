"""The C-ABI libraries load without a GPU and export every symbol the headers declare."""
import ctypes
import os
import re

from harness import build as harness_build
from harness import kernels as harness
from paper_2608_13263_b200 import binding, build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def declared_functions(header):
    text = open(header).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(vtoken_[a-z_]+)\s*\(", text)))


def test_library_exports_every_declared_symbol():
    build.build()
    lib = ctypes.CDLL(binding.LIB_PATH)
    names = declared_functions(os.path.join(ROOT, "include", "vtoken.h"))
    assert "vtoken_plan" in names and "vtoken_repack" in names and "vtoken_gather_logical" in names
    for n in names:
        assert hasattr(lib, n), n
    # the binding carries the same names
    assert sorted(binding.SYMBOLS) == [n for n in names]
    for n in names:
        assert hasattr(binding, n) or n in ("vtoken_strerror", "vtoken_last_cuda_error"), n


def test_harness_library_loads():
    harness_build.build()
    lib = ctypes.CDLL(harness.LIB_PATH)
    for n in harness.SYMBOLS:
        assert hasattr(lib, n), n


def test_strerror_and_argument_errors_without_gpu():
    assert binding.strerror(0) == "ok"
    assert "capacity" in binding.strerror(binding.ECAPACITY)
    lib = binding.load()
    # NULL arguments are rejected before any CUDA call
    assert lib.vtoken_create(None, None) == binding.EINVAL
    assert lib.vtoken_repack(None, None) == binding.EINVAL
    cfg = binding.Config(1, 4, 16, 1, 4, 2, 256, 512, 0, 1, 16, 4, 4)   # row_bytes = 8: not a multiple of 16
    ctx = ctypes.c_void_p()
    assert lib.vtoken_create(ctypes.byref(cfg), ctypes.byref(ctx)) == binding.EINVAL
    cfg = binding.Config(1, 4, 16, 1, 8, 2, 257, 512, 0, 1, 16, 4, 4)   # misaligned pool
    assert lib.vtoken_create(ctypes.byref(cfg), ctypes.byref(ctx)) == binding.EINVAL


def test_header_is_plain_c_and_ctypes_layouts_match(tmp_path):
    """include/vtoken.h compiles as C99 on its own, and every struct the binding mirrors with
    ctypes has the size and field offsets the C compiler gives it."""
    import subprocess
    structs = {"vtoken_config": binding.Config, "vtoken_plan_in": binding.PlanIn, "vtoken_counts": binding.Counts,
               "vtoken_plan_out": binding.PlanOut, "vtoken_partial_opts": binding.PartialOpts,
               "vtoken_host_tables": binding.HostTables, "vtoken_waves_out": binding.WavesOut,
               "vtoken_copy_tuning": binding.CopyTuning}
    lines = ['#include <stddef.h>', '#include <stdio.h>', '#include "vtoken.h"', 'int main(void) {']
    for cname, cls in structs.items():
        lines.append(f'printf("{cname} %zu", sizeof({cname}));')
        for fname, _ in cls._fields_:
            lines.append(f'printf(" %zu", offsetof({cname}, {fname}));')
        lines.append('printf("\\n");')
    lines += ['return 0; }']
    src = tmp_path / "layout.c"
    src.write_text("\n".join(lines))
    exe = tmp_path / "layout"
    subprocess.check_call(["gcc", "-std=c99", "-pedantic", "-Wall", "-Werror", "-I", os.path.join(ROOT, "include"),
                           "-o", str(exe), str(src)])
    out = subprocess.check_output([str(exe)], text=True).strip().splitlines()
    assert len(out) == len(structs)
    for line, (cname, cls) in zip(out, structs.items()):
        parts = line.split()
        assert parts[0] == cname
        assert int(parts[1]) == ctypes.sizeof(cls), cname
        offsets = [getattr(cls, f).offset for f, _ in cls._fields_]
        assert [int(x) for x in parts[2:]] == offsets, cname
