"""ctypes binding of ``libvtoken_harness.so`` (pool fill, whole-pool verifier, decode-read
proxy) -- measurement and test support, not part of the repack path."""
from __future__ import annotations

import ctypes
import os

from paper_2608_13263_b200.binding import _ptr, _stream

_PKG = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_PKG, "libvtoken_harness.so")
SYMBOLS = ["vth_fill", "vth_fill_address", "vth_verify", "vth_decode_read"]

_lib = None


def load():
    global _lib
    if _lib is None:
        from . import build as _build
        try:
            _build._nvcc()
            _build.build()
        except RuntimeError:
            pass                    # no compiler here: use the library as shipped (or fail below)
        if not os.path.exists(LIB_PATH):
            raise ImportError(f"{LIB_PATH} is missing: run `python -m harness.build`")
        lib = ctypes.CDLL(LIB_PATH)
        lib.vth_fill.argtypes = [ctypes.c_void_p, ctypes.c_int, ctypes.c_int, ctypes.c_int, ctypes.c_int,
                                 ctypes.c_int64, ctypes.c_int, ctypes.c_int64, ctypes.c_uint64, ctypes.c_void_p]
        lib.vth_fill_address.argtypes = [ctypes.c_void_p, ctypes.c_int, ctypes.c_int, ctypes.c_int, ctypes.c_int,
                                         ctypes.c_int64, ctypes.c_int, ctypes.c_int64, ctypes.c_void_p]
        lib.vth_verify.argtypes = [ctypes.c_void_p, ctypes.c_int, ctypes.c_int, ctypes.c_int64, ctypes.c_int,
                                   ctypes.c_int64, ctypes.c_uint64, ctypes.c_void_p, ctypes.c_void_p, ctypes.c_void_p]
        lib.vth_decode_read.argtypes = [ctypes.c_void_p, ctypes.c_void_p, ctypes.c_void_p, ctypes.c_void_p,
                                        ctypes.c_void_p, ctypes.c_int32, ctypes.c_int, ctypes.c_int64, ctypes.c_int64,
                                        ctypes.c_void_p, ctypes.c_int, ctypes.c_void_p]
        _lib = lib
    return _lib


def vth_fill(dst, kv, num_layers, layer_begin, layer_end, slots_per_layer, row_elems, seed,
             layer_stride_bytes=0, stream=None) -> None:
    rc = load().vth_fill(_ptr(dst), kv, num_layers, layer_begin, layer_end, slots_per_layer, row_elems,
                         layer_stride_bytes, seed, _stream(stream))
    if rc != 0:
        raise RuntimeError(f"vth_fill failed: {rc}")


def vth_fill_address(dst, kv, num_layers, layer_begin, layer_end, slots_per_layer, row_elems,
                     layer_stride_bytes=0, stream=None) -> None:
    rc = load().vth_fill_address(_ptr(dst), kv, num_layers, layer_begin, layer_end, slots_per_layer, row_elems,
                                 layer_stride_bytes, _stream(stream))
    if rc != 0:
        raise RuntimeError(f"vth_fill_address failed: {rc}")


def vth_verify(pool, kv, num_layers, slots_per_layer, row_elems, seed, origin, mismatches,
               layer_stride_bytes=0, stream=None) -> None:
    rc = load().vth_verify(_ptr(pool), kv, num_layers, slots_per_layer, row_elems, layer_stride_bytes, seed,
                           _ptr(origin), _ptr(mismatches), _stream(stream))
    if rc != 0:
        raise RuntimeError(f"vth_verify failed: {rc}")


def vth_decode_read(k_pool, v_pool, bt_offsets, bt_blocks, bt_owner, total_blocks, num_layers, block_bytes,
                    layer_stride_bytes, checksums, ctas=0, stream=None) -> None:
    rc = load().vth_decode_read(_ptr(k_pool), _ptr(v_pool), _ptr(bt_offsets), _ptr(bt_blocks), _ptr(bt_owner),
                                total_blocks, num_layers, block_bytes, layer_stride_bytes, _ptr(checksums), ctas,
                                _stream(stream))
    if rc != 0:
        raise RuntimeError(f"vth_decode_read failed: {rc}")
