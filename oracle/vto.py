"""ctypes front end of the CPU oracle (``vtoken_oracle.c``).  TEST INFRASTRUCTURE ONLY.

Only the tests, the smoke check and the benchmark's CPU-baseline leg may import this
module; the product package never does.  It builds ``libvto.so`` with gcc on first use
(plain C, ``-O2``, OpenMP only for the slab loop of ``apply_moves_pools``).
"""
from __future__ import annotations

import ctypes
import dataclasses
import os
import subprocess
from typing import Optional

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "vtoken_oracle.c")
_HDR = os.path.join(_HERE, "vtoken_oracle.h")
_LIB = os.path.join(_HERE, "libvto.so")

NOT_SELECTED, REPACKED, NO_GAIN, DEFERRED_NO_FREE = 0, 1, 2, 3


def build(force: bool = False) -> str:
    """Compile the oracle into ``oracle/libvto.so`` when missing or older than its sources."""
    stale = (not os.path.exists(_LIB)
             or os.path.getmtime(_LIB) < max(os.path.getmtime(_SRC), os.path.getmtime(_HDR)))
    if force or stale:
        tmp = _LIB + f".{os.getpid()}.tmp"
        subprocess.check_call(["gcc", "-std=c99", "-O2", "-fPIC", "-shared", "-fopenmp",
                               "-Wall", "-Wextra", "-o", tmp, _SRC])
        os.replace(tmp, _LIB)
    return _LIB


class _Counts(ctypes.Structure):
    _fields_ = [(n, ctypes.c_int32) for n in
                ("num_moves", "num_dst_blocks", "num_freed", "num_free_consumed",
                 "num_admitted", "num_deferred", "num_released")]


_lib = None


def lib():
    global _lib
    if _lib is None:
        _lib = ctypes.CDLL(build())
        _lib.vto_gather_logical.restype = ctypes.c_int64
        _lib.vto_build_slot_mapping.restype = ctypes.c_int64
        _lib.vto_waste_ratio.restype = ctypes.c_double
    return _lib


def _p(a: Optional[np.ndarray], dtype):
    if a is None:
        return None
    assert a.dtype == dtype and a.flags["C_CONTIGUOUS"], (a.dtype, dtype)
    return a.ctypes.data_as(ctypes.c_void_p)


def _i32(a):
    return np.ascontiguousarray(a, dtype=np.int32)


def _u8(a):
    return None if a is None else np.ascontiguousarray(a, dtype=np.uint8)


@dataclasses.dataclass
class Plan:
    new_bt_offsets: np.ndarray
    new_bt_blocks: np.ndarray     # trimmed to new_bt_offsets[R]
    new_tt_slots: np.ndarray
    freed_blocks: np.ndarray      # trimmed to num_freed
    req_status: np.ndarray
    move_src: np.ndarray          # trimmed to num_moves
    move_dst: np.ndarray
    num_moves: int
    num_dst_blocks: int
    num_freed: int
    num_free_consumed: int
    num_admitted: int
    num_deferred: int
    released_blocks: np.ndarray = None    # references to shared blocks dropped by a copy-on-write detach


def plan(S, bt_offsets, bt_blocks, tt_offsets, tt_slots, keep, free_blocks,
         select=None, thr_num=0, thr_den=0, num_free=None) -> Plan:
    bt_offsets, bt_blocks = _i32(bt_offsets), _i32(bt_blocks)
    tt_offsets, tt_slots = _i32(tt_offsets), _i32(tt_slots)
    keep, select, free_blocks = _u8(keep), _u8(select), _i32(free_blocks)
    R = len(tt_offsets) - 1
    T = int(tt_offsets[-1])
    nbt = int(bt_offsets[-1])
    if num_free is None:
        num_free = len(free_blocks)
    new_bt_offsets = np.zeros(R + 1, np.int32)
    new_bt_blocks = np.full(max(nbt, 1), -7, np.int32)
    new_tt_slots = np.full(max(T, 1), -7, np.int32)
    freed = np.full(max(nbt, 1), -7, np.int32)
    status = np.full(max(R, 1), -7, np.int32)
    msrc = np.full(max(T, 1), -7, np.int32)
    mdst = np.full(max(T, 1), -7, np.int32)
    c = _Counts()
    rc = lib().vto_plan(ctypes.c_int32(R), ctypes.c_int32(S),
                        _p(bt_offsets, np.int32), _p(bt_blocks, np.int32),
                        _p(tt_offsets, np.int32), _p(tt_slots, np.int32), _p(keep, np.uint8),
                        _p(select, np.uint8), ctypes.c_uint32(thr_num), ctypes.c_uint32(thr_den),
                        _p(free_blocks, np.int32), ctypes.c_int32(num_free),
                        _p(new_bt_offsets, np.int32), _p(new_bt_blocks, np.int32),
                        _p(new_tt_slots, np.int32), _p(freed, np.int32), _p(status, np.int32),
                        _p(msrc, np.int32), _p(mdst, np.int32), ctypes.byref(c))
    if rc != 0:
        raise ValueError(f"vto_plan failed: {rc}")
    return Plan(new_bt_offsets, new_bt_blocks[:int(new_bt_offsets[R])].copy(), new_tt_slots[:T].copy(),
                freed[:c.num_freed].copy(), status[:R].copy(),
                msrc[:c.num_moves].copy(), mdst[:c.num_moves].copy(),
                c.num_moves, c.num_dst_blocks, c.num_freed, c.num_free_consumed,
                c.num_admitted, c.num_deferred)


def plan_workload(w, num_free=None) -> Plan:
    return plan(w.block_size, w.bt_offsets, w.bt_blocks, w.tt_offsets, w.tt_slots, w.keep,
                w.free_blocks, w.select, w.thr_num, w.thr_den, num_free)


def apply_moves_slab(slab: np.ndarray, move_src, move_dst) -> None:
    """In place on one slab: a C-contiguous 2-D array [num_slots, row] of any dtype."""
    assert slab.ndim == 2 and slab.flags["C_CONTIGUOUS"]
    move_src, move_dst = _i32(move_src), _i32(move_dst)
    rc = lib().vto_apply_moves_slab(ctypes.c_void_p(slab.ctypes.data), ctypes.c_int64(slab.shape[0]),
                                    ctypes.c_int64(slab.shape[1] * slab.itemsize),
                                    _p(move_src, np.int32), _p(move_dst, np.int32),
                                    ctypes.c_int32(len(move_src)))
    if rc != 0:
        raise ValueError(f"vto_apply_moves_slab failed: {rc}")


def apply_moves_pools(k_pool: np.ndarray, v_pool: np.ndarray, move_src, move_dst, threads: int = 1) -> None:
    """In place on K and V pools shaped [L, num_slots, row] (C-contiguous)."""
    assert k_pool.ndim == 3 and k_pool.shape == v_pool.shape
    assert k_pool.flags["C_CONTIGUOUS"] and v_pool.flags["C_CONTIGUOUS"]
    move_src, move_dst = _i32(move_src), _i32(move_dst)
    L, ns, row = k_pool.shape
    rc = lib().vto_apply_moves_pools(ctypes.c_void_p(k_pool.ctypes.data), ctypes.c_void_p(v_pool.ctypes.data),
                                     ctypes.c_int32(L), ctypes.c_int64(0), ctypes.c_int64(ns),
                                     ctypes.c_int64(row * k_pool.itemsize),
                                     _p(move_src, np.int32), _p(move_dst, np.int32),
                                     ctypes.c_int32(len(move_src)), ctypes.c_int32(threads))
    if rc != 0:
        raise ValueError(f"vto_apply_moves_pools failed: {rc}")


def gather_logical(slab: np.ndarray, tt_slots, keep=None) -> np.ndarray:
    """Rows of one request's active tokens in token-id order from one slab [num_slots, row]."""
    assert slab.ndim == 2 and slab.flags["C_CONTIGUOUS"]
    tt_slots, keep = _i32(tt_slots), _u8(keep)
    out = np.empty((max(len(tt_slots), 1), slab.shape[1]), slab.dtype)
    n = lib().vto_gather_logical(ctypes.c_void_p(slab.ctypes.data), ctypes.c_int64(slab.shape[0]),
                                 ctypes.c_int64(slab.shape[1] * slab.itemsize),
                                 _p(tt_slots, np.int32), _p(keep, np.uint8), ctypes.c_int32(len(tt_slots)),
                                 ctypes.c_void_p(out.ctypes.data), ctypes.c_int64(out.shape[0]))
    if n < 0:
        raise ValueError(f"vto_gather_logical failed: {n}")
    return out[:n].copy()


def validate(S, NB, bt_offsets, bt_blocks, tt_offsets, tt_slots, keep, free_blocks) -> int:
    """0 when the input preconditions hold, else the code of the first failed check."""
    bt_offsets, bt_blocks = _i32(bt_offsets), _i32(bt_blocks)
    tt_offsets, tt_slots = _i32(tt_offsets), _i32(tt_slots)
    keep, free_blocks = _u8(keep), _i32(free_blocks)
    bad = ctypes.c_int32(0)
    rc = lib().vto_validate(ctypes.c_int32(len(tt_offsets) - 1), ctypes.c_int32(S), ctypes.c_int32(NB),
                            _p(bt_offsets, np.int32), _p(bt_blocks, np.int32),
                            _p(tt_offsets, np.int32), _p(tt_slots, np.int32), _p(keep, np.uint8),
                            _p(free_blocks, np.int32), ctypes.c_int32(len(free_blocks)), ctypes.byref(bad))
    if rc == -1:
        raise ValueError("vto_validate: bad argument")
    return bad.value


def check_tables(S, NB, bt_offsets, bt_blocks, tt_offsets, tt_slots, free_blocks, protect=None) -> int:
    """Bit set of every violated input precondition (0 = valid); see vto_check_tables."""
    bt_offsets, bt_blocks = _i32(bt_offsets), _i32(bt_blocks)
    tt_offsets, tt_slots, free_blocks, protect = _i32(tt_offsets), _i32(tt_slots), _i32(free_blocks), _u8(protect)
    bits = ctypes.c_uint32(0)
    rc = lib().vto_check_tables(ctypes.c_int32(len(tt_offsets) - 1), ctypes.c_int32(S), ctypes.c_int32(NB),
                                _p(bt_offsets, np.int32), _p(bt_blocks, np.int32), _p(tt_offsets, np.int32),
                                _p(tt_slots, np.int32), _p(free_blocks, np.int32), ctypes.c_int32(len(free_blocks)),
                                _p(protect, np.uint8), ctypes.byref(bits))
    if rc != 0:
        raise ValueError(f"vto_check_tables failed: {rc}")
    return bits.value


def check_semantics(S, bt_offsets, bt_blocks, tt_offsets, tt_slots, keep, free_blocks,
                    new_bt_offsets, new_bt_blocks, new_tt_slots, freed_blocks, num_free_consumed,
                    req_status, select=None, thr_num=0, thr_den=0, num_free=None) -> int:
    """0 when the result is a valid repack of the inputs under any ordering, else a check code."""
    bt_offsets, bt_blocks = _i32(bt_offsets), _i32(bt_blocks)
    tt_offsets, tt_slots = _i32(tt_offsets), _i32(tt_slots)
    keep, select, free_blocks = _u8(keep), _u8(select), _i32(free_blocks)
    new_bt_offsets, new_bt_blocks = _i32(new_bt_offsets), _i32(new_bt_blocks)
    new_tt_slots, freed_blocks, req_status = _i32(new_tt_slots), _i32(freed_blocks), _i32(req_status)
    if num_free is None:
        num_free = len(free_blocks)
    bad = ctypes.c_int32(0)
    rc = lib().vto_check_semantics(
        ctypes.c_int32(len(tt_offsets) - 1), ctypes.c_int32(S),
        _p(bt_offsets, np.int32), _p(bt_blocks, np.int32), _p(tt_offsets, np.int32),
        _p(tt_slots, np.int32), _p(keep, np.uint8), _p(select, np.uint8),
        ctypes.c_uint32(thr_num), ctypes.c_uint32(thr_den),
        _p(free_blocks, np.int32), ctypes.c_int32(num_free),
        _p(new_bt_offsets, np.int32), _p(new_bt_blocks, np.int32), _p(new_tt_slots, np.int32),
        _p(freed_blocks, np.int32), ctypes.c_int32(len(freed_blocks)),
        ctypes.c_int32(num_free_consumed), _p(req_status, np.int32), ctypes.byref(bad))
    if rc == -1:
        raise ValueError("vto_check_semantics: bad argument")
    return bad.value


def waste_ratio(S, num_allocated_blocks, tt_slots, keep=None) -> float:
    tt_slots, keep = _i32(tt_slots), _u8(keep)
    return float(lib().vto_waste_ratio(ctypes.c_int32(S), ctypes.c_int64(num_allocated_blocks),
                                       _p(tt_slots, np.int32), _p(keep, np.uint8),
                                       ctypes.c_int64(len(tt_slots))))


def openmp_threads() -> int:
    return int(lib().vto_openmp_threads())


# ---- token-table runtime ------------------------------------------------------------------
def evict_tokens(tt_offsets, tt_len, keep: np.ndarray, victim_req, victim_tok) -> int:
    """In place on ``keep`` (uint8).  Returns the number of skipped (out-of-range) victims."""
    tt_offsets, tt_len = _i32(tt_offsets), _i32(tt_len)
    victim_req, victim_tok = _i32(victim_req), _i32(victim_tok)
    assert keep.dtype == np.uint8 and keep.flags["C_CONTIGUOUS"]
    bad = ctypes.c_int32(0)
    rc = lib().vto_evict_tokens(ctypes.c_int32(len(tt_len)), _p(tt_offsets, np.int32), _p(tt_len, np.int32),
                                _p(keep, np.uint8), _p(victim_req, np.int32), _p(victim_tok, np.int32),
                                ctypes.c_int32(len(victim_req)), ctypes.byref(bad))
    if rc != 0:
        raise ValueError(f"vto_evict_tokens failed: {rc}")
    return bad.value


def sync_new_tokens(S, tt_offsets, tt_slots: np.ndarray, keep: np.ndarray, tt_len: np.ndarray,
                    phys_len: np.ndarray, bt_offsets, bt_blocks, new_len) -> int:
    """In place on tt_slots, keep, tt_len, phys_len.  Returns the number of requests that stopped early."""
    tt_offsets, bt_offsets, bt_blocks, new_len = _i32(tt_offsets), _i32(bt_offsets), _i32(bt_blocks), _i32(new_len)
    for a, d in ((tt_slots, np.int32), (keep, np.uint8), (tt_len, np.int32), (phys_len, np.int32)):
        assert a.dtype == d and a.flags["C_CONTIGUOUS"]
    bad = ctypes.c_int32(0)
    rc = lib().vto_sync_new_tokens(ctypes.c_int32(len(tt_len)), ctypes.c_int32(S), _p(tt_offsets, np.int32),
                                   _p(tt_slots, np.int32), _p(keep, np.uint8), _p(tt_len, np.int32),
                                   _p(phys_len, np.int32), _p(bt_offsets, np.int32), _p(bt_blocks, np.int32),
                                   _p(new_len, np.int32), ctypes.byref(bad))
    if rc != 0:
        raise ValueError(f"vto_sync_new_tokens failed: {rc}")
    return bad.value


def evict_tokens_counted(S, tt_offsets, tt_len, tt_slots, keep: np.ndarray, victim_req, victim_tok, n_b: np.ndarray,
                         live_total: np.ndarray) -> int:
    """evict_tokens that also keeps ``n_b`` (int32 [NB]) and ``live_total`` (int64 [1]) current."""
    tt_offsets, tt_len, tt_slots = _i32(tt_offsets), _i32(tt_len), _i32(tt_slots)
    victim_req, victim_tok = _i32(victim_req), _i32(victim_tok)
    assert keep.dtype == np.uint8 and n_b.dtype == np.int32 and live_total.dtype == np.int64
    bad = ctypes.c_int32(0)
    rc = lib().vto_evict_tokens_counted(ctypes.c_int32(len(tt_len)), ctypes.c_int32(S), ctypes.c_int32(len(n_b)),
                                        _p(tt_offsets, np.int32), _p(tt_len, np.int32), _p(tt_slots, np.int32),
                                        _p(keep, np.uint8), _p(victim_req, np.int32), _p(victim_tok, np.int32),
                                        ctypes.c_int32(len(victim_req)), _p(n_b, np.int32), _p(live_total, np.int64),
                                        ctypes.byref(bad))
    if rc != 0:
        raise ValueError(f"vto_evict_tokens_counted failed: {rc}")
    return bad.value


def sync_new_tokens_counted(S, tt_offsets, tt_slots: np.ndarray, keep: np.ndarray, tt_len: np.ndarray,
                            phys_len: np.ndarray, bt_offsets, bt_blocks, new_len, n_b: np.ndarray,
                            live_total: np.ndarray) -> int:
    """sync_new_tokens that also keeps ``n_b`` and ``live_total`` current."""
    tt_offsets, bt_offsets, bt_blocks, new_len = _i32(tt_offsets), _i32(bt_offsets), _i32(bt_blocks), _i32(new_len)
    assert n_b.dtype == np.int32 and live_total.dtype == np.int64
    bad = ctypes.c_int32(0)
    rc = lib().vto_sync_new_tokens_counted(ctypes.c_int32(len(tt_len)), ctypes.c_int32(S), ctypes.c_int32(len(n_b)),
                                           _p(tt_offsets, np.int32), _p(tt_slots, np.int32), _p(keep, np.uint8),
                                           _p(tt_len, np.int32), _p(phys_len, np.int32), _p(bt_offsets, np.int32),
                                           _p(bt_blocks, np.int32), _p(new_len, np.int32), _p(n_b, np.int32),
                                           _p(live_total, np.int64), ctypes.byref(bad))
    if rc != 0:
        raise ValueError(f"vto_sync_new_tokens_counted failed: {rc}")
    return bad.value


def build_slot_mapping(tt_offsets, tt_slots, keep=None, select=None):
    """Returns (slots, token_ids, offsets[R+1]) of the active tokens, request order then token id."""
    tt_offsets, tt_slots = _i32(tt_offsets), _i32(tt_slots)
    keep, select = _u8(keep), _u8(select)
    R = len(tt_offsets) - 1
    cap = max(1, len(tt_slots))
    slots = np.full(cap, -7, np.int32)
    ids = np.full(cap, -7, np.int32)
    off = np.zeros(R + 1, np.int32)
    n = lib().vto_build_slot_mapping(ctypes.c_int32(R), _p(tt_offsets, np.int32), _p(tt_slots, np.int32),
                                     _p(keep, np.uint8), _p(select, np.uint8), _p(slots, np.int32),
                                     _p(ids, np.int32), _p(off, np.int32), ctypes.c_int64(cap))
    if n < 0:
        raise ValueError(f"vto_build_slot_mapping failed: {n}")
    return slots[:n].copy(), ids[:n].copy(), off


def apply_moves(tt_offsets, tt_slots: np.ndarray, keep: np.ndarray, phys_len, new_tt_slots, req_status, S=1,
                new_bt_offsets=None, append_pos=None) -> None:
    """Commit of a repack, in place on tt_slots, keep and phys_len (phys_len may be None).  With
    ``S`` and ``new_bt_offsets`` the append position also holds after partial plans."""
    tt_offsets, new_tt_slots, req_status = _i32(tt_offsets), _i32(new_tt_slots), _i32(req_status)
    nbo = None if new_bt_offsets is None else _i32(new_bt_offsets)
    apos = None if append_pos is None else _i32(append_pos)
    assert tt_slots.dtype == np.int32 and keep.dtype == np.uint8
    rc = lib().vto_apply_moves(ctypes.c_int32(len(tt_offsets) - 1), ctypes.c_int32(S), _p(tt_offsets, np.int32),
                               _p(tt_slots, np.int32), _p(keep, np.uint8),
                               None if phys_len is None else _p(phys_len, np.int32), _p(new_tt_slots, np.int32),
                               _p(req_status, np.int32), None if nbo is None else _p(nbo, np.int32),
                               None if apos is None else _p(apos, np.int32))
    if rc != 0:
        raise ValueError(f"vto_apply_moves failed: {rc}")


# ---- cached slot-translation arrays ------------------------------------------------------------
def slot_cache_mark(dirty: np.ndarray, victim_req=None, req_status=None) -> None:
    """In place on ``dirty`` (uint8 [R])."""
    assert dirty.dtype == np.uint8 and dirty.flags["C_CONTIGUOUS"]
    victim_req = _i32([] if victim_req is None else victim_req)
    req_status = None if req_status is None else _i32(req_status)
    rc = lib().vto_slot_cache_mark(ctypes.c_int32(len(dirty)), _p(dirty, np.uint8), _p(victim_req, np.int32),
                                   ctypes.c_int32(len(victim_req)), _p(req_status, np.int32))
    if rc != 0:
        raise ValueError(f"vto_slot_cache_mark failed: {rc}")


def slot_cache_update(tt_offsets, tt_slots, keep, tt_len, dirty: np.ndarray, cache_slots: np.ndarray,
                      cache_ids, cache_len: np.ndarray, cache_seen: np.ndarray):
    """In place on dirty, cache_slots, cache_ids (may be None), cache_len, cache_seen.
    Returns (requests rebuilt, requests appended to)."""
    tt_offsets, tt_slots, keep, tt_len = _i32(tt_offsets), _i32(tt_slots), _u8(keep), _i32(tt_len)
    for a, d in ((dirty, np.uint8), (cache_slots, np.int32), (cache_len, np.int32), (cache_seen, np.int32)):
        assert a.dtype == d and a.flags["C_CONTIGUOUS"]
    nr, na = ctypes.c_int32(0), ctypes.c_int32(0)
    rc = lib().vto_slot_cache_update(ctypes.c_int32(len(tt_len)), _p(tt_offsets, np.int32), _p(tt_slots, np.int32),
                                     _p(keep, np.uint8), _p(tt_len, np.int32), _p(dirty, np.uint8),
                                     _p(cache_slots, np.int32), None if cache_ids is None else _p(cache_ids, np.int32),
                                     _p(cache_len, np.int32), _p(cache_seen, np.int32), ctypes.byref(nr),
                                     ctypes.byref(na))
    if rc != 0:
        raise ValueError(f"vto_slot_cache_update failed: {rc}")
    return nr.value, na.value


# ---- eligibility metadata and partial plans ---------------------------------------------------
class _PartialOpts(ctypes.Structure):
    _fields_ = [("protect", ctypes.c_void_p), ("util_num", ctypes.c_uint32), ("util_den", ctypes.c_uint32),
                ("max_source_blocks", ctypes.c_int32), ("theta_num", ctypes.c_uint32), ("theta_den", ctypes.c_uint32),
                ("detach_num", ctypes.c_uint32), ("detach_den", ctypes.c_uint32),
                ("detach_rule", ctypes.c_uint32)]


def block_liveness(S, NB, bt_offsets, bt_blocks, tt_offsets, tt_slots, keep=None):
    """Returns (n_b[NB], hist[S+1], live_total, num_allocated)."""
    bt_offsets, bt_blocks = _i32(bt_offsets), _i32(bt_blocks)
    tt_offsets, tt_slots, keep = _i32(tt_offsets), _i32(tt_slots), _u8(keep)
    n_b = np.zeros(max(1, NB), np.int32)
    hist = np.zeros(S + 1, np.int64)
    live, alloc = ctypes.c_int64(0), ctypes.c_int64(0)
    rc = lib().vto_block_liveness(ctypes.c_int32(len(tt_offsets) - 1), ctypes.c_int32(S), ctypes.c_int32(NB),
                                  _p(bt_offsets, np.int32), _p(bt_blocks, np.int32), _p(tt_offsets, np.int32),
                                  _p(tt_slots, np.int32), _p(keep, np.uint8), _p(n_b, np.int32),
                                  hist.ctypes.data_as(ctypes.c_void_p), ctypes.byref(live), ctypes.byref(alloc))
    if rc != 0:
        raise ValueError(f"vto_block_liveness failed: {rc}")
    return n_b[:NB], hist, live.value, alloc.value


def plan_partial(S, NB, bt_offsets, bt_blocks, tt_offsets, tt_slots, keep, free_blocks, select=None, thr_num=0,
                 thr_den=0, num_free=None, protect=None, util=(0, 0), max_source_blocks=0, theta=(0, 0),
                 detach=(0, 0), detach_rule=0) -> Plan:
    bt_offsets, bt_blocks = _i32(bt_offsets), _i32(bt_blocks)
    tt_offsets, tt_slots = _i32(tt_offsets), _i32(tt_slots)
    keep, select, free_blocks, protect = _u8(keep), _u8(select), _i32(free_blocks), _u8(protect)
    R, T, nbt = len(tt_offsets) - 1, int(tt_offsets[-1]), int(bt_offsets[-1])
    if num_free is None:
        num_free = len(free_blocks)
    if protect is not None:
        assert len(protect) == NB
    # a partial plan may hold on to blocks AND take destinations: size the table for both
    new_bt_offsets = np.zeros(R + 1, np.int32)
    new_bt_blocks = np.full(max(nbt + num_free, 1), -7, np.int32)
    new_tt_slots = np.full(max(T, 1), -7, np.int32)
    freed = np.full(max(nbt, 1), -7, np.int32)
    status = np.full(max(R, 1), -7, np.int32)
    msrc = np.full(max(T, 1), -7, np.int32)
    mdst = np.full(max(T, 1), -7, np.int32)
    c = _Counts()
    released = np.full(max(nbt, 1), -7, np.int32)
    o = _PartialOpts(None if protect is None else protect.ctypes.data, util[0], util[1], max_source_blocks,
                     theta[0], theta[1], detach[0], detach[1], int(detach_rule))
    rc = lib().vto_plan_partial(ctypes.c_int32(R), ctypes.c_int32(S), ctypes.c_int32(NB),
                                _p(bt_offsets, np.int32), _p(bt_blocks, np.int32), _p(tt_offsets, np.int32),
                                _p(tt_slots, np.int32), _p(keep, np.uint8), _p(select, np.uint8),
                                ctypes.c_uint32(thr_num), ctypes.c_uint32(thr_den), _p(free_blocks, np.int32),
                                ctypes.c_int32(num_free), ctypes.byref(o), _p(new_bt_offsets, np.int32),
                                _p(new_bt_blocks, np.int32), _p(new_tt_slots, np.int32), _p(freed, np.int32),
                                _p(status, np.int32), _p(msrc, np.int32), _p(mdst, np.int32), ctypes.byref(c),
                                _p(released, np.int32))
    if rc != 0:
        raise ValueError(f"vto_plan_partial failed: {rc}")
    return Plan(new_bt_offsets, new_bt_blocks[:int(new_bt_offsets[R])].copy(), new_tt_slots[:T].copy(),
                freed[:c.num_freed].copy(), status[:R].copy(), msrc[:c.num_moves].copy(), mdst[:c.num_moves].copy(),
                c.num_moves, c.num_dst_blocks, c.num_freed, c.num_free_consumed, c.num_admitted, c.num_deferred,
                released[:c.num_released].copy())


# ---- online relocation check ------------------------------------------------------------------
def digest_logical(k_pool: np.ndarray, v_pool: np.ndarray, tt_slots, keep=None, layer_begin=0, layer_end=None):
    """Order-sensitive digest of one request's active tokens over pools [L, num_slots, row].
    Returns (digest as Python int, number of active tokens)."""
    assert k_pool.ndim == 3 and k_pool.shape == v_pool.shape
    assert k_pool.flags["C_CONTIGUOUS"] and v_pool.flags["C_CONTIGUOUS"]
    tt_slots, keep = _i32(tt_slots), _u8(keep)
    L, ns, row = k_pool.shape
    if layer_end is None:
        layer_end = L
    d = ctypes.c_uint64(0)
    n = ctypes.c_int32(0)
    rc = lib().vto_digest_logical(ctypes.c_void_p(k_pool.ctypes.data), ctypes.c_void_p(v_pool.ctypes.data),
                                  ctypes.c_int64(0), ctypes.c_int64(ns), ctypes.c_int64(row * k_pool.itemsize),
                                  ctypes.c_int32(layer_begin), ctypes.c_int32(layer_end), _p(tt_slots, np.int32),
                                  _p(keep, np.uint8), ctypes.c_int32(len(tt_slots)), ctypes.byref(d), ctypes.byref(n))
    if rc != 0:
        raise ValueError(f"vto_digest_logical failed: {rc}")
    return d.value, n.value


# ---- repack in waves --------------------------------------------------------------------------
@dataclasses.dataclass
class WavePlan:
    new_bt_offsets: np.ndarray
    new_bt_blocks: np.ndarray     # trimmed to new_bt_offsets[R]
    new_tt_slots: np.ndarray
    req_status: np.ndarray
    req_wave: np.ndarray
    req_append_pos: np.ndarray    # append position of every repacked request in its final block list, -1 = none
    free_out: np.ndarray          # the pool after the last wave
    move_src: np.ndarray          # all waves back to back; apply in this order
    move_dst: np.ndarray
    wave_move_offsets: np.ndarray
    wave_counts: list             # one dict per wave
    released_blocks: np.ndarray = None    # references dropped by copy-on-write detaches, wave after wave


def plan_waves(S, NB, bt_offsets, bt_blocks, tt_offsets, tt_slots, keep, free_blocks, num_waves, select=None,
               thr_num=0, thr_den=0, partial=None) -> WavePlan:
    """``partial``: None (whole-request planner) or a dict with the keyword options of plan_partial."""
    bt_offsets, bt_blocks = _i32(bt_offsets), _i32(bt_blocks)
    tt_offsets, tt_slots = _i32(tt_offsets), _i32(tt_slots)
    keep, select, free_blocks = _u8(keep), _u8(select), _i32(free_blocks)
    R, T, nbt = len(tt_offsets) - 1, int(tt_offsets[-1]), int(bt_offsets[-1])
    num_free = len(free_blocks)
    new_bt_offsets = np.zeros(R + 1, np.int32)
    new_bt_blocks = np.full(max(nbt, 1), -7, np.int32)
    new_tt_slots = np.full(max(T, 1), -7, np.int32)
    status = np.full(max(R, 1), -7, np.int32)
    wave = np.full(max(R, 1), -7, np.int32)
    apos = np.full(max(R, 1), -7, np.int32)
    free_out = np.full(max(num_free + nbt, 1), -7, np.int32)
    nfo = ctypes.c_int32(0)
    cap = max(1, T * num_waves)
    msrc = np.full(cap, -7, np.int32)
    mdst = np.full(cap, -7, np.int32)
    offs = np.zeros(num_waves + 1, np.int64)
    counts = (_Counts * num_waves)()
    o, protect = None, None
    if partial is not None:
        protect = _u8(partial.get("protect"))
        util, theta, detach = partial.get("util", (0, 0)), partial.get("theta", (0, 0)), partial.get("detach", (0, 0))
        o = _PartialOpts(None if protect is None else protect.ctypes.data, util[0], util[1],
                         partial.get("max_source_blocks", 0), theta[0], theta[1], detach[0], detach[1],
                         int(partial.get("detach_rule", 0)))
    released = np.full(max(nbt, 1), -7, np.int32)
    rc = lib().vto_plan_waves(ctypes.c_int32(R), ctypes.c_int32(S), ctypes.c_int32(NB),
                              _p(bt_offsets, np.int32), _p(bt_blocks, np.int32), _p(tt_offsets, np.int32),
                              _p(tt_slots, np.int32), _p(keep, np.uint8), _p(select, np.uint8),
                              ctypes.c_uint32(thr_num), ctypes.c_uint32(thr_den), _p(free_blocks, np.int32),
                              ctypes.c_int32(num_free), None if o is None else ctypes.byref(o),
                              ctypes.c_int32(num_waves), _p(new_bt_offsets, np.int32), _p(new_bt_blocks, np.int32),
                              _p(new_tt_slots, np.int32), _p(status, np.int32), _p(wave, np.int32),
                              _p(apos, np.int32), _p(free_out, np.int32), ctypes.byref(nfo), _p(msrc, np.int32), _p(mdst, np.int32),
                              ctypes.c_int64(cap), offs.ctypes.data_as(ctypes.c_void_p), counts, _p(released, np.int32))
    if rc != 0:
        raise ValueError(f"vto_plan_waves failed: {rc}")
    total = int(offs[num_waves])
    wc = [{n: getattr(c, n) for n, _ in _Counts._fields_} for c in counts]
    return WavePlan(new_bt_offsets, new_bt_blocks[:int(new_bt_offsets[R])].copy(), new_tt_slots[:T].copy(),
                    status[:R].copy(), wave[:R].copy(), apos[:R].copy(), free_out[:nfo.value].copy(),
                    msrc[:total].copy(),
                    mdst[:total].copy(), offs, wc, released[:sum(c["num_released"] for c in wc)].copy())
