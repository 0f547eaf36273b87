"""ctypes binding of ``libvtoken.so``: same names as the C ABI in ``include/vtoken.h``,
argument marshalling only.  Device pointers may be given as ints or as anything with a
``data_ptr()`` method (torch tensors); streams as ints or objects with ``cuda_stream``.

There is no CPU fallback: importing the library fails loudly when it has not been built.
"""
from __future__ import annotations

import ctypes
import os

_PKG = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_PKG, "libvtoken.so")
CHECKED_LIB_PATH = os.path.join(_PKG, "libvtoken_checked.so")     # same ABI, every index range-checked

OK, EINVAL, ECAPACITY, ECUDA, ENOMEM, ESTATE = 0, -1, -2, -3, -4, -5
NOT_SELECTED, REPACKED, NO_GAIN, DEFERRED_NO_FREE = 0, 1, 2, 3
FLAG_BAD_SLOT, FLAG_BAD_BLOCK, FLAG_BAD_FREE, FLAG_CAPACITY, FLAG_TIMEOUT, FLAG_GATHER_OVERFLOW = 1, 2, 4, 8, 16, 32
FLAG_BAD_VICTIM, FLAG_APPEND_STOPPED, FLAG_CHECK_FAILED = 64, 128, 256

SYMBOLS = ["vtoken_create", "vtoken_destroy", "vtoken_plan", "vtoken_repack", "vtoken_gather_logical",
           "vtoken_read_counts", "vtoken_repack_host", "vtoken_strerror", "vtoken_last_cuda_error",
           "vtoken_copy_grid", "vtoken_scratch_bytes", "vtoken_plan_form", "vtoken_gather_logical_noalloc", "vtoken_evict_tokens",
           "vtoken_sync_new_tokens", "vtoken_build_slot_mapping", "vtoken_apply_moves",
           "vtoken_block_liveness", "vtoken_plan_partial", "vtoken_digest_logical",
           "vtoken_waves_workspace_bytes", "vtoken_repack_waves", "vtoken_slot_cache_mark",
           "vtoken_slot_cache_update", "vtoken_repack_host_partial", "vtoken_check_tables",
           "vtoken_evict_tokens_counted", "vtoken_sync_new_tokens_counted", "vtoken_checked_build",
           "vtoken_debug_probe"]


class VtokenError(RuntimeError):
    def __init__(self, code: int, where: str, cuda_error: int = 0):
        self.code = code
        self.cuda_error = cuda_error
        msg = f"{where}: {strerror(code)} (code {code})"
        if cuda_error:
            msg += f", cudaError {cuda_error}"
        super().__init__(msg)


class CopyTuning(ctypes.Structure):
    _fields_ = [("enabled", ctypes.c_int32), ("warps", ctypes.c_int32), ("stages", ctypes.c_int32),
                ("rows", ctypes.c_int32), ("depth", ctypes.c_int32), ("ahead", ctypes.c_int32),
                ("fixed_shares", ctypes.c_int32), ("chunk", ctypes.c_int32), ("ctas", ctypes.c_int32)]


class Config(ctypes.Structure):
    _fields_ = [("num_layers", ctypes.c_int32), ("num_blocks", ctypes.c_int32), ("block_size", ctypes.c_int32),
                ("num_kv_heads", ctypes.c_int32), ("head_dim", ctypes.c_int32), ("elem_bytes", ctypes.c_int32),
                ("k_pool", ctypes.c_void_p), ("v_pool", ctypes.c_void_p),
                ("layer_stride_bytes", ctypes.c_int64), ("max_requests", ctypes.c_int32),
                ("max_tokens", ctypes.c_int64), ("max_table_blocks", ctypes.c_int64),
                ("max_free_blocks", ctypes.c_int32), ("max_ctas", ctypes.c_int32),
                ("copy_variant", ctypes.c_int32), ("wait_limit_ms", ctypes.c_int32),
                ("plain_launches", ctypes.c_int32), ("plan_variant", ctypes.c_int32), ("tuning", CopyTuning),
                ("debug_stall_item", ctypes.c_int64)]


class PlanIn(ctypes.Structure):
    _fields_ = [("num_requests", ctypes.c_void_p), ("bt_offsets", ctypes.c_void_p), ("bt_blocks", ctypes.c_void_p),
                ("tt_offsets", ctypes.c_void_p), ("tt_slots", ctypes.c_void_p), ("keep", ctypes.c_void_p),
                ("select", ctypes.c_void_p), ("thr_num", ctypes.c_uint32), ("thr_den", ctypes.c_uint32),
                ("free_blocks", ctypes.c_void_p), ("num_free", ctypes.c_void_p)]


class Counts(ctypes.Structure):
    _fields_ = [("num_moves", ctypes.c_int32), ("num_dst_blocks", ctypes.c_int32), ("num_freed", ctypes.c_int32),
                ("num_free_consumed", ctypes.c_int32), ("num_admitted", ctypes.c_int32),
                ("num_deferred", ctypes.c_int32), ("error_flags", ctypes.c_uint32), ("num_released", ctypes.c_int32)]

    def as_dict(self):
        return {n: getattr(self, n) for n, _ in self._fields_}


class PlanOut(ctypes.Structure):
    _fields_ = [("new_bt_offsets", ctypes.c_void_p), ("new_bt_blocks", ctypes.c_void_p),
                ("new_tt_slots", ctypes.c_void_p), ("freed_blocks", ctypes.c_void_p),
                ("req_status", ctypes.c_void_p), ("counts", ctypes.c_void_p), ("released_blocks", ctypes.c_void_p)]


class PartialOpts(ctypes.Structure):
    _fields_ = [("protect", ctypes.c_void_p), ("util_num", ctypes.c_uint32), ("util_den", ctypes.c_uint32),
                ("max_source_blocks", ctypes.c_int32), ("theta_num", ctypes.c_uint32), ("theta_den", ctypes.c_uint32),
                ("detach_num", ctypes.c_uint32), ("detach_den", ctypes.c_uint32),
                ("detach_rule", ctypes.c_uint32)]


class WavesOut(ctypes.Structure):
    _fields_ = [("new_bt_offsets", ctypes.c_void_p), ("new_bt_blocks", ctypes.c_void_p),
                ("new_tt_slots", ctypes.c_void_p), ("req_status", ctypes.c_void_p), ("req_wave", ctypes.c_void_p),
                ("req_append_pos", ctypes.c_void_p), ("free_out", ctypes.c_void_p), ("num_free_out", ctypes.c_void_p), ("wave_counts", ctypes.c_void_p),
                ("free_capacity", ctypes.c_int32), ("workspace", ctypes.c_void_p),
                ("workspace_bytes", ctypes.c_int64), ("released_blocks", ctypes.c_void_p),
                ("num_released", ctypes.c_void_p)]


class HostTables(ctypes.Structure):
    _fields_ = [("num_requests", ctypes.c_int32),
                ("bt_offsets", ctypes.c_void_p), ("bt_blocks", ctypes.c_void_p),
                ("tt_offsets", ctypes.c_void_p), ("tt_slots", ctypes.c_void_p),
                ("keep", ctypes.c_void_p), ("select", ctypes.c_void_p),
                ("thr_num", ctypes.c_uint32), ("thr_den", ctypes.c_uint32),
                ("free_blocks", ctypes.c_void_p), ("num_free", ctypes.c_int32),
                ("new_bt_offsets", ctypes.c_void_p), ("new_bt_blocks", ctypes.c_void_p),
                ("new_tt_slots", ctypes.c_void_p), ("freed_blocks", ctypes.c_void_p),
                ("req_status", ctypes.c_void_p), ("counts", ctypes.c_void_p), ("released_blocks", ctypes.c_void_p)]


_lib = None
_libs = {}
_flavour = "production"


def _build_if_needed():
    """Compiles the CUDA libraries in-tree when they are missing or older than their sources and
    nvcc is available; a build failure is reported, never papered over."""
    from . import build as _build
    try:
        _build._nvcc()
    except RuntimeError:
        return                      # no compiler here: use the library as shipped (or fail below)
    _build.build()


def load():
    """Loads libvtoken.so (once), building it first when needed.  Raises when it cannot be had:
    there is no fallback."""
    global _lib
    if _lib is None:
        _build_if_needed()
        path = LIB_PATH if _flavour == "production" else CHECKED_LIB_PATH
        if not os.path.exists(path):
            raise ImportError(f"{path} is missing: run `python -m paper_2608_13263_b200.build` "
                              "(needs nvcc); this package has no CPU fallback")
        if path in _libs:
            _lib = _libs[path]
            return _lib
        lib = ctypes.CDLL(path)
        lib.vtoken_create.argtypes = [ctypes.POINTER(Config), ctypes.POINTER(ctypes.c_void_p)]
        lib.vtoken_destroy.argtypes = [ctypes.c_void_p]
        lib.vtoken_destroy.restype = None
        lib.vtoken_plan.argtypes = [ctypes.c_void_p, ctypes.POINTER(PlanIn), ctypes.POINTER(PlanOut), ctypes.c_void_p]
        lib.vtoken_repack.argtypes = [ctypes.c_void_p, ctypes.c_void_p]
        lib.vtoken_gather_logical.argtypes = [ctypes.c_void_p] * 6 + [ctypes.c_int32, ctypes.c_int32, ctypes.c_void_p,
                                                                       ctypes.c_void_p, ctypes.c_int64, ctypes.c_void_p,
                                                                       ctypes.c_void_p]
        lib.vtoken_read_counts.argtypes = [ctypes.c_void_p, ctypes.POINTER(Counts), ctypes.c_void_p]
        lib.vtoken_repack_host.argtypes = [ctypes.c_void_p, ctypes.POINTER(HostTables), ctypes.c_void_p]
        lib.vtoken_repack_host_partial.argtypes = [ctypes.c_void_p, ctypes.POINTER(HostTables),
                                                   ctypes.POINTER(PartialOpts), ctypes.c_void_p]
        lib.vtoken_check_tables.argtypes = [ctypes.c_void_p, ctypes.POINTER(PlanIn), ctypes.c_void_p, ctypes.c_void_p,
                                            ctypes.c_void_p]
        lib.vtoken_evict_tokens_counted.argtypes = [ctypes.c_void_p, ctypes.c_void_p, ctypes.c_int32] + \
                                                   [ctypes.c_void_p] * 10
        lib.vtoken_sync_new_tokens_counted.argtypes = [ctypes.c_void_p] * 13
        lib.vtoken_strerror.argtypes = [ctypes.c_int]
        lib.vtoken_strerror.restype = ctypes.c_char_p
        lib.vtoken_last_cuda_error.argtypes = [ctypes.c_void_p]
        lib.vtoken_copy_grid.argtypes = [ctypes.c_void_p] + [ctypes.POINTER(ctypes.c_int32)] * 4
        lib.vtoken_scratch_bytes.argtypes = [ctypes.c_void_p]
        lib.vtoken_scratch_bytes.restype = ctypes.c_int64
        lib.vtoken_plan_form.argtypes = [ctypes.c_void_p]
        lib.vtoken_plan_form.restype = ctypes.c_int
        lib.vtoken_gather_logical_noalloc.argtypes = (
            [ctypes.c_void_p, ctypes.c_void_p, ctypes.c_int32, ctypes.c_int32, ctypes.c_int32, ctypes.c_int64,
             ctypes.c_int64, ctypes.c_void_p, ctypes.c_int32] + [ctypes.c_void_p] * 4 +
            [ctypes.c_int32, ctypes.c_int32, ctypes.c_void_p, ctypes.c_void_p, ctypes.c_int64, ctypes.c_void_p,
             ctypes.c_void_p, ctypes.c_void_p])
        lib.vtoken_evict_tokens.argtypes = [ctypes.c_void_p, ctypes.c_void_p, ctypes.c_int32] + [ctypes.c_void_p] * 7
        lib.vtoken_sync_new_tokens.argtypes = [ctypes.c_void_p] * 11
        lib.vtoken_build_slot_mapping.argtypes = [ctypes.c_void_p] * 8 + [ctypes.c_int64, ctypes.c_void_p, ctypes.c_void_p]
        lib.vtoken_apply_moves.argtypes = [ctypes.c_void_p] * 11
        lib.vtoken_block_liveness.argtypes = [ctypes.c_void_p] * 11
        lib.vtoken_digest_logical.argtypes = [ctypes.c_void_p] * 6 + [ctypes.c_int32, ctypes.c_int32] + [ctypes.c_void_p] * 3
        lib.vtoken_plan_partial.argtypes = [ctypes.c_void_p, ctypes.POINTER(PlanIn), ctypes.POINTER(PartialOpts),
                                            ctypes.POINTER(PlanOut), ctypes.c_void_p]
        lib.vtoken_waves_workspace_bytes.argtypes = [ctypes.c_void_p, ctypes.c_int32]
        lib.vtoken_waves_workspace_bytes.restype = ctypes.c_int64
        lib.vtoken_repack_waves.argtypes = [ctypes.c_void_p, ctypes.POINTER(PlanIn), ctypes.POINTER(PartialOpts),
                                            ctypes.c_int32, ctypes.POINTER(WavesOut), ctypes.c_void_p]
        lib.vtoken_slot_cache_mark.argtypes = [ctypes.c_void_p, ctypes.c_void_p, ctypes.c_void_p, ctypes.c_int32] + \
                                              [ctypes.c_void_p] * 4
        lib.vtoken_slot_cache_update.argtypes = [ctypes.c_void_p] * 13
        lib.vtoken_checked_build.argtypes = []
        lib.vtoken_debug_probe.argtypes = [ctypes.c_void_p, ctypes.c_int64, ctypes.c_void_p, ctypes.c_void_p]
        _libs[path] = lib
        _lib = lib
    return _lib


def use_library(flavour: str) -> str:
    """Selects the build every later call of this module goes to: "production" (libvtoken.so) or
    "checked" (libvtoken_checked.so: the same sources compiled with -DVTOKEN_CHECKED, every index
    into scratch, tables and pools range-checked, an out-of-range access skipped and reported as
    VTOKEN_FLAG_CHECK_FAILED).  Returns the previous flavour.  Contexts belong to the library that
    created them: destroy them before switching."""
    global _lib, _flavour
    if flavour not in ("production", "checked"):
        raise ValueError(flavour)
    prev, _flavour = _flavour, flavour
    _lib = None
    return prev


def _ptr(x):
    if x is None:
        return None
    if isinstance(x, int):
        return x
    if hasattr(x, "data_ptr"):
        return x.data_ptr()
    if hasattr(x, "ctypes"):          # numpy array (host pointers of vtoken_repack_host)
        return x.ctypes.data
    raise TypeError(f"cannot take a pointer from {type(x)}")


def _stream(s):
    if s is None:
        return None
    if isinstance(s, int):
        return s
    return s.cuda_stream


def strerror(code: int) -> str:
    return load().vtoken_strerror(code).decode()


def _check(rc, where, ctx=None):
    if rc != OK:
        cuda = load().vtoken_last_cuda_error(ctx) if (ctx and rc in (ECUDA, ENOMEM)) else 0
        raise VtokenError(rc, where, cuda)


def vtoken_create(num_layers, num_blocks, block_size, num_kv_heads, head_dim, k_pool, v_pool, max_requests,
                  max_tokens, max_table_blocks, max_free_blocks, elem_bytes=2, layer_stride_bytes=0, max_ctas=0,
                  copy_variant=0, wait_limit_ms=0, plain_launches=0, tuning=None, plan_variant=0,
                  debug_stall_item=0) -> int:
    """``tuning``: dict with any of warps, stages, rows, depth, ahead, fixed_shares, chunk, ctas (the fields of
    vtoken_copy_tuning; giving it sets ``enabled``)."""
    t = CopyTuning()
    if tuning:
        t.enabled = 1
        t.depth, t.ahead = 2, 2                   # the defaults of the two fields whose zero means something
        for k, v in tuning.items():
            setattr(t, k, int(v))
    cfg = Config(num_layers, num_blocks, block_size, num_kv_heads, head_dim, elem_bytes, _ptr(k_pool), _ptr(v_pool),
                 layer_stride_bytes, max_requests, max_tokens, max_table_blocks, max_free_blocks, max_ctas,
                 copy_variant, wait_limit_ms, plain_launches, plan_variant, t, debug_stall_item)
    ctx = ctypes.c_void_p()
    _check(load().vtoken_create(ctypes.byref(cfg), ctypes.byref(ctx)), "vtoken_create")
    return ctx.value


def vtoken_destroy(ctx) -> None:
    load().vtoken_destroy(ctx)


def vtoken_plan(ctx, *, num_requests, bt_offsets, bt_blocks, tt_offsets, tt_slots, keep, free_blocks, num_free,
                new_bt_offsets, new_bt_blocks, new_tt_slots, freed_blocks, req_status, counts,
                select=None, thr_num=0, thr_den=0, stream=None) -> None:
    pin = PlanIn(_ptr(num_requests), _ptr(bt_offsets), _ptr(bt_blocks), _ptr(tt_offsets), _ptr(tt_slots), _ptr(keep),
                 _ptr(select), thr_num, thr_den, _ptr(free_blocks), _ptr(num_free))
    pout = PlanOut(_ptr(new_bt_offsets), _ptr(new_bt_blocks), _ptr(new_tt_slots), _ptr(freed_blocks),
                   _ptr(req_status), _ptr(counts))
    _check(load().vtoken_plan(ctx, ctypes.byref(pin), ctypes.byref(pout), _stream(stream)), "vtoken_plan", ctx)


def vtoken_repack(ctx, stream=None) -> None:
    _check(load().vtoken_repack(ctx, _stream(stream)), "vtoken_repack", ctx)


def vtoken_gather_logical(ctx, *, num_requests, tt_offsets, tt_slots, keep, select, layer_begin, layer_end,
                          out_k, out_v, out_capacity_tokens, out_offsets, stream=None) -> None:
    _check(load().vtoken_gather_logical(ctx, _ptr(num_requests), _ptr(tt_offsets), _ptr(tt_slots), _ptr(keep),
                                        _ptr(select), layer_begin, layer_end, _ptr(out_k), _ptr(out_v),
                                        out_capacity_tokens, _ptr(out_offsets), _stream(stream)),
           "vtoken_gather_logical", ctx)


def vtoken_read_counts(ctx, stream=None) -> dict:
    c = Counts()
    _check(load().vtoken_read_counts(ctx, ctypes.byref(c), _stream(stream)), "vtoken_read_counts", ctx)
    return c.as_dict()


def vtoken_repack_host(ctx, *, num_requests, bt_offsets, bt_blocks, tt_offsets, tt_slots, keep, free_blocks,
                       num_free, new_bt_offsets, new_bt_blocks, new_tt_slots, freed_blocks, req_status,
                       select=None, thr_num=0, thr_den=0, stream=None) -> dict:
    """All table arguments are HOST arrays (numpy or pinned torch tensors)."""
    c = Counts()
    h = HostTables(num_requests, _ptr(bt_offsets), _ptr(bt_blocks), _ptr(tt_offsets), _ptr(tt_slots), _ptr(keep),
                   _ptr(select), thr_num, thr_den, _ptr(free_blocks), num_free, _ptr(new_bt_offsets),
                   _ptr(new_bt_blocks), _ptr(new_tt_slots), _ptr(freed_blocks), _ptr(req_status),
                   ctypes.addressof(c))
    _check(load().vtoken_repack_host(ctx, ctypes.byref(h), _stream(stream)), "vtoken_repack_host", ctx)
    return c.as_dict()


def vtoken_repack_host_partial(ctx, *, num_requests, bt_offsets, bt_blocks, tt_offsets, tt_slots, keep, free_blocks,
                               num_free, new_bt_offsets, new_bt_blocks, new_tt_slots, freed_blocks, req_status,
                               select=None, thr_num=0, thr_den=0, protect=None, util=(0, 0), max_source_blocks=0,
                               theta=(0, 0), detach=(0, 0), released_blocks=None, detach_rule=0,
                               stream=None) -> dict:
    """vtoken_repack_host with the partial planner; ``protect`` is a HOST array of num_blocks bytes,
    ``released_blocks`` a HOST array of bt_offsets[R] entries (needed with a detach threshold)."""
    c = Counts()
    h = HostTables(num_requests, _ptr(bt_offsets), _ptr(bt_blocks), _ptr(tt_offsets), _ptr(tt_slots), _ptr(keep),
                   _ptr(select), thr_num, thr_den, _ptr(free_blocks), num_free, _ptr(new_bt_offsets),
                   _ptr(new_bt_blocks), _ptr(new_tt_slots), _ptr(freed_blocks), _ptr(req_status),
                   ctypes.addressof(c), _ptr(released_blocks))
    po = PartialOpts(_ptr(protect), util[0], util[1], max_source_blocks, theta[0], theta[1], detach[0], detach[1],
                     int(detach_rule))
    _check(load().vtoken_repack_host_partial(ctx, ctypes.byref(h), ctypes.byref(po), _stream(stream)),
           "vtoken_repack_host_partial", ctx)
    return c.as_dict()


def vtoken_check_tables(ctx, *, num_requests, bt_offsets, bt_blocks, tt_offsets, tt_slots, free_blocks, num_free,
                        out_bits, protect=None, stream=None) -> None:
    """Bit set of violated input preconditions into ``out_bits`` (device uint32); 0 = valid."""
    pin = PlanIn(_ptr(num_requests), _ptr(bt_offsets), _ptr(bt_blocks), _ptr(tt_offsets), _ptr(tt_slots), None,
                 None, 0, 0, _ptr(free_blocks), _ptr(num_free))
    _check(load().vtoken_check_tables(ctx, ctypes.byref(pin), _ptr(protect), _ptr(out_bits), _stream(stream)),
           "vtoken_check_tables", ctx)


def vtoken_copy_grid(ctx) -> dict:
    v = [ctypes.c_int32() for _ in range(4)]
    _check(load().vtoken_copy_grid(ctx, *[ctypes.byref(x) for x in v]), "vtoken_copy_grid")
    return dict(ctas=v[0].value, threads=v[1].value, smem_bytes=v[2].value, variant=v[3].value)


def vtoken_checked_build() -> int:
    return int(load().vtoken_checked_build())


def vtoken_debug_probe(ctx, index: int, out_value, stream=None) -> None:
    _check(load().vtoken_debug_probe(ctx, index, _ptr(out_value), _stream(stream)), "vtoken_debug_probe", ctx)


def vtoken_scratch_bytes(ctx) -> int:
    return load().vtoken_scratch_bytes(ctx)


def vtoken_plan_form(ctx) -> int:
    return load().vtoken_plan_form(ctx)


NOALLOC_MAX_REQUESTS = 4096
NOALLOC_MAX_TOKENS = 262144


def vtoken_gather_logical_noalloc(*, k_pool, v_pool, num_layers, num_blocks, block_size, row_bytes, num_requests,
                                  max_requests, tt_offsets, tt_slots, keep, select, layer_begin, layer_end, out_k,
                                  out_v, out_capacity_tokens, out_offsets, error_flags=None, layer_stride_bytes=0,
                                  stream=None) -> None:
    """The logical gather without a context and without any device allocation: for callers
    whose memory is fully committed to the KV pool or who may not call the allocator.  Limits:
    max_requests <= 4096 and out_capacity_tokens <= 262144 (VtokenError ECAPACITY beyond).  Calls
    on one device share a fixed scratch array, so they must not overlap on the GPU."""
    _check(load().vtoken_gather_logical_noalloc(
        _ptr(k_pool), _ptr(v_pool), num_layers, num_blocks, block_size, row_bytes, layer_stride_bytes,
        _ptr(num_requests), max_requests, _ptr(tt_offsets), _ptr(tt_slots), _ptr(keep), _ptr(select), layer_begin,
        layer_end, _ptr(out_k), _ptr(out_v), out_capacity_tokens, _ptr(out_offsets), _ptr(error_flags),
        _stream(stream)), "vtoken_gather_logical_noalloc")


# ---- token-table runtime ------------------------------------------------------------------
def vtoken_evict_tokens(ctx, *, num_victims, max_victims, victim_req, victim_tok, num_requests, tt_offsets, tt_len,
                        keep, stream=None) -> None:
    _check(load().vtoken_evict_tokens(ctx, _ptr(num_victims), max_victims, _ptr(victim_req), _ptr(victim_tok),
                                      _ptr(num_requests), _ptr(tt_offsets), _ptr(tt_len), _ptr(keep),
                                      _stream(stream)), "vtoken_evict_tokens", ctx)


def vtoken_sync_new_tokens(ctx, *, num_requests, tt_offsets, tt_slots, keep, tt_len, phys_len, bt_offsets, bt_blocks,
                           new_len, stream=None) -> None:
    _check(load().vtoken_sync_new_tokens(ctx, _ptr(num_requests), _ptr(tt_offsets), _ptr(tt_slots), _ptr(keep),
                                         _ptr(tt_len), _ptr(phys_len), _ptr(bt_offsets), _ptr(bt_blocks),
                                         _ptr(new_len), _stream(stream)), "vtoken_sync_new_tokens", ctx)


def vtoken_evict_tokens_counted(ctx, *, num_victims, max_victims, victim_req, victim_tok, num_requests, tt_offsets,
                                tt_len, tt_slots, keep, n_b, live_total=None, stream=None) -> None:
    _check(load().vtoken_evict_tokens_counted(ctx, _ptr(num_victims), max_victims, _ptr(victim_req), _ptr(victim_tok),
                                              _ptr(num_requests), _ptr(tt_offsets), _ptr(tt_len), _ptr(tt_slots),
                                              _ptr(keep), _ptr(n_b), _ptr(live_total), _stream(stream)),
           "vtoken_evict_tokens_counted", ctx)


def vtoken_sync_new_tokens_counted(ctx, *, num_requests, tt_offsets, tt_slots, keep, tt_len, phys_len, bt_offsets,
                                   bt_blocks, new_len, n_b, live_total=None, stream=None) -> None:
    _check(load().vtoken_sync_new_tokens_counted(ctx, _ptr(num_requests), _ptr(tt_offsets), _ptr(tt_slots),
                                                 _ptr(keep), _ptr(tt_len), _ptr(phys_len), _ptr(bt_offsets),
                                                 _ptr(bt_blocks), _ptr(new_len), _ptr(n_b), _ptr(live_total),
                                                 _stream(stream)), "vtoken_sync_new_tokens_counted", ctx)


def vtoken_build_slot_mapping(ctx, *, num_requests, tt_offsets, tt_slots, keep, select, out_slots, out_token_ids,
                              out_capacity, out_offsets, stream=None) -> None:
    _check(load().vtoken_build_slot_mapping(ctx, _ptr(num_requests), _ptr(tt_offsets), _ptr(tt_slots), _ptr(keep),
                                            _ptr(select), _ptr(out_slots), _ptr(out_token_ids), out_capacity,
                                            _ptr(out_offsets), _stream(stream)), "vtoken_build_slot_mapping", ctx)


def vtoken_apply_moves(ctx, *, num_requests, tt_offsets, tt_slots, keep, phys_len, new_tt_slots, req_status,
                       new_bt_offsets=None, append_pos=None, stream=None) -> None:
    _check(load().vtoken_apply_moves(ctx, _ptr(num_requests), _ptr(tt_offsets), _ptr(tt_slots), _ptr(keep),
                                     _ptr(phys_len), _ptr(new_tt_slots), _ptr(req_status), _ptr(new_bt_offsets),
                                     _ptr(append_pos), _stream(stream)),
           "vtoken_apply_moves", ctx)


def vtoken_slot_cache_mark(ctx, *, dirty, num_requests, num_victims=None, max_victims=0, victim_req=None,
                           req_status=None, stream=None) -> None:
    _check(load().vtoken_slot_cache_mark(ctx, _ptr(dirty), _ptr(num_victims), max_victims, _ptr(victim_req),
                                         _ptr(req_status), _ptr(num_requests), _stream(stream)),
           "vtoken_slot_cache_mark", ctx)


def vtoken_slot_cache_update(ctx, *, num_requests, tt_offsets, tt_slots, keep, tt_len, dirty, cache_slots, cache_len,
                             cache_seen, cache_ids=None, stats=None, stream=None) -> None:
    _check(load().vtoken_slot_cache_update(ctx, _ptr(num_requests), _ptr(tt_offsets), _ptr(tt_slots), _ptr(keep),
                                           _ptr(tt_len), _ptr(dirty), _ptr(cache_slots), _ptr(cache_ids),
                                           _ptr(cache_len), _ptr(cache_seen), _ptr(stats), _stream(stream)),
           "vtoken_slot_cache_update", ctx)


# ---- eligibility metadata and partial plans ---------------------------------------------------
def vtoken_block_liveness(ctx, *, num_requests, bt_offsets, bt_blocks, tt_offsets, tt_slots, keep, n_b, hist=None,
                          summary=None, stream=None) -> None:
    _check(load().vtoken_block_liveness(ctx, _ptr(num_requests), _ptr(bt_offsets), _ptr(bt_blocks), _ptr(tt_offsets),
                                        _ptr(tt_slots), _ptr(keep), _ptr(n_b), _ptr(hist), _ptr(summary),
                                        _stream(stream)), "vtoken_block_liveness", ctx)


def vtoken_plan_partial(ctx, *, num_requests, bt_offsets, bt_blocks, tt_offsets, tt_slots, keep, free_blocks, num_free,
                        new_bt_offsets, new_bt_blocks, new_tt_slots, freed_blocks, req_status, counts, select=None,
                        thr_num=0, thr_den=0, protect=None, util=(0, 0), max_source_blocks=0, theta=(0, 0),
                        detach=(0, 0), released_blocks=None, detach_rule=0, stream=None) -> None:
    pin = PlanIn(_ptr(num_requests), _ptr(bt_offsets), _ptr(bt_blocks), _ptr(tt_offsets), _ptr(tt_slots), _ptr(keep),
                 _ptr(select), thr_num, thr_den, _ptr(free_blocks), _ptr(num_free))
    pout = PlanOut(_ptr(new_bt_offsets), _ptr(new_bt_blocks), _ptr(new_tt_slots), _ptr(freed_blocks),
                   _ptr(req_status), _ptr(counts), _ptr(released_blocks))
    po = PartialOpts(_ptr(protect), util[0], util[1], max_source_blocks, theta[0], theta[1], detach[0], detach[1],
                     int(detach_rule))
    _check(load().vtoken_plan_partial(ctx, ctypes.byref(pin), ctypes.byref(po), ctypes.byref(pout), _stream(stream)),
           "vtoken_plan_partial", ctx)


def vtoken_digest_logical(ctx, *, num_requests, tt_offsets, tt_slots, keep, select, layer_begin, layer_end, out_digest,
                          out_offsets=None, stream=None) -> None:
    _check(load().vtoken_digest_logical(ctx, _ptr(num_requests), _ptr(tt_offsets), _ptr(tt_slots), _ptr(keep),
                                        _ptr(select), layer_begin, layer_end, _ptr(out_digest), _ptr(out_offsets),
                                        _stream(stream)), "vtoken_digest_logical", ctx)


# ---- repack in waves --------------------------------------------------------------------------
def vtoken_waves_workspace_bytes(ctx, free_capacity: int) -> int:
    return load().vtoken_waves_workspace_bytes(ctx, free_capacity)


def vtoken_repack_waves(ctx, *, num_requests, bt_offsets, bt_blocks, tt_offsets, tt_slots, keep, free_blocks, num_free,
                        num_waves, new_bt_offsets, new_bt_blocks, new_tt_slots, req_status, req_wave, free_out,
                        num_free_out, wave_counts, free_capacity, workspace, workspace_bytes, select=None, thr_num=0,
                        thr_den=0, partial=None, req_append_pos=None, released_blocks=None, num_released=None,
                        stream=None) -> None:
    """``partial``: None for the whole-request planner, else a dict with the option keywords of
    vtoken_plan_partial (protect, util, max_source_blocks, theta, detach)."""
    pin = PlanIn(_ptr(num_requests), _ptr(bt_offsets), _ptr(bt_blocks), _ptr(tt_offsets), _ptr(tt_slots), _ptr(keep),
                 _ptr(select), thr_num, thr_den, _ptr(free_blocks), _ptr(num_free))
    wout = WavesOut(_ptr(new_bt_offsets), _ptr(new_bt_blocks), _ptr(new_tt_slots), _ptr(req_status), _ptr(req_wave),
                    _ptr(req_append_pos), _ptr(free_out), _ptr(num_free_out), _ptr(wave_counts), free_capacity, _ptr(workspace),
                    workspace_bytes, _ptr(released_blocks), _ptr(num_released))
    po = None
    if partial is not None:
        util, theta = partial.get("util", (0, 0)), partial.get("theta", (0, 0))
        detach = partial.get("detach", (0, 0))
        po = ctypes.byref(PartialOpts(_ptr(partial.get("protect")), util[0], util[1],
                                      partial.get("max_source_blocks", 0), theta[0], theta[1], detach[0], detach[1],
                                      int(partial.get("detach_rule", 0))))
    _check(load().vtoken_repack_waves(ctx, ctypes.byref(pin), po, num_waves, ctypes.byref(wout), _stream(stream)),
           "vtoken_repack_waves", ctx)
