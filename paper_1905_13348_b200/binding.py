"""Thin ctypes binding of the C ABI in include/infaas.h (argument marshalling only).

Every step of the path runs inside the CUDA library; this module passes pointers and
sizes.  Device arrays are torch CUDA tensors (torch is used for device memory and streams
only).  There is no CPU fallback: if the library has not been built, importing the symbols
raises.
"""
from __future__ import annotations

import ctypes
import os

import numpy as np

from .build import LIB_PATH

NO_FEASIBLE = 0x80000000
INVALID = 0xFFFFFFFF
STATE_INACTIVE, STATE_ACTIVE, STATE_OVERLOADED, STATE_INTERFERED = 0, 1, 2, 3
AUTOSCALE_NONE, AUTOSCALE_ESCALATE = 0xFFFFFFFF, 0xFFFFFFFE

_lib = None

EXPORTS = ("infaas_catalog_load", "infaas_select_batch", "infaas_load_update",
           "infaas_catalog_get_state", "infaas_catalog_get_frontier", "infaas_catalog_free",
           "infaas_strerror", "infaas_last_cuda_error", "infaas_tally_static", "infaas_catalog_get_info",
           "infaas_intpipe_probe", "infaas_select_update",
           "infaas_tally", "infaas_pending_counts", "infaas_advance",
           "infaas_catalog_set_states", "infaas_catalog_get_states",
           "infaas_autoscale_config", "infaas_autoscale_step",
           "infaas_workers_config", "infaas_assign_workers")


class InfaasError(RuntimeError):
    def __init__(self, code: int, where: str):
        lib = _load()
        msg = lib.infaas_strerror(code).decode()
        cuda = lib.infaas_last_cuda_error().decode()
        super().__init__(f"{where}: {msg} ({code})" + (f" [{cuda}]" if code == -7 and cuda else ""))
        self.code = code


def _load():
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(LIB_PATH):
        raise RuntimeError(f"CUDA library not built: {LIB_PATH} is missing "
                           "(run `python -m paper_1905_13348_b200.build`); there is no fallback")
    lib = ctypes.CDLL(LIB_PATH)
    vp, u32, u64, i32 = ctypes.c_void_p, ctypes.c_uint32, ctypes.c_uint64, ctypes.c_int
    lib.infaas_catalog_load.argtypes = [vp, u32, u32, i32, ctypes.POINTER(vp)]
    lib.infaas_select_batch.argtypes = [vp, vp, vp, vp, u64, vp, vp]
    lib.infaas_load_update.argtypes = [vp, vp, u64, u32, vp]
    lib.infaas_select_update.argtypes = [vp, vp, vp, vp, u64, vp, u32, vp]
    lib.infaas_select_update.restype = i32
    lib.infaas_catalog_get_state.argtypes = [vp, vp, vp, vp, vp, vp]
    lib.infaas_catalog_get_frontier.argtypes = [vp, u32, vp, u32, ctypes.POINTER(u32), vp]
    lib.infaas_catalog_get_info.argtypes = [vp, vp, vp]
    lib.infaas_catalog_get_info.restype = i32
    lib.infaas_catalog_free.argtypes = [vp]
    lib.infaas_catalog_free.restype = None
    for name in ("infaas_catalog_load", "infaas_select_batch", "infaas_load_update",
                 "infaas_catalog_get_state", "infaas_catalog_get_frontier"):
        getattr(lib, name).restype = i32
    lib.infaas_tally.argtypes = [vp, vp, u64, vp]
    lib.infaas_pending_counts.argtypes = [vp, vp, i32, vp]
    lib.infaas_advance.argtypes = [vp, u32, vp]
    for name in ("infaas_tally", "infaas_pending_counts", "infaas_advance"):
        getattr(lib, name).restype = i32
    lib.infaas_catalog_set_states.argtypes = [vp, vp, vp, vp]
    lib.infaas_catalog_get_states.argtypes = [vp, vp, vp]
    lib.infaas_catalog_set_states.restype = lib.infaas_catalog_get_states.restype = i32
    lib.infaas_autoscale_config.argtypes = [vp, vp, vp, vp]
    lib.infaas_autoscale_step.argtypes = [vp, u32, u32, u32, vp, vp, vp]
    lib.infaas_autoscale_config.restype = lib.infaas_autoscale_step.restype = i32
    lib.infaas_workers_config.argtypes = [vp, vp, vp, vp, u32, vp, vp, u32, vp]
    lib.infaas_assign_workers.argtypes = [vp, vp, u64, vp, vp]
    lib.infaas_workers_config.restype = lib.infaas_assign_workers.restype = i32
    lib.infaas_tally_static.argtypes = [vp, u64, u32, vp, vp, i32, vp]
    lib.infaas_tally_static.restype = i32
    lib.infaas_intpipe_probe.argtypes = [u32, vp, i32, ctypes.POINTER(u64), vp]
    lib.infaas_intpipe_probe.restype = i32
    lib.infaas_strerror.argtypes = [i32]
    lib.infaas_strerror.restype = ctypes.c_char_p
    lib.infaas_last_cuda_error.argtypes = []
    lib.infaas_last_cuda_error.restype = ctypes.c_char_p
    _lib = lib
    return lib


def _check(code: int, where: str) -> None:
    if code != 0:
        raise InfaasError(code, where)


def _dev_ptr(t, dtype_name: str):
    """Device pointer of a contiguous torch CUDA tensor of the given integer width."""
    import torch
    widths = {"u16": (torch.int16, torch.uint16), "u32": (torch.int32, torch.uint32)}
    if t is None:
        return None
    if not t.is_cuda or not t.is_contiguous() or t.dtype not in widths[dtype_name]:
        raise TypeError(f"expected a contiguous CUDA tensor of {dtype_name}, got {t.dtype} on {t.device}")
    return t.data_ptr()


def _stream_ptr(stream):
    import torch
    if stream is None:
        stream = torch.cuda.current_stream()
    return ctypes.c_void_p(stream.cuda_stream)


class Catalog:
    """Owner of an `infaas_catalog*` handle."""

    def __init__(self, handle: int, n_variants: int, n_tasks: int, device: int):
        self.handle = ctypes.c_void_p(handle)
        self.n_variants, self.n_tasks, self.device = n_variants, n_tasks, device

    def free(self) -> None:
        if self.handle:
            _load().infaas_catalog_free(self.handle)
            self.handle = ctypes.c_void_p(None)

    def __del__(self):
        try:
            self.free()
        except Exception:
            pass


def infaas_catalog_load(rows: np.ndarray, n_tasks: int, cuda_device: int = 0) -> Catalog:
    """rows: host numpy array of 24-byte catalog rows (variant id = index)."""
    rows = np.ascontiguousarray(rows)
    if rows.dtype.itemsize != 24:
        raise TypeError("rows must be an array of 24-byte catalog rows")
    out = ctypes.c_void_p(None)
    _check(_load().infaas_catalog_load(rows.ctypes.data, rows.shape[0], n_tasks, cuda_device,
                                       ctypes.byref(out)), "infaas_catalog_load")
    return Catalog(out.value, int(rows.shape[0]), int(n_tasks), int(cuda_device))


def infaas_select_batch(cat: Catalog, d_task, d_slo_us, d_min_acc_bp, d_decision, n=None,
                        stream=None) -> None:
    n = int(d_task.shape[0]) if n is None else int(n)
    _check(_load().infaas_select_batch(cat.handle, _dev_ptr(d_task, "u16"), _dev_ptr(d_slo_us, "u32"),
                                       _dev_ptr(d_min_acc_bp, "u16"), n, _dev_ptr(d_decision, "u32"),
                                       _stream_ptr(stream)), "infaas_select_batch")


def infaas_load_update(cat: Catalog, d_decision, window_us: int, n=None, stream=None) -> None:
    n = int(d_decision.shape[0]) if n is None else int(n)
    _check(_load().infaas_load_update(cat.handle, _dev_ptr(d_decision, "u32"), n, int(window_us),
                                      _stream_ptr(stream)), "infaas_load_update")


def infaas_select_update(cat: Catalog, d_task, d_slo_us, d_min_acc_bp, d_decision, window_us: int, n=None,
                         stream=None) -> None:
    """One window: decide its queries, then fold the decisions into the load (one call)."""
    n = int(d_task.shape[0]) if n is None else int(n)
    _check(_load().infaas_select_update(cat.handle, _dev_ptr(d_task, "u16"), _dev_ptr(d_slo_us, "u32"),
                                        _dev_ptr(d_min_acc_bp, "u16"), n, _dev_ptr(d_decision, "u32"),
                                        int(window_us), _stream_ptr(stream)), "infaas_select_update")


def infaas_tally(cat: Catalog, d_decision, n=None, stream=None) -> None:
    n = int(d_decision.shape[0]) if n is None else int(n)
    _check(_load().infaas_tally(cat.handle, _dev_ptr(d_decision, "u32"), n, _stream_ptr(stream)),
           "infaas_tally")


def infaas_pending_counts(cat: Catalog, d_counts, set: bool, stream=None) -> None:
    """d_counts: int32/uint32 CUDA tensor of n_variants; written (set=False) or read (set=True)."""
    if d_counts.numel() < cat.n_variants:
        raise ValueError("d_counts is shorter than n_variants")
    _check(_load().infaas_pending_counts(cat.handle, _dev_ptr(d_counts, "u32"), 1 if set else 0,
                                         _stream_ptr(stream)), "infaas_pending_counts")


def infaas_advance(cat: Catalog, window_us: int, stream=None) -> None:
    _check(_load().infaas_advance(cat.handle, int(window_us), _stream_ptr(stream)), "infaas_advance")


def infaas_catalog_set_states(cat: Catalog, state, load_lat_us=None, stream=None) -> None:
    """state: host array of n_variants INFAAS_STATE_* bytes; load_lat_us: host u32 array or None."""
    state = np.ascontiguousarray(state, np.uint8)
    if state.shape != (cat.n_variants,):
        raise ValueError("state must have n_variants entries")
    if load_lat_us is not None:
        load_lat_us = np.ascontiguousarray(load_lat_us, np.uint32)
        if load_lat_us.shape != (cat.n_variants,):
            raise ValueError("load_lat_us must have n_variants entries")
    _check(_load().infaas_catalog_set_states(cat.handle, state.ctypes.data,
                                             None if load_lat_us is None else load_lat_us.ctypes.data,
                                             _stream_ptr(stream)), "infaas_catalog_set_states")


def infaas_catalog_get_states(cat: Catalog, stream=None) -> np.ndarray:
    state = np.empty(cat.n_variants, np.uint8)
    _check(_load().infaas_catalog_get_states(cat.handle, state.ctypes.data, _stream_ptr(stream)),
           "infaas_catalog_get_states")
    return state


def infaas_autoscale_config(cat: Catalog, instances, task_slo_us, stream=None) -> None:
    """instances: host u32 array of n_variants; task_slo_us: host u32 array of n_tasks."""
    instances = np.ascontiguousarray(instances, np.uint32)
    task_slo_us = np.ascontiguousarray(task_slo_us, np.uint32)
    if instances.shape != (cat.n_variants,) or task_slo_us.shape != (cat.n_tasks,):
        raise ValueError("instances needs n_variants entries and task_slo_us n_tasks")
    _check(_load().infaas_autoscale_config(cat.handle, instances.ctypes.data, task_slo_us.ctypes.data,
                                           _stream_ptr(stream)), "infaas_autoscale_config")


def infaas_autoscale_step(cat: Catalog, window_us: int, slack_pct: int, lambda_milli: int, d_variant, d_delta,
                          stream=None) -> None:
    """d_variant, d_delta: int32/uint32 CUDA tensors of n_tasks, overwritten."""
    if d_variant.numel() < cat.n_tasks or d_delta.numel() < cat.n_tasks:
        raise ValueError("outputs are shorter than n_tasks")
    _check(_load().infaas_autoscale_step(cat.handle, int(window_us), int(slack_pct), int(lambda_milli),
                                         _dev_ptr(d_variant, "u32"), _dev_ptr(d_delta, "u32"),
                                         _stream_ptr(stream)), "infaas_autoscale_step")


def infaas_workers_config(cat: Catalog, inst_variant, inst_worker, inst_load, worker_hw, worker_util,
                          stream=None) -> None:
    """Host arrays: the instance table (three u32 arrays of equal length) and the worker table
    (u8 hardware codes, u32 utilisations; worker id = index)."""
    iv, iw, il = (np.ascontiguousarray(a, np.uint32) for a in (inst_variant, inst_worker, inst_load))
    hw = np.ascontiguousarray(worker_hw, np.uint8)
    ut = np.ascontiguousarray(worker_util, np.uint32)
    if not (iv.shape == iw.shape == il.shape and iv.ndim == 1 and hw.shape == ut.shape and hw.ndim == 1):
        raise ValueError("instance arrays must have one length, worker arrays another")
    p = lambda a: a.ctypes.data if a.size else None
    _check(_load().infaas_workers_config(cat.handle, p(iv), p(iw), p(il), iv.shape[0], p(hw), p(ut), hw.shape[0],
                                         _stream_ptr(stream)), "infaas_workers_config")


def infaas_assign_workers(cat: Catalog, d_decision, d_worker, n=None, stream=None) -> None:
    n = int(d_decision.shape[0]) if n is None else int(n)
    _check(_load().infaas_assign_workers(cat.handle, _dev_ptr(d_decision, "u32"), n, _dev_ptr(d_worker, "u32"),
                                         _stream_ptr(stream)), "infaas_assign_workers")


def infaas_catalog_get_state(cat: Catalog, stream=None) -> dict:
    queued = np.empty(cat.n_variants, np.uint32)
    pred = np.empty(cat.n_variants, np.uint32)
    served = np.empty(cat.n_variants, np.uint64)
    counters = np.zeros(3, np.uint64)
    _check(_load().infaas_catalog_get_state(cat.handle, queued.ctypes.data, pred.ctypes.data,
                                            served.ctypes.data, counters.ctypes.data,
                                            _stream_ptr(stream)), "infaas_catalog_get_state")
    return {"queued": queued, "pred_lat_us": pred, "served_total": served, "counters": counters}


def infaas_catalog_get_info(cat: Catalog, stream=None) -> dict:
    info = np.zeros(8, np.uint32)
    _check(_load().infaas_catalog_get_info(cat.handle, info.ctypes.data, _stream_ptr(stream)),
           "infaas_catalog_get_info")
    return {"image_bytes": int(info[0]), "longest_list": int(info[1]), "list_entries": int(info[2]),
            "tasks_not_indexed": int(info[3]), "image_smem": int(info[4])}


def infaas_catalog_get_frontier(cat: Catalog, task: int, stream=None) -> np.ndarray:
    ids = np.empty(max(1, cat.n_variants), np.uint32)
    ln = ctypes.c_uint32(0)
    _check(_load().infaas_catalog_get_frontier(cat.handle, int(task), ids.ctypes.data, ids.shape[0],
                                               ctypes.byref(ln), _stream_ptr(stream)),
           "infaas_catalog_get_frontier")
    return ids[:ln.value].copy()


def infaas_intpipe_probe(iters: int, d_sink, stream=None) -> int:
    """Launches the integer-pipe probe on d_sink's device (see include/infaas.h); returns the
    number of lane-operations the launch executes.  The caller times it with CUDA events."""
    ops = ctypes.c_uint64(0)
    _check(_load().infaas_intpipe_probe(int(iters), _dev_ptr(d_sink, "u32"), d_sink.device.index,
                                        ctypes.byref(ops), _stream_ptr(stream)), "infaas_intpipe_probe")
    return int(ops.value)


def infaas_tally_static(d_decision, n_variants: int, d_count, d_counters, n=None, stream=None) -> None:
    """Allocation-free tallies: d_count (int32/uint32 CUDA tensor of n_variants) and
    d_counters (int64 CUDA tensor of 3) are overwritten; see include/infaas.h."""
    import torch
    n = int(d_decision.shape[0]) if n is None else int(n)
    if not (d_counters.is_cuda and d_counters.is_contiguous() and d_counters.dtype in (torch.int64, torch.uint64)
            and d_counters.numel() >= 3):
        raise TypeError("d_counters must be a contiguous CUDA tensor of 3 64-bit integers")
    if d_count.numel() < n_variants:
        raise ValueError("d_count is shorter than n_variants")
    _check(_load().infaas_tally_static(_dev_ptr(d_decision, "u32"), n, int(n_variants),
                                       _dev_ptr(d_count, "u32"), d_counters.data_ptr(),
                                       d_count.device.index, _stream_ptr(stream)), "infaas_tally_static")
