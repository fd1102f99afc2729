"""ctypes front for the plain C++ oracle in infaas_oracle.cpp.

TEST INFRASTRUCTURE ONLY: imported by the tests, by the smoke check and by the
benchmark's CPU-baseline leg.  It holds the per-variant load state (`queued`,
`served_total`, counters) as numpy arrays and passes plain pointers to the C++ code,
which is where every formula lives (Section 4.1 "Case I" selection, the cost objective
of Section 2.2, the load bookkeeping of Section 4.2.2).
"""
from __future__ import annotations

import ctypes
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
# INFAAS_ORACLE_SRC: another copy of the source to build and load instead (the test that plants
# mistakes in a scratch copy and checks that the pins notice uses it).
_SRC = os.environ.get("INFAAS_ORACLE_SRC") or os.path.join(_HERE, "infaas_oracle.cpp")
_LIB = os.path.join(os.path.dirname(os.path.abspath(_SRC)), "libinfaas_oracle.so")
_lib = None

NO_FEASIBLE_BIT = 0x80000000
INVALID = 0xFFFFFFFF
# life-cycle states of a variant (Section 4, state machine)
INACTIVE, ACTIVE, OVERLOADED, INTERFERED = 0, 1, 2, 3
# Model-Autoscaler answers that are not a variant id (Section 4.2.2)
AUTOSCALE_NONE, AUTOSCALE_ESCALATE = 0xFFFFFFFF, 0xFFFFFFFE


def build(force: bool = False) -> str:
    """Compile the oracle with the host compiler (-O2, no tuning flags)."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        tmp = _LIB + f".tmp{os.getpid()}"
        subprocess.check_call(["g++", "-O2", "-std=c++17", "-shared", "-fPIC", "-pthread",
                               _SRC, "-o", tmp])
        os.replace(tmp, _LIB)
    return _LIB


def _load():
    global _lib
    if _lib is None:
        lib = ctypes.CDLL(build())
        lib.oracle_pred_lat.restype = ctypes.c_uint32
        lib.oracle_pred_lat.argtypes = [ctypes.c_uint32, ctypes.c_uint32, ctypes.c_uint16]
        lib.oracle_select.restype = None
        lib.oracle_select.argtypes = [ctypes.c_void_p, ctypes.c_uint32, ctypes.c_uint32,
                                      ctypes.c_void_p, ctypes.c_void_p, ctypes.c_void_p,
                                      ctypes.c_void_p, ctypes.c_uint64, ctypes.c_void_p,
                                      ctypes.c_int]
        lib.oracle_load_update.restype = None
        lib.oracle_load_update.argtypes = [ctypes.c_void_p, ctypes.c_uint32, ctypes.c_void_p,
                                           ctypes.c_void_p, ctypes.c_void_p, ctypes.c_void_p,
                                           ctypes.c_uint64, ctypes.c_uint32]
        lib.oracle_select_stateful.restype = None
        lib.oracle_select_stateful.argtypes = [ctypes.c_void_p, ctypes.c_uint32, ctypes.c_uint32,
                                               ctypes.c_void_p, ctypes.c_void_p, ctypes.c_void_p,
                                               ctypes.c_void_p, ctypes.c_void_p, ctypes.c_void_p,
                                               ctypes.c_uint64, ctypes.c_void_p, ctypes.c_int]
        lib.oracle_load_update_stateful.restype = None
        lib.oracle_load_update_stateful.argtypes = [ctypes.c_void_p, ctypes.c_uint32, ctypes.c_void_p,
                                                    ctypes.c_void_p, ctypes.c_void_p, ctypes.c_void_p,
                                                    ctypes.c_void_p, ctypes.c_uint64, ctypes.c_uint32]
        lib.oracle_autoscale_step.restype = None
        lib.oracle_autoscale_step.argtypes = [ctypes.c_void_p, ctypes.c_uint32, ctypes.c_uint32] + \
            [ctypes.c_void_p] * 4 + [ctypes.c_uint32] * 3 + [ctypes.c_void_p] * 2
        lib.oracle_assign_workers.restype = None
        lib.oracle_assign_workers.argtypes = [ctypes.c_void_p, ctypes.c_uint32] + [ctypes.c_void_p] * 3 + \
            [ctypes.c_uint32] + [ctypes.c_void_p] * 2 + [ctypes.c_uint32, ctypes.c_void_p, ctypes.c_uint64,
                                                         ctypes.c_void_p]
        lib.oracle_frontier.restype = ctypes.c_uint32
        lib.oracle_frontier.argtypes = [ctypes.c_void_p, ctypes.c_uint32, ctypes.c_uint32, ctypes.c_void_p,
                                        ctypes.c_uint32, ctypes.c_void_p, ctypes.c_uint32]
        lib.oracle_scan_ops.restype = ctypes.c_uint64
        lib.oracle_scan_ops.argtypes = [ctypes.c_void_p, ctypes.c_uint32, ctypes.c_uint32, ctypes.c_void_p,
                                        ctypes.c_void_p, ctypes.c_void_p, ctypes.c_uint64, ctypes.c_void_p]
        _lib = lib
    return _lib


def pred_lat(lat_us: int, queued: int, batch: int) -> int:
    return int(_load().oracle_pred_lat(lat_us, queued, batch))


def _ptr(a: np.ndarray) -> int:
    assert a.flags["C_CONTIGUOUS"]
    return a.ctypes.data


class OracleCatalog:
    """Catalog rows + load state; `select` and `load_update` mirror the library's calls."""

    def __init__(self, rows: np.ndarray, n_tasks: int):
        assert rows.dtype.itemsize == 24
        self.rows = np.ascontiguousarray(rows).copy()
        self.n_tasks = int(n_tasks)
        self.n_variants = int(rows.shape[0])
        self.queued = self.rows["queued"].astype(np.uint32).copy()
        self.served_total = np.zeros(self.n_variants, np.uint64)
        self.counters = np.zeros(3, np.uint64)

    def pred_lat(self) -> np.ndarray:
        r = self.rows
        return np.array([pred_lat(int(r["lat_us"][v]), int(self.queued[v]), int(r["batch"][v]))
                         for v in range(self.n_variants)], np.uint32)

    def select(self, task, slo_us, min_acc_bp, n_threads: int = 1) -> np.ndarray:
        task = np.ascontiguousarray(task, np.uint16)
        slo_us = np.ascontiguousarray(slo_us, np.uint32)
        min_acc_bp = np.ascontiguousarray(min_acc_bp, np.uint16)
        n = task.shape[0]
        assert slo_us.shape[0] == n and min_acc_bp.shape[0] == n
        out = np.empty(n, np.uint32)
        _load().oracle_select(_ptr(self.rows), self.n_variants, self.n_tasks, _ptr(self.queued),
                              _ptr(task), _ptr(slo_us), _ptr(min_acc_bp), n, _ptr(out),
                              int(n_threads))
        return out

    def load_update(self, decision, window_us: int) -> None:
        decision = np.ascontiguousarray(decision, np.uint32)
        _load().oracle_load_update(_ptr(self.rows), self.n_variants, _ptr(self.queued),
                                   _ptr(self.served_total), _ptr(self.counters),
                                   _ptr(decision), decision.shape[0], int(window_us))

    def frontier(self, task: int) -> np.ndarray:
        """Ids of the task's non-dominated variants in (cost, pred, -acc, id) order at the current load."""
        ids = np.empty(max(1, self.n_variants), np.uint32)
        ln = _load().oracle_frontier(_ptr(self.rows), self.n_variants, self.n_tasks, _ptr(self.queued),
                                     int(task), _ptr(ids), ids.shape[0])
        return ids[:ln].copy()

    def scan_ops(self, task, decision, want_pos: bool = False):
        """Integer operations a 32-wide scan of the pruned lists needs for these decisions (see
        oracle_scan_ops in infaas_oracle.cpp); with want_pos also every query's list position."""
        task = np.ascontiguousarray(task, np.uint16)
        decision = np.ascontiguousarray(decision, np.uint32)
        pos = np.empty(task.shape[0], np.uint32) if want_pos else None
        ops = _load().oracle_scan_ops(_ptr(self.rows), self.n_variants, self.n_tasks, _ptr(self.queued),
                                      _ptr(task), _ptr(decision), task.shape[0],
                                      _ptr(pos) if want_pos else None)
        return (int(ops), pos) if want_pos else int(ops)


class StatefulOracleCatalog(OracleCatalog):
    """Catalog with a life-cycle state and a loading latency per variant (Section 4, state
    machine; Section 4.1, Case I): `select` looks at Active variants, then at Inactive ones,
    then suggests; `load_update` also moves the states."""

    def __init__(self, rows: np.ndarray, n_tasks: int, state, load_lat_us):
        super().__init__(rows, n_tasks)
        self.state = np.ascontiguousarray(state, np.uint8).copy()
        self.load_lat_us = np.ascontiguousarray(load_lat_us, np.uint32).copy()
        assert self.state.shape == (self.n_variants,) and self.load_lat_us.shape == (self.n_variants,)

    def select(self, task, slo_us, min_acc_bp, n_threads: int = 1) -> np.ndarray:
        task = np.ascontiguousarray(task, np.uint16)
        slo_us = np.ascontiguousarray(slo_us, np.uint32)
        min_acc_bp = np.ascontiguousarray(min_acc_bp, np.uint16)
        n = task.shape[0]
        assert slo_us.shape[0] == n and min_acc_bp.shape[0] == n
        out = np.empty(n, np.uint32)
        _load().oracle_select_stateful(_ptr(self.rows), self.n_variants, self.n_tasks,
                                       _ptr(self.queued), _ptr(self.state), _ptr(self.load_lat_us),
                                       _ptr(task), _ptr(slo_us), _ptr(min_acc_bp), n, _ptr(out),
                                       int(n_threads))
        return out

    def load_update(self, decision, window_us: int) -> None:
        decision = np.ascontiguousarray(decision, np.uint32)
        _load().oracle_load_update_stateful(_ptr(self.rows), self.n_variants, _ptr(self.queued),
                                            _ptr(self.served_total), _ptr(self.counters),
                                            _ptr(self.state), _ptr(decision), decision.shape[0],
                                            int(window_us))


def autoscale_step(rows: np.ndarray, n_tasks: int, count, instances, load_lat_us, task_slo_us,
                   window_us: int, slack_pct: int = 105, lambda_milli: int = 0):
    """Scaling-up step of the Model-Autoscaler for every task (Section 4.2.2): returns
    (variant, delta) arrays of n_tasks; see oracle_autoscale_step in infaas_oracle.cpp."""
    rows = np.ascontiguousarray(rows)
    nv = rows.shape[0]
    count, instances, load_lat_us = (np.ascontiguousarray(a, np.uint32) for a in (count, instances, load_lat_us))
    task_slo_us = np.ascontiguousarray(task_slo_us, np.uint32)
    assert count.shape == instances.shape == load_lat_us.shape == (nv,) and task_slo_us.shape == (n_tasks,)
    assert window_us >= 1
    variant, delta = np.empty(n_tasks, np.uint32), np.empty(n_tasks, np.uint32)
    _load().oracle_autoscale_step(_ptr(rows), nv, n_tasks, _ptr(count), _ptr(instances), _ptr(load_lat_us),
                                  _ptr(task_slo_us), int(window_us), int(slack_pct), int(lambda_milli),
                                  _ptr(variant), _ptr(delta))
    return variant, delta


def assign_workers(rows: np.ndarray, inst_variant, inst_worker, inst_load, worker_hw, worker_util, decision):
    """Worker for every decision against one snapshot of the instance and worker tables
    (Section 4.1, Case I); see oracle_assign_workers in infaas_oracle.cpp."""
    rows = np.ascontiguousarray(rows)
    iv, iw, il = (np.ascontiguousarray(a, np.uint32) for a in (inst_variant, inst_worker, inst_load))
    hw = np.ascontiguousarray(worker_hw, np.uint8)
    ut = np.ascontiguousarray(worker_util, np.uint32)
    decision = np.ascontiguousarray(decision, np.uint32)
    assert iv.shape == iw.shape == il.shape and hw.shape == ut.shape
    out = np.empty(decision.shape[0], np.uint32)
    _load().oracle_assign_workers(_ptr(rows), rows.shape[0], _ptr(iv), _ptr(iw), _ptr(il), iv.shape[0],
                                  _ptr(hw), _ptr(ut), hw.shape[0], _ptr(decision), decision.shape[0], _ptr(out))
    return out
