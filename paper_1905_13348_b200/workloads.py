"""Seeded synthetic catalogs and query streams (inputs only).

This module draws the *inputs* of the model-variant selection path: catalog rows
(one profiled model-variant each) and query arrays (task, latency SLO, minimum
accuracy).  It contains none of the method's arithmetic -- no feasibility test,
no predicted latency, no ordering of variants -- so that both the CUDA path and
the CPU oracle can be fed from it without sharing any logic.

Value ranges follow what the paper prints about its variant population
(Section 1 / Section 2.1: accuracy 56.6-82.5 %, single-query latency 1.5 ms -
5.7 s, 32x hardware cost spread; Section 5: batch sizes in powers of two;
Section 6.2: normalised cost 0.031 / 0.190 / 0.498 for CPU / Inferentia / GPU;
Section 6.1: Zipf model popularity).  The paper's own trace and profile table
are not available; these are stand-ins of the same shape.
"""
from __future__ import annotations

import dataclasses
import math

import numpy as np

# One catalog row; the layout equals `infaas_variant` in include/infaas.h (24 bytes).
VARIANT_DTYPE = np.dtype(
    [
        ("task", "<u2"),
        ("arch", "<u2"),
        ("hw", "u1"),
        ("opt", "u1"),
        ("batch", "<u2"),
        ("lat_us", "<u4"),
        ("acc_bp", "<u2"),
        ("reserved", "<u2"),
        ("cost", "<u4"),
        ("queued", "<u4"),
    ],
    align=False,
)
assert VARIANT_DTYPE.itemsize == 24


@dataclasses.dataclass
class Workload:
    name: str
    n_tasks: int
    rows: np.ndarray          # VARIANT_DTYPE[n_variants]; variant id = index
    task: np.ndarray          # u16[N]
    slo_us: np.ndarray        # u32[N]
    min_acc_bp: np.ndarray    # u16[N]
    window: int               # queries per load-update window (0 = single snapshot)
    window_us: int            # length of one window in microseconds (0 if window == 0)
    recipe: str

    @property
    def n_queries(self) -> int:
        return int(self.task.shape[0])

    @property
    def n_variants(self) -> int:
        return int(self.rows.shape[0])


# ----------------------------------------------------------------------------------
# small helpers (plain draws; nothing here knows what a "feasible" variant is)
# ----------------------------------------------------------------------------------

def _rng(seed: int, stream: int = 0) -> np.random.Generator:
    return np.random.Generator(np.random.PCG64([seed, stream]))


def _lognormal_us(rng, median_us: float, sigma: float, size) -> np.ndarray:
    return median_us * np.exp(sigma * rng.standard_normal(size))


def _log_uniform_int(rng, lo: int, hi: int, size: int) -> np.ndarray:
    u = rng.random(size)
    v = np.floor(np.exp(math.log(lo) + u * (math.log(hi + 1) - math.log(lo))))
    return np.clip(v, lo, hi).astype(np.uint32)


def _zipf_pmf(n: int, s: float) -> np.ndarray:
    w = 1.0 / np.arange(1, n + 1, dtype=np.float64) ** s
    return w / w.sum()


def _draw_categorical(rng, pmf: np.ndarray, size: int) -> np.ndarray:
    cdf = np.cumsum(pmf)
    cdf[-1] = 1.0
    return np.searchsorted(cdf, rng.random(size), side="right").astype(np.int64)


def _per_task_acc_stats(rows: np.ndarray, n_tasks: int):
    """min / median / max accuracy of each task's variants (plain order statistics)."""
    lo = np.zeros(n_tasks, np.int64)
    med = np.zeros(n_tasks, np.int64)
    hi = np.zeros(n_tasks, np.int64)
    for t in range(n_tasks):
        a = np.sort(rows["acc_bp"][rows["task"] == t].astype(np.int64))
        if a.size == 0:
            continue
        lo[t], med[t], hi[t] = a[0], a[(a.size - 1) // 2], a[-1]
    return lo, med, hi


# ----------------------------------------------------------------------------------
# catalogs
# ----------------------------------------------------------------------------------

# Four hardware tiers: CPU, Inferentia-like, V100-like, one faster/pricier tier.
# Price factors 31 : 190 : 498 are the paper's normalised costs (Section 6.2); the fourth
# brings the spread to 32x (Section 1).  Speed factors follow the 200 / 20 / 15 ms example
# of Table 2.  alpha is the exponent of the sub-linear latency growth with batch size.
_HW_PRICE = np.array([31.0, 190.0, 498.0, 992.0])
_HW_SPEED = np.array([1.0, 0.10, 0.075, 0.04])
_HW_ALPHA = np.array([0.90, 0.70, 0.55, 0.50])
_HW_ACC_LOSS_BP = np.array([0, 25, 60, 40])     # small loss from the graph optimiser


def structured_catalog(rng, n_tasks: int, n_arch: int, n_hw: int, batches, *,
                       base_median_us: float = 20000.0, sigma: float = 0.8,
                       queued_hi: int = 0) -> np.ndarray:
    """T tasks x (n_arch x n_hw x len(batches)) variants, rows interleaved across tasks.

    Rows are emitted in a seeded random order, so a task's variant ids are scattered
    through the id space (the packer has to bucket them).
    """
    batches = np.asarray(batches, dtype=np.int64)
    nb = batches.size
    v_per_task = n_arch * n_hw * nb
    rows = np.zeros(n_tasks * v_per_task, VARIANT_DTYPE)
    k = 0
    for t in range(n_tasks):
        arch_lat = _lognormal_us(rng, base_median_us, sigma, n_arch)          # CPU, batch 1
        arch_acc = rng.integers(5660, 8251, n_arch)
        arch_mem = np.exp(rng.uniform(0.0, math.log(8.0), n_arch))            # footprint 1..8
        jitter = np.exp(0.25 * rng.standard_normal((n_arch, n_hw)))
        opt_loss = rng.integers(0, 16, (n_arch, n_hw))
        for a in range(n_arch):
            for h in range(n_hw):
                hh = h % 4
                lat1 = arch_lat[a] * _HW_SPEED[hh] * jitter[a, h]
                for bi in range(nb):
                    b = int(batches[bi])
                    r = rows[k]
                    r["task"] = t
                    r["arch"] = a
                    r["hw"] = h
                    r["opt"] = hh
                    r["batch"] = b
                    r["lat_us"] = max(1, int(round(lat1 * b ** _HW_ALPHA[hh])))
                    r["acc_bp"] = max(0, int(arch_acc[a]) - int(_HW_ACC_LOSS_BP[hh]) - int(opt_loss[a, h]))
                    r["cost"] = max(1, int(round(_HW_PRICE[hh] * arch_mem[a] * (1.0 + 0.05 * bi))))
                    k += 1
    if queued_hi > 0:
        rows["queued"] = rng.integers(0, queued_hi + 1, rows.size)
    perm = rng.permutation(rows.size)
    return rows[perm].copy()


def tradeoff_catalog(rng, n_tasks: int, v_per_task: int) -> np.ndarray:
    """Variants drawn along a latency / cost / accuracy trade-off surface.

    cost ~ K / lat^gamma x noise and accuracy rising with log-latency + noise, so few
    variants dominate others and the non-dominated set is long.
    """
    rows = np.zeros(n_tasks * v_per_task, VARIANT_DTYPE)
    for t in range(n_tasks):
        s = slice(t * v_per_task, (t + 1) * v_per_task)
        loglat = rng.uniform(math.log(1500.0), math.log(5.7e6), v_per_task)
        lat = np.exp(loglat)
        gamma = 0.6
        cost = 4.0e5 / lat ** gamma * np.exp(0.35 * rng.standard_normal(v_per_task))
        frac = (loglat - math.log(1500.0)) / (math.log(5.7e6) - math.log(1500.0))
        acc = 5660.0 + (8250.0 - 5660.0) * frac ** 0.7 + 120.0 * rng.standard_normal(v_per_task)
        rows["task"][s] = t
        idx = np.arange(v_per_task)
        rows["arch"][s] = idx // 64
        rows["hw"][s] = (idx // 8) % 8
        rows["opt"][s] = (idx // 8) % 4
        rows["batch"][s] = 1 << (idx % 8)
        rows["lat_us"][s] = np.maximum(1, np.round(lat)).astype(np.uint32)
        rows["acc_bp"][s] = np.clip(np.round(acc), 0, 10000).astype(np.uint16)
        rows["cost"][s] = np.maximum(1, np.round(cost)).astype(np.uint32)
    perm = rng.permutation(rows.size)
    return rows[perm].copy()


# ----------------------------------------------------------------------------------
# query streams
# ----------------------------------------------------------------------------------

def _min_acc_split(rng, task: np.ndarray, rows: np.ndarray, n_tasks: int, frac_above: float):
    """min-acc: `frac_above` of the queries uniform in (task median, task max], the rest
    uniform in [task min, task median]."""
    lo, med, hi = _per_task_acc_stats(rows, n_tasks)
    n = task.size
    above = rng.random(n) < frac_above
    u = rng.random(n)
    t = task.astype(np.int64)
    a_lo = np.where(above, med[t] + 1, lo[t])
    a_hi = np.where(above, np.maximum(hi[t], med[t] + 1), med[t])
    v = a_lo + np.floor(u * (a_hi - a_lo + 1)).astype(np.int64)
    return np.clip(v, 0, 65535).astype(np.uint16)


def _min_acc_uniform(rng, task: np.ndarray, rows: np.ndarray, n_tasks: int):
    lo, _, hi = _per_task_acc_stats(rows, n_tasks)
    t = task.astype(np.int64)
    v = lo[t] + np.floor(rng.random(task.size) * (hi[t] - lo[t] + 1)).astype(np.int64)
    return np.clip(v, 0, 65535).astype(np.uint16)


# ----------------------------------------------------------------------------------
# the five configurations
# ----------------------------------------------------------------------------------

C3_WINDOW = 65536
C3_WINDOW_US = 40000
C5_WINDOW_US = 25000
# Scale on the accuracy quantile of C4's queries; set so that about 10 % of the queries
# have no feasible variant (the value comes from tests/golden/calibrate_c4.py).
C4_ACC_QUANTILE_SCALE = 0.337


def config_c1(n_queries: int = 10_000) -> Workload:
    rng = _rng(1)
    v = 32
    rows = np.zeros(v, VARIANT_DTYPE)
    idx = np.arange(v)
    rows["task"] = 0
    rows["arch"] = idx // 8
    rows["hw"] = (idx // 4) % 2
    rows["opt"] = (idx // 4) % 2
    rows["batch"] = 1 << (idx % 4)
    rows["lat_us"] = np.maximum(1, np.round(_lognormal_us(rng, 20000.0, 0.8, v))).astype(np.uint32)
    rows["acc_bp"] = rng.integers(6000, 8001, v)
    rows["cost"] = rng.integers(1, 1001, v)
    task = np.zeros(n_queries, np.uint16)
    slo = rng.integers(5000, 200001, n_queries).astype(np.uint32)
    acc = rng.integers(6000, 8001, n_queries).astype(np.uint16)
    return Workload("C1", 1, rows, task, slo, acc, 0, 0,
                    "1 task x 32 variants, uniform SLO [5,200] ms, min-acc [6000,8000], zero load")


def config_c2(n_queries: int = 1_000_000) -> Workload:
    rng = _rng(2)
    T = 20
    rows = structured_catalog(rng, T, 8, 4, [1, 2, 4, 8, 16, 32, 64, 128], queued_hi=16)
    task = rng.integers(0, T, n_queries).astype(np.uint16)
    slo = _log_uniform_int(rng, 2000, 500000, n_queries)
    acc = _min_acc_uniform(rng, task, rows, T)
    return Workload("C2", T, rows, task, slo, acc, 0, 0,
                    "20 tasks x 256 variants, uniform tasks, SLO log-uniform [2,500] ms, "
                    "static load uniform [0,16] queued")


def config_c3(n_queries: int = 1 << 24, window: int = C3_WINDOW) -> Workload:
    rng = _rng(3)
    T = 64
    rows = structured_catalog(rng, T, 8, 4, [1, 2, 4, 8, 16, 32, 64, 128])
    perm = rng.permutation(T)
    task = perm[_draw_categorical(rng, _zipf_pmf(T, 1.1), n_queries)].astype(np.uint16)
    slo = _log_uniform_int(rng, 1000, 1_000_000, n_queries)
    acc = _min_acc_split(rng, task, rows, T, 0.30)
    return Workload("C3", T, rows, task, slo, acc, window, C3_WINDOW_US,
                    "64 tasks x 256 variants, Zipf(1.1) tasks, SLO log-uniform [1 ms,1 s], "
                    "30 % min-acc above task median, load update every window")


def config_c4(n_queries: int = 1 << 22) -> Workload:
    rng = _rng(4)
    T = 4
    rows = tradeoff_catalog(rng, T, 4096)
    task = rng.integers(0, T, n_queries).astype(np.uint16)
    lat_sorted = [np.sort(rows["lat_us"][rows["task"] == t]) for t in range(T)]
    acc_sorted = [np.sort(rows["acc_bp"][rows["task"] == t]) for t in range(T)]
    u = rng.random(n_queries)
    w = rng.random(n_queries) * C4_ACC_QUANTILE_SCALE
    slo = np.zeros(n_queries, np.uint32)
    acc = np.zeros(n_queries, np.uint16)
    for t in range(T):
        m = task == t
        k = lat_sorted[t].size
        slo[m] = lat_sorted[t][np.minimum(k - 1, (u[m] * k).astype(np.int64))]
        acc[m] = acc_sorted[t][np.minimum(k - 1, (w[m] * k).astype(np.int64))]
    return Workload("C4", T, rows, task, slo, acc, 0, 0,
                    "4 tasks x 4096 variants on a trade-off surface, SLO / min-acc from the "
                    "task's attribute quantiles, about 10 % infeasible")


def config_c5(n_windows: int = 1000, window: int = 65536) -> Workload:
    rng = _rng(5)
    T = 128
    rows = structured_catalog(rng, T, 16, 4, [1, 2, 4, 8, 16, 32, 64, 128])
    perms = [rng.permutation(T), rng.permutation(T)]
    pmf = _zipf_pmf(T, 1.5)
    n = n_windows * window
    task = np.empty(n, np.uint16)
    for w0 in range(0, n_windows, 50):
        w1 = min(n_windows, w0 + 50)
        p = perms[(w0 // 50) % 2]
        task[w0 * window:w1 * window] = p[_draw_categorical(rng, pmf, (w1 - w0) * window)]
    slo = _log_uniform_int(rng, 1000, 1_000_000, n)
    acc = _min_acc_split(rng, task, rows, T, 0.30)
    return Workload("C5", T, rows, task, slo, acc, window, C5_WINDOW_US,
                    "128 tasks x 512 variants, 1000 windows of 65,536 queries, task mix "
                    "switching between two Zipf(1.5) permutations every 50 windows")


# Share of the variants that start Inactive / Active / Overloaded / Interfered in the
# state-aware runs (codes 0..3 as in include/infaas.h).  The paper prints no such mix; it
# says that every variant starts Inactive and is loaded on demand, so most are Inactive.
STATE_MIX = (0.85, 0.05, 0.05, 0.05)


def variant_states(n_variants: int, seed: int = 6, mix=STATE_MIX):
    """A life-cycle state per variant drawn from `mix`, and a loading latency per variant,
    log-uniform over the range the paper prints for its models (Section 2.1: 590 ms - 11 s)."""
    rng = _rng(seed)
    state = np.searchsorted(np.cumsum(mix), rng.random(n_variants), side="right").clip(0, 3).astype(np.uint8)
    load_lat_us = _log_uniform_int(rng, 590_000, 11_000_000, n_variants)
    return state, load_lat_us


CONFIGS = {"C1": config_c1, "C2": config_c2, "C3": config_c3, "C4": config_c4, "C5": config_c5}


def make(name: str, **kw) -> Workload:
    return CONFIGS[name](**kw)
