"""Pins for the CPU oracle: each test checks it against something other than itself --
the paper's worked example, brute force on tiny catalogs, closed forms, library routines,
exact rationals, invariants."""
import itertools
import os

import numpy as np
import pytest

from oracle import OracleCatalog, pred_lat
from paper_1905_13348_b200 import workloads as W
from tests.helpers import (INVALID, NO_FEASIBLE_BIT, feasible_set, py_pred, rows_from,
                           sorted_head)

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def _select(rows, n_tasks, task, slo, acc, queued=None, threads=1):
    o = OracleCatalog(rows, n_tasks)
    if queued is not None:
        o.queued[:] = queued
    return o.select(np.asarray(task, np.uint16), np.asarray(slo, np.uint32),
                    np.asarray(acc, np.uint16), threads)


# -- P1: the worked example of Section 2.2 (Table 2) ---------------------------------------
def test_table2_worked_example():
    names, lat, cost, cases = [], [], [], []
    for line in open(os.path.join(GOLDEN, "table2_example.txt")):
        f = line.split()
        if not f or f[0] == "#":
            continue
        if f[0] == "variant":
            names.append(f[1]); lat.append(int(f[2]) * 1000); cost.append(int(f[3]))
        elif f[0] == "paper":
            cases.append((int(f[1]) * 1000, f[2], None))
        elif f[0] == "implied":
            cases.append((int(f[1]), f[2], f[3] if len(f) > 3 else None))
    assert names == ["A", "B", "C"] and len(cases) == 8
    rows = rows_from([0] * 3, [1] * 3, lat, [7600] * 3, cost)
    for slo, want, miss in cases:
        d = int(_select(rows, 1, [0], [slo], [7000])[0])
        if want == "NONE":
            assert d == (NO_FEASIBLE_BIT | names.index(miss))
        else:
            assert d == names.index(want), (slo, want, d)


# -- P2 / P7: brute force on tiny catalogs against "materialise, sort, take the head" -------
@pytest.mark.parametrize("seed", range(6))
def test_bruteforce_tiny_catalogs(seed):
    rng = np.random.default_rng(100 + seed)
    nv = int(rng.integers(1, 9))
    n_tasks = 2
    rows = rows_from(rng.integers(0, n_tasks, nv), rng.choice([1, 2, 4, 7], nv),
                     rng.integers(1, 40, nv), rng.integers(6990, 7010, nv),
                     rng.integers(1, 4, nv), rng.integers(0, 5, nv))   # many ties on purpose
    queued = rows["queued"].copy()
    preds = sorted({py_pred(int(r["lat_us"]), int(r["queued"]), int(r["batch"])) for r in rows})
    accs = sorted({int(a) for a in rows["acc_bp"]})
    slos = sorted({max(0, p + e) for p in preds for e in (-1, 0, 1)} | {0})
    maccs = sorted({a + e for a in accs for e in (-1, 0, 1)} | {0, 10001, 65535})
    grid = [(t, s, a) for t in range(n_tasks + 1) for s in slos for a in maccs]
    task, slo, acc = (np.array(x) for x in zip(*grid))
    got = _select(rows, n_tasks, task, slo, acc)
    for (t, s, a), d in zip(grid, got):
        want = INVALID if t >= n_tasks else sorted_head(rows, queued, t, s, a)
        assert int(d) == want, (t, s, a, int(d), want)


# -- P3: the four invariants, on a sample of every configuration ---------------------------
@pytest.mark.parametrize("name,kw", [("C1", {}), ("C2", {"n_queries": 20000}),
                                     ("C3", {"n_queries": 20000}), ("C4", {"n_queries": 4000}),
                                     ("C5", {"n_windows": 1, "window": 8192})])
def test_invariants_on_configs(name, kw):
    w = W.make(name, **kw)
    o = OracleCatalog(w.rows, w.n_tasks)
    rng = np.random.default_rng(7)
    o.queued[:] = rng.integers(0, 6, w.n_variants)          # some load everywhere
    d = o.select(w.task, w.slo_us, w.min_acc_bp, 4)
    pred = np.array([py_pred(int(r["lat_us"]), int(q), int(r["batch"]))
                     for r, q in zip(w.rows, o.queued)], np.int64)
    assert np.array_equal(pred.astype(np.uint32), o.pred_lat())
    acc, cost, tk = (w.rows[k].astype(np.int64) for k in ("acc_bp", "cost", "task"))
    by_task = [np.flatnonzero(tk == t) for t in range(w.n_tasks)]
    for q in rng.choice(w.n_queries, 1500, replace=False):
        m = by_task[int(w.task[q])]
        ok = (pred[m] <= int(w.slo_us[q])) & (acc[m] >= int(w.min_acc_bp[q]))
        if d[q] >> 31:
            assert not ok.any()                              # infeasible only if F is empty
            assert (int(d[q]) & 0x7FFFFFFF) in m
        else:
            v = int(d[q])
            assert v in m[ok]                                # chosen is feasible
            assert cost[v] == cost[m[ok]].min()              # nothing feasible is cheaper
    before = o.served_total.copy()
    o.load_update(d, 1000)
    feas = d[(d >> 31) == 0]
    assert int((o.served_total - before).sum()) == feas.size == int(o.counters[0])
    assert int(o.counters[1]) == int(((d >> 31) == 1).sum()) and int(o.counters[2]) == 0


# -- P4: special cases that reduce to library routines --------------------------------------
def test_no_accuracy_constraint_reduces_to_prefix_min():
    rng = np.random.default_rng(11)
    nv = 300
    lat = rng.integers(1000, 100000, nv)
    cost = rng.permutation(nv) + 1                            # distinct costs: unique answer
    rows = rows_from([0] * nv, [1] * nv, lat, rng.integers(5000, 9000, nv), cost)
    slo = rng.integers(500, 120000, 5000)
    got = _select(rows, 1, np.zeros(5000), slo, np.zeros(5000))
    order = np.argsort(lat, kind="stable")
    run_min = np.minimum.accumulate(cost[order])
    k = np.searchsorted(lat[order], slo, side="right")        # variants with lat <= slo
    id_of_cost = np.empty(nv + 1, np.int64); id_of_cost[cost] = np.arange(nv)
    feas = k > 0
    assert np.array_equal(got[feas], id_of_cost[run_min[k[feas] - 1]].astype(np.uint32))
    # nothing meets the SLO, every variant meets the accuracy: nearest miss = fastest variant
    fastest = int(np.lexsort((np.arange(nv), cost, lat))[0])
    assert np.all(got[~feas] == (NO_FEASIBLE_BIT | fastest)) and (~feas).any()


def test_equal_costs_reduce_to_min_latency_and_single_variant():
    rng = np.random.default_rng(12)
    nv = 64
    lat = rng.permutation(nv) * 10 + 100
    rows = rows_from([0] * nv, [1] * nv, lat, [7000] * nv, [5] * nv)
    got = _select(rows, 1, [0] * 3, [10**6, 400, 100], [7000] * 3)
    assert list(got) == [int(np.argmin(lat))] * 3
    one = rows_from([0], [1], [100], [7000], [9])
    got = _select(one, 1, [0] * 4, [100, 99, 100, 99], [7000, 7000, 7001, 7001])
    assert list(got) == [0, NO_FEASIBLE_BIT, NO_FEASIBLE_BIT, NO_FEASIBLE_BIT]


def test_every_variant_meets_latency_nearest_miss_is_max_accuracy():
    rng = np.random.default_rng(13)
    nv = 40
    acc = rng.integers(6000, 7000, nv)
    cost = rng.integers(1, 5, nv)
    lat = rng.integers(10, 50, nv)
    rows = rows_from([0] * nv, [1] * nv, lat, acc, cost)
    got = int(_select(rows, 1, [0], [1000], [9000])[0])
    best = sorted(range(nv), key=lambda v: (-acc[v], cost[v], lat[v], v))[0]
    assert got == (NO_FEASIBLE_BIT | best)


# -- ties: cost, then predicted latency, then accuracy, then id -----------------------------
def test_tie_break_order():
    #            id0   id1   id2   id3   id4
    lat = [300, 200, 200, 200, 200]
    acc = [7000, 7000, 7500, 7500, 7400]
    rows = rows_from([0] * 5, [1] * 5, lat, acc, [4] * 5)
    assert int(_select(rows, 1, [0], [1000], [0])[0]) == 2     # lat 200, acc 7500, lowest id
    rows["cost"][0] = 3
    assert int(_select(rows, 1, [0], [1000], [0])[0]) == 0     # cost wins over latency
    rows["cost"][0] = 4; rows["queued"][:] = [0, 1, 1, 1, 1]    # load doubles 1..4 to 400
    assert int(_select(rows, 1, [0], [1000], [0])[0]) == 0     # predicted, not profiled, latency


# -- ties between nearest misses at equal distance: cost, then predicted latency, then accuracy,
#    then id (the order of the feasible branch, after the distance).  Every case pits two
#    criteria against each other, so that a key with two fields swapped answers differently. --
def test_nearest_miss_tie_break_order():
    def miss(rows, slo, acc):
        d = int(_select(rows, 1, [0], [slo], [acc])[0])
        assert d & NO_FEASIBLE_BIT
        return d & 0x7FFFFFFF
    # both meet the SLO and miss the accuracy by one basis point (d = 100 each):
    # id0 is slower and cheaper, id1 faster and dearer -> cost decides
    rows = rows_from([0, 0], [1, 1], [20, 10], [7000, 7000], [1, 2])
    assert miss(rows, 100, 7001) == 0
    rows = rows_from([0, 0], [1, 1], [10, 20], [7000, 7000], [2, 1])
    assert miss(rows, 100, 7001) == 1
    # one misses the SLO by 1 us (d = 10^4), the other the accuracy by 100 bp at slo 100
    # (d = 10^4): id0 slower and cheaper -> cost decides, not latency
    rows = rows_from([0, 0], [1, 1], [101, 50], [7000, 6900], [1, 2])
    assert miss(rows, 100, 7000) == 0
    rows = rows_from([0, 0], [1, 1], [50, 101], [6900, 7000], [2, 1])
    assert miss(rows, 100, 7000) == 1
    # a strictly smaller distance beats a lower cost
    rows = rows_from([0, 0], [1, 1], [101, 50], [7000, 6901], [1, 9])      # d = 10000, 9900
    assert miss(rows, 100, 7000) == 1
    rows = rows_from([0, 0], [1, 1], [101, 50], [7000, 6899], [9, 1])      # d = 10000, 10100
    assert miss(rows, 100, 7000) == 0
    # equal distance and cost: the faster one, although it is the less accurate and has the higher id
    rows = rows_from([0, 0], [1, 1], [101, 60], [7000, 6900], [3, 3])
    assert miss(rows, 100, 7000) == 1
    # equal distance, cost and latency (both miss the SLO only): higher accuracy, then lower id
    rows = rows_from([0, 0, 0], [1, 1, 1], [150, 150, 150], [7100, 7300, 7300], [3, 3, 3])
    assert miss(rows, 100, 7000) == 1
    # predicted latency, not the profiled one, enters both the distance and the tie
    rows = rows_from([0, 0], [1, 1], [30, 50], [7000, 7000], [4, 4], [1, 0])   # pred 60, 50
    assert miss(rows, 100, 7001) == 1


# -- P5: permuting the catalog rows (ids carried along) permutes the answers ---------------
def test_row_permutation_equivariance():
    w = W.make("C2", n_queries=5000)
    d0 = _select(w.rows, w.n_tasks, w.task, w.slo_us, w.min_acc_bp, threads=3)
    perm = np.random.default_rng(5).permutation(w.n_variants)
    d1 = _select(w.rows[perm], w.n_tasks, w.task, w.slo_us, w.min_acc_bp)
    flag, idx = d1 & NO_FEASIBLE_BIT, d1 & 0x7FFFFFFF
    r0, r1 = w.rows[d0 & 0x7FFFFFFF], w.rows[perm][idx]
    assert np.array_equal(flag, d0 & NO_FEASIBLE_BIT)
    for k in ("cost", "lat_us", "acc_bp", "batch", "queued"):   # same variant up to id ties
        assert np.array_equal(r0[k], r1[k])


# -- P6: monotonicity --------------------------------------------------------------------
def test_monotone_in_slo_and_accuracy():
    w = W.make("C2", n_queries=4000)
    cost = w.rows["cost"].astype(np.int64)
    d0 = _select(w.rows, w.n_tasks, w.task, w.slo_us, w.min_acc_bp)
    d1 = _select(w.rows, w.n_tasks, w.task, w.slo_us + 5000, np.maximum(w.min_acc_bp, 50) - 50)
    f0, f1 = (d0 >> 31) == 0, (d1 >> 31) == 0
    assert np.all(f1[f0])                                     # feasible stays feasible
    assert np.all(cost[d1[f0]] <= cost[d0[f0]])               # and never gets dearer
    # loading the chosen variants never lowers the cost of the choice
    queued = w.rows["queued"].copy(); queued[np.unique(d0[f0])] += 50
    d2 = _select(w.rows, w.n_tasks, w.task, w.slo_us, w.min_acc_bp, queued=queued)
    both = f0 & ((d2 >> 31) == 0)
    assert np.all(cost[d2[both]] >= cost[d0[both]])


# -- P8: tallies are a histogram; the queue follows the closed form under constant arrivals --
def test_tally_is_bincount_and_queue_closed_form():
    rows = rows_from([0, 0, 0], [2, 1, 4], [1000, 500, 100], [7000] * 3, [1, 2, 3], [10, 0, 7])
    o = OracleCatalog(rows, 1)
    rng = np.random.default_rng(3)
    dec = rng.choice(np.array([0, 1, 2, NO_FEASIBLE_BIT | 1, INVALID, 17], np.uint32), 1000)
    o.load_update(dec, 1)                                     # drain = floor(batch/lat) = 0
    assert np.array_equal(o.served_total, np.bincount(dec[dec < 3], minlength=3))
    assert list(o.counters) == [int((dec < 3).sum()), int((dec == (NO_FEASIBLE_BIT | 1)).sum()),
                                int((dec == INVALID).sum() + (dec == 17).sum())]
    # constant arrivals a per window, drain r per window: queued_k = max(0, q0 + k (a - r))
    o = OracleCatalog(rows, 1)
    window_us = 2500                                          # r = floor(2500*b/lat) = 5, 5, 100
    arrivals = np.array([0] * 8 + [1] * 3 + [2] * 60, np.uint32)   # a = 8, 3, 60
    q0, a, r = np.array([10, 0, 7]), np.array([8, 3, 60]), np.array([5, 5, 100])
    for k in range(1, 6):
        o.load_update(arrivals, window_us)
        assert np.array_equal(o.queued, np.maximum(0, q0 + k * (a - r))[:2].tolist()
                              + [max(0, 7 + 60 - 100)] * (k == 1) + [0] * (k > 1))


# -- P9: arithmetic edges ----------------------------------------------------------------
def test_pred_lat_against_python_integers_and_saturation():
    rng = np.random.default_rng(4)
    cases = [(1, 0, 1), (1, 2**32 - 1, 65535), (2**32 - 1, 2**32 - 1, 1), (2**32 - 1, 1, 65535),
             (5, 7, 2), (5, 8, 2), (3, 1, 2)]
    cases += [(int(l), int(q), int(b)) for l, q, b in
              zip(rng.integers(1, 2**32, 200), rng.integers(0, 2**32, 200), rng.integers(1, 65536, 200))]
    for lat, q, b in cases:
        assert pred_lat(lat, q, b) == py_pred(lat, q, b)
    assert pred_lat(5, 7, 2) == 5 + 17 and pred_lat(2**31, 3, 1) == 2**32 - 1


def test_saturating_queue_and_extreme_queries():
    rows = rows_from([0, 0], [1, 65535], [2**32 - 1, 1], [0, 10000], [2**32 - 1, 1],
                     [2**32 - 2, 5])
    o = OracleCatalog(rows, 1)
    o.load_update(np.zeros(10, np.uint32), 0)                 # queued + count saturates
    assert int(o.queued[0]) == 2**32 - 1
    o.load_update(np.zeros(0, np.uint32), 2**32 - 1)          # drain(0) = 1, drain(1) saturates
    assert list(o.queued) == [2**32 - 2, 0]
    d = o.select(np.array([0, 0, 0, 1], np.uint16), np.array([0, 2**32 - 1, 1, 5], np.uint32),
                 np.array([0, 10001, 10000, 0], np.uint16))
    assert list(d) == [NO_FEASIBLE_BIT | 1, NO_FEASIBLE_BIT | 1, 1, INVALID]


# -- the pruned list behind the benchmark's scan-operation count: checked against the dominance
#    definition in plain Python, and against the brute-force oracle (first feasible entry of the
#    list = the oracle's decision, which never prunes) ---------------------------------------
@pytest.mark.parametrize("seed", range(4))
def test_frontier_and_scan_ops(seed):
    rng = np.random.default_rng(900 + seed)
    nv, n_tasks = int(rng.integers(20, 60)), 2
    rows = rows_from(rng.integers(0, n_tasks, nv), rng.choice([1, 2, 4], nv), rng.integers(1, 30, nv),
                     rng.integers(6995, 7005, nv), rng.integers(1, 6, nv), rng.integers(0, 4, nv))
    o = OracleCatalog(rows, n_tasks)
    pred = [py_pred(int(r["lat_us"]), int(r["queued"]), int(r["batch"])) for r in rows]
    attr = [(pred[v], -int(rows["acc_bp"][v]), int(rows["cost"][v])) for v in range(nv)]

    def dominates(a, b):
        return a != b and all(x <= y for x, y in zip(attr[a], attr[b])) and (attr[a] != attr[b] or a < b)

    lists = []
    for t in range(n_tasks):
        mem = [v for v in range(nv) if int(rows["task"][v]) == t]
        want = sorted([b for b in mem if not any(dominates(a, b) for a in mem)],
                      key=lambda v: (attr[v][2], attr[v][0], attr[v][1], v))
        got = [int(x) for x in o.frontier(t)]
        assert got == want
        lists.append(got)
    n = 3000
    task = rng.integers(0, n_tasks + 1, n).astype(np.uint16)
    slo, acc = rng.integers(0, 70, n).astype(np.uint32), rng.integers(6990, 7010, n).astype(np.uint16)
    d = o.select(task, slo, acc)
    ops, pos = o.scan_ops(task, d, want_pos=True)
    total = 0
    for q in range(n):
        if task[q] >= n_tasks or d[q] == INVALID:
            assert pos[q] == 0xFFFFFFFF
            continue
        L = lists[int(task[q])]
        first = next((i for i, v in enumerate(L) if pred[v] <= slo[q] and rows["acc_bp"][v] >= acc[q]), None)
        if d[q] >> 31:
            assert first is None and pos[q] == 0xFFFFFFFF
            total += 9 * len(L)
        else:
            assert first is not None and L[first] == int(d[q]) and pos[q] == first
            total += 96 * (first // 32 + 1)
    assert ops == total
