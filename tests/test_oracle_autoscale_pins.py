"""Pins for the Model-Autoscaler step of the CPU oracle (Section 4.2.1 cost function and
constraints, Section 4.2.2 scaling-up algorithm): the worked example of Tables 2 and 3, a
restatement by enumeration with exact rationals, invariants, closed forms, saturation."""
import os
from fractions import Fraction

import numpy as np
import pytest

from oracle import AUTOSCALE_ESCALATE, AUTOSCALE_NONE, autoscale_step
from tests.helpers import rows_from

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def _rows(task, batch, lat_us, cost, arch):
    r = rows_from(task, batch, lat_us, [7000] * len(task), cost)
    r["arch"] = arch
    return r


# -- Tables 2 and 3 ---------------------------------------------------------------------------
def test_table3_worked_example():
    names, lat, rps, cost, paper, steps = [], [], [], [], [], []
    for line in open(os.path.join(GOLDEN, "table3_example.txt")):
        f = line.split()
        if not f or f[0] == "#":
            continue
        if f[0] == "variant":
            names.append(f[1]); lat.append(int(f[2]) * 1000); rps.append(int(f[3])); cost.append(int(f[4]))
        elif f[0] == "paper":
            paper.append([int(x) for x in f[1:]])
        elif f[0] == "step":
            steps.append(([int(x) for x in f[1:6]], f[6], int(f[7])))
    assert names == ["A", "B", "C"] and len(paper) == len(steps) == 3
    # batch sizes that give Table 2's saturation throughput at Table 2's latency
    batch = [r * l // 10**6 for r, l in zip(rps, lat)]
    assert [b * 10**6 // l for b, l in zip(batch, lat)] == rps
    rows = _rows([0] * 3, batch, lat, cost, [5] * 3)
    for (qps, slo_ms, *running), want_name, want_delta in steps:
        count = np.zeros(3, np.uint32)
        if any(running):
            count[int(np.argmax(running))] = qps            # one second of this load
        else:
            count[0] = qps                                   # served by nobody who still meets the SLO
        v, d = autoscale_step(rows, 1, count, running, [0] * 3, [slo_ms * 1000], 10**6, 100, 0)
        assert (names[int(v[0])], int(d[0])) == (want_name, want_delta)
        after = list(running); after[int(v[0])] += int(d[0])
        row = next(p for p in paper if p[0] == qps and p[1] == slo_ms)
        assert after == row[2:5] and sum(a * c for a, c in zip(after, cost)) == row[5]
        # the configuration reached sustains the load: no further action
        v2, d2 = autoscale_step(rows, 1, count, after, [0] * 3, [slo_ms * 1000], 10**6, 100, 0)
        assert int(v2[0]) == AUTOSCALE_NONE and int(d2[0]) == 0


# -- restatement by enumeration, exact rationals ------------------------------------------------
def plain_step(rows, count, inst, load, slo, window_us, slack_pct, lam_milli):
    """One task.  Instances are added one at a time until the capacity reaches the need."""
    nv = len(rows)
    q = [Fraction(int(rows["batch"][v]) * 10**9 // int(rows["lat_us"][v])) for v in range(nv)]
    served = min(2**32 - 1, int(sum(int(c) for c in count)))
    L = served * 10**9 // window_us
    need = Fraction(-(-L * slack_pct // 100))
    cap = sum(int(inst[v]) * q[v] for v in range(nv))
    if cap >= need:
        return AUTOSCALE_NONE, 0
    running = [v for v in range(nv) if inst[v] > 0]
    r = max(running, key=lambda v: (int(count[v]), -v)) if running else None
    options = []
    for v in range(nv):
        if int(rows["lat_us"][v]) > slo or q[v] == 0:
            continue
        if r is not None and v != r and (rows["arch"][v] != rows["arch"][r] or q[v] <= q[r]):
            continue
        delta = 0
        while cap + delta * q[v] < need:
            delta += 1
            if delta > 200000:
                break
        else:
            price = int(rows["cost"][v]) * (delta + Fraction(lam_milli, 1000) * Fraction(int(load[v]), 10**6) * delta)
            options.append((price, 0 if v == r else 1, v, delta))
    if not options:
        return AUTOSCALE_ESCALATE, 0
    best = min(options)
    return best[2], best[3]


@pytest.mark.parametrize("seed", range(12))
def test_enumeration_on_small_tasks(seed):
    # few distinct values on purpose: equal throughputs, equal tallies, latencies on the SLO
    rng = np.random.default_rng(300 + seed)
    nv = int(rng.integers(1, 9))
    rows = _rows([0] * nv, rng.choice([1, 2, 4, 8], nv), rng.choice([20_000, 40_000, 80_000, 333_333], nv),
                 rng.integers(1, 6, nv), rng.integers(0, 2, nv))
    load = rng.integers(0, 3_000_000, nv)
    for _ in range(60):
        inst = rng.integers(0, 3, nv) * (rng.random(nv) < 0.5)
        count = rng.choice([0, 7, 7, 90, 400], nv)
        slo = int(rng.choice([19_999, 20_000, 40_000, 80_000, 400_000]))
        slack, lam = int(rng.choice([100, 105, 150])), int(rng.choice([0, 50, 5000]))
        window_us = int(rng.choice([1_000_000, 999_983, 31_337]))
        v, d = autoscale_step(rows, 1, count, inst, load, [slo], window_us, slack, lam)
        assert (int(v[0]), int(d[0])) == plain_step(rows, count, inst, load, slo, window_us, slack, lam)


# -- invariants on a larger catalog -------------------------------------------------------------
def test_invariants_many_tasks():
    rng = np.random.default_rng(41)
    T, nv = 12, 400
    task = rng.integers(0, T - 1, nv)                          # the last task has no variants
    rows = _rows(task, rng.choice([1, 2, 4, 8, 16, 32], nv), rng.integers(1500, 2_000_000, nv),
                 rng.integers(1, 500, nv), rng.integers(0, 4, nv))
    load = rng.integers(590_000, 11_000_000, nv)
    inst = rng.integers(0, 4, nv) * (rng.random(nv) < 0.2)
    count = (rng.integers(0, 3000, nv) * (inst > 0)).astype(np.uint32)
    slo = rng.integers(2000, 1_000_000, T)
    window_us = 250_000
    v, d = autoscale_step(rows, T, count, inst, load, slo, window_us, 105, 100)
    q = rows["batch"].astype(object) * 10**9 // rows["lat_us"].astype(object)
    kinds = set()
    for t in range(T):
        m = np.flatnonzero(task == t)
        need = -(-(int(count[m].sum()) * 10**9 // window_us) * 105 // 100)
        cap = int(sum(int(inst[x]) * int(q[x]) for x in m))
        if cap >= need:
            assert int(v[t]) == AUTOSCALE_NONE and int(d[t]) == 0
            kinds.add("none")
        elif int(v[t]) == AUTOSCALE_ESCALATE:
            assert int(d[t]) == 0
            kinds.add("escalate")
        else:
            x, dl = int(v[t]), int(d[t])
            assert x in m and rows["lat_us"][x] <= slo[t] and dl >= 1
            assert cap + dl * int(q[x]) >= need > cap + (dl - 1) * int(q[x])   # just enough
            kinds.add("act")
    assert int(v[T - 1]) == AUTOSCALE_NONE                       # nothing served, nothing needed
    assert kinds == {"none", "escalate", "act"}, kinds


# -- the weight on the loading latency flips the choice where the formula says so ---------------
def test_lambda_threshold():
    # r = id0 runs; id1 and id2 are faster variants of its architecture, id3 of another one
    rows = _rows([0] * 4, [1, 4, 4, 64], [100_000] * 4, [2, 7, 8, 1], [1, 1, 1, 2])   # Q = 10, 40, 40, 640 /s
    inst, count, load = [1, 0, 0, 0], [50, 0, 0, 0], [0, 4_000_000, 1_000_000, 0]
    # need 50/s, capacity 10/s, deficit 40/s: replicate id0 4x (cost 8), or 1x id1 (7), or 1x id2 (8)
    pick = lambda lam: tuple(int(a[0]) for a in autoscale_step(rows, 1, count, inst, load, [200_000], 10**6, 100, lam))
    assert pick(0) == (1, 1)
    # id1: 7 (1 + 4 lam), id2: 8 (1 + lam), id0: 8 -- id1 wins while 7 + 28 lam < 8, i.e. lam < 1/28
    assert pick(35) == (1, 1) and pick(36) == (0, 4)
    assert autoscale_step(rows, 1, count, inst, load, [99_999], 10**6, 100, 0)[0][0] == AUTOSCALE_ESCALATE
    rows["arch"][3] = 1                                             # now id3 qualifies: 1 instance, cost 1
    assert pick(0) == (3, 1)
    # equal cost: replication before an upgrade, then the lower id
    rows2 = _rows([0] * 3, [1, 4, 4], [100_000] * 3, [2, 8, 8], [1, 1, 1])
    assert tuple(int(a[0]) for a in autoscale_step(rows2, 1, [50, 0, 0], [1, 0, 0], [0] * 3, [200_000], 10**6, 100, 0)) == (0, 4)
    rows2["cost"][0] = 5                                            # nothing runs: 5 x id0 = 25, 2 x id1 = 2 x id2 = 16
    assert tuple(int(a[0]) for a in autoscale_step(rows2, 1, [50, 0, 0], [0, 0, 0], [0] * 3, [200_000], 10**6, 100, 0)) == (1, 2)


# -- saturating arithmetic ----------------------------------------------------------------------
def test_saturation_edges():
    rows = _rows([0, 0], [65535, 1], [1, 2**32 - 1], [1, 1], [0, 0])   # Q = 6.5e13 and 0 milli-queries/s
    big = 2**32 - 1
    # capacity 2^32-1 instances x 6.5e13 saturates at 2^64-1 and covers any need
    v, d = autoscale_step(rows, 1, [big, big], [big, 0], [0, 0], [10], 1, 1000, 0)
    assert int(v[0]) == AUTOSCALE_NONE
    # served saturates at 2^32-1 queries; at window 1 us the need is far above one instance's worth
    v, d = autoscale_step(rows, 1, [big, big], [1, 0], [0, 0], [10], 1, 100, 0)
    L = (2**32 - 1) * 10**9
    assert int(v[0]) == 0 and int(d[0]) == -(-(L - 65535 * 10**9) // (65535 * 10**9))
    # a variant whose saturation throughput rounds to zero can never cover a deficit
    v, d = autoscale_step(rows, 1, [0, 5], [0, 1], [0, 0], [2**32 - 1], 10**6, 100, 0)
    assert (int(v[0]), int(d[0])) == (0, 1)                         # nothing else of its architecture is barred: id0 qualifies
    rows["arch"][0] = 9
    v, d = autoscale_step(rows, 1, [0, 5], [0, 1], [0, 0], [2**32 - 1], 10**6, 100, 0)
    assert int(v[0]) == AUTOSCALE_ESCALATE


def test_need_is_rounded_up():
    # Q = 1 milli-query/s per instance; L = floor(10^9 / 3) = 333,333,333; x 1.01 = 336,666,666.33
    rows = _rows([0], [1], [10**9], [1], [0])
    for inst, want in ((336_666_666, (0, 1)), (336_666_667, (AUTOSCALE_NONE, 0)), (336_666_000, (0, 667))):
        v, d = autoscale_step(rows, 1, [1], [inst], [0], [2**32 - 1], 3, 101, 0)
        assert (int(v[0]), int(d[0])) == want


# -- monotone in the load and in what already runs -------------------------------------------------
def test_more_load_never_needs_less_and_more_instances_never_need_more():
    rng = np.random.default_rng(43)
    nv = 40
    rows = _rows([0] * nv, rng.choice([1, 2, 4, 8], nv), rng.integers(2000, 200000, nv), rng.integers(1, 50, nv), [3] * nv)
    inst = np.zeros(nv, np.uint32); inst[5] = 2
    load = np.zeros(nv, np.uint32)
    prev = 0
    for served in (0, 10, 100, 1000, 10000, 100000):
        count = np.zeros(nv, np.uint32); count[5] = served
        v, d = autoscale_step(rows, 1, count, inst, load, [10**6], 10**6, 105, 0)
        cost = 0 if int(v[0]) >= AUTOSCALE_ESCALATE else int(rows["cost"][int(v[0])]) * int(d[0])
        assert cost >= prev
        prev = cost
    assert prev > 0
    count = np.zeros(nv, np.uint32); count[5] = 100000
    prev = None
    for n in (1, 2, 8, 64, 10**6):
        inst[5] = n
        v, d = autoscale_step(rows, 1, count, inst, load, [10**6], 10**6, 105, 0)
        cost = 0 if int(v[0]) >= AUTOSCALE_ESCALATE else int(rows["cost"][int(v[0])]) * int(d[0])
        assert prev is None or cost <= prev
        prev = cost
    assert prev == 0 and int(v[0]) == AUTOSCALE_NONE
