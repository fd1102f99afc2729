"""Small independent checkers used by the CPU tests (plain Python, tiny inputs only)."""
from fractions import Fraction

import numpy as np

from paper_1905_13348_b200.workloads import VARIANT_DTYPE

NO_FEASIBLE_BIT = 0x80000000
INVALID = 0xFFFFFFFF


def rows_from(task, batch, lat_us, acc_bp, cost, queued=None):
    n = len(task)
    r = np.zeros(n, VARIANT_DTYPE)
    r["task"], r["batch"], r["lat_us"], r["acc_bp"], r["cost"] = task, batch, lat_us, acc_bp, cost
    if queued is not None:
        r["queued"] = queued
    return r


def py_pred(lat, queued, batch):
    return min(2**32 - 1, lat + (queued * lat) // batch)


def feasible_set(rows, queued, t, slo, min_acc):
    """Materialised feasible set of one query, as python ints."""
    out = []
    for v in range(len(rows)):
        if int(rows["task"][v]) != t:
            continue
        p = py_pred(int(rows["lat_us"][v]), int(queued[v]), int(rows["batch"][v]))
        if p <= slo and int(rows["acc_bp"][v]) >= min_acc:
            out.append(v)
    return out


def sorted_head(rows, queued, t, slo, min_acc):
    """Plain restatement by sorting: materialise, sort, take the head.

    Feasible set non-empty: sort it by (cost, pred, -acc, id).  Empty: sort all of the
    task's variants by the exact rational miss  over_lat/slo + under_acc/10^4  (slo > 0)
    and then by the same tuple; return the head with bit 31 set."""
    members = [v for v in range(len(rows)) if int(rows["task"][v]) == t]
    if not members:
        return INVALID

    def attrs(v):
        p = py_pred(int(rows["lat_us"][v]), int(queued[v]), int(rows["batch"][v]))
        return p, int(rows["acc_bp"][v]), int(rows["cost"][v])

    F = feasible_set(rows, queued, t, slo, min_acc)
    if F:
        return sorted(F, key=lambda v: (attrs(v)[2], attrs(v)[0], -attrs(v)[1], v))[0]

    def miss(v):
        p, a, c = attrs(v)
        over, under = max(0, p - slo), max(0, min_acc - a)
        if slo > 0:
            m = Fraction(over, slo) + Fraction(under, 10000)
        else:
            m = Fraction(10000 * over)          # accuracy term vanishes at slo = 0
        return (m, c, p, -a, v)

    return NO_FEASIBLE_BIT | sorted(members, key=miss)[0]


def sorted_head_stateful(rows, queued, state, load_lat, t, slo, min_acc):
    """State-aware selection restated by materialising and sorting three sets.

    Active matches sorted by (cost, pred, -acc, id); else Inactive matches (latency = pred +
    loading latency, capped at 2^32-1) sorted by (that latency, -acc, id); else every Active
    or Inactive variant of the task sorted by the exact rational miss, Active before
    Inactive on equal miss, then by the same tuples.  States: 0 Inactive, 1 Active; other
    values are skipped."""
    act, ina = [], []
    for v in range(len(rows)):
        if int(rows["task"][v]) != t or int(state[v]) not in (0, 1):
            continue
        p = py_pred(int(rows["lat_us"][v]), int(queued[v]), int(rows["batch"][v]))
        a, c = int(rows["acc_bp"][v]), int(rows["cost"][v])
        if int(state[v]) == 1:
            act.append((v, p, a, (c, p, -a, v)))
        else:
            e = min(2**32 - 1, p + int(load_lat[v]))
            ina.append((v, e, a, (e, -a, v)))
    if not act and not ina:
        return INVALID
    for group in (act, ina):
        ok = [x for x in group if x[1] <= slo and x[2] >= min_acc]
        if ok:
            return sorted(ok, key=lambda x: x[3])[0][0]

    def miss(x, cls):
        over, under = max(0, x[1] - slo), max(0, min_acc - x[2])
        m = Fraction(over, slo) + Fraction(under, 10000) if slo > 0 else Fraction(10000 * over)
        return (m, cls) + x[3]

    cand = [(miss(x, 0), x[0]) for x in act] + [(miss(x, 1), x[0]) for x in ina]
    return NO_FEASIBLE_BIT | sorted(cand)[0][1]
