"""Pins for the state-aware part of the CPU oracle (Section 4, state machine; Section 4.1,
Case I): reductions to the stateless oracle (itself pinned in test_oracle_pins.py), brute
force against a sort-based restatement, a library routine, invariants, closed forms."""
import numpy as np
import pytest

from oracle import (ACTIVE, INACTIVE, INTERFERED, OVERLOADED, OracleCatalog,
                    StatefulOracleCatalog)
from paper_1905_13348_b200 import workloads as W
from tests.helpers import (INVALID, NO_FEASIBLE_BIT, py_pred, rows_from, sorted_head_stateful)


def _random_states(rng, n, p=(0.35, 0.45, 0.1, 0.1)):
    return rng.choice(np.array([INACTIVE, ACTIVE, OVERLOADED, INTERFERED], np.uint8), n, p=p)


# -- all variants Active: the loading latency plays no part, answers = stateless oracle -------
def test_all_active_equals_stateless():
    w = W.make("C2", n_queries=6000)
    rng = np.random.default_rng(1)
    s = StatefulOracleCatalog(w.rows, w.n_tasks, np.full(w.n_variants, ACTIVE),
                              rng.integers(0, 10**6, w.n_variants))
    o = OracleCatalog(w.rows, w.n_tasks)
    assert np.array_equal(s.select(w.task, w.slo_us, w.min_acc_bp, 3),
                          o.select(w.task, w.slo_us, w.min_acc_bp, 3))


# -- all variants Inactive: the stateless oracle on a catalog whose latency and cost are both
#    the combined loading + inference latency gives the same answers (its key (cost, pred,
#    -acc, id) is then (combined, combined, -acc, id), its distance uses the combined latency)
def test_all_inactive_equals_stateless_on_combined_latency():
    w = W.make("C2", n_queries=6000)
    rng = np.random.default_rng(2)
    load = rng.integers(0, 300000, w.n_variants).astype(np.uint32)
    s = StatefulOracleCatalog(w.rows, w.n_tasks, np.full(w.n_variants, INACTIVE), load)
    pred = np.array([py_pred(int(r["lat_us"]), int(r["queued"]), int(r["batch"])) for r in w.rows])
    rows2 = w.rows.copy()
    rows2["lat_us"] = pred + load; rows2["queued"] = 0; rows2["cost"] = pred + load
    o = OracleCatalog(rows2, w.n_tasks)
    got = s.select(w.task, w.slo_us, w.min_acc_bp, 3)
    assert np.array_equal(got, o.select(w.task, w.slo_us, w.min_acc_bp, 3))
    assert ((got >> 31) == 0).any() and ((got >> 31) == 1).any()


# -- all Inactive, no accuracy requirement: lowest combined latency = sort + searchsorted -----
def test_inactive_without_accuracy_is_min_combined_latency():
    rng = np.random.default_rng(3)
    nv = 200
    lat = rng.permutation(nv) * 7 + 50
    load = rng.permutation(nv) * 1000
    rows = rows_from([0] * nv, [1] * nv, lat, rng.integers(5000, 9000, nv), rng.integers(1, 9, nv))
    s = StatefulOracleCatalog(rows, 1, np.zeros(nv), load)
    comb = lat + load
    best = int(np.argmin(comb))
    assert np.unique(comb).size == nv                           # so the answer is unique
    slo = rng.integers(0, comb.max() + 10, 500).astype(np.uint32)
    got = s.select(np.zeros(500, np.uint16), slo, np.zeros(500, np.uint16))
    feas = np.searchsorted(np.sort(comb), slo, side="right") > 0
    assert np.all(got[feas] == best) and np.all(got[~feas] == (NO_FEASIBLE_BIT | best))
    assert feas.any() and (~feas).any()


# -- brute force on tiny catalogs against "materialise three sets, sort, take the head" --------
@pytest.mark.parametrize("seed", range(8))
def test_bruteforce_tiny_catalogs_stateful(seed):
    rng = np.random.default_rng(200 + seed)
    nv = int(rng.integers(1, 10))
    n_tasks = 2
    rows = rows_from(rng.integers(0, n_tasks, nv), rng.choice([1, 2, 4, 7], nv),
                     rng.integers(1, 40, nv), rng.integers(6990, 7010, nv),
                     rng.integers(1, 4, nv), rng.integers(0, 5, nv))
    state = _random_states(rng, nv, (0.4, 0.4, 0.1, 0.1))
    load = rng.integers(0, 30, nv).astype(np.uint32)
    load[rng.random(nv) < 0.1] = 2**32 - 1                       # the sum saturates
    s = StatefulOracleCatalog(rows, n_tasks, state, load)
    lats = set()
    for v in range(nv):
        p = py_pred(int(rows["lat_us"][v]), int(rows["queued"][v]), int(rows["batch"][v]))
        lats |= {p, min(2**32 - 1, p + int(load[v]))}
    slos = sorted({min(2**32 - 1, max(0, x + e)) for x in lats for e in (-1, 0, 1)} | {0})
    maccs = sorted({int(a) + e for a in rows["acc_bp"] for e in (-1, 0, 1)} | {0, 10001, 65535})
    grid = [(t, x, a) for t in range(n_tasks + 1) for x in slos for a in maccs]
    task, slo, acc = (np.array(x) for x in zip(*grid))
    got = s.select(task, slo, acc)
    for (t, x, a), d in zip(grid, got):
        want = INVALID if t >= n_tasks else sorted_head_stateful(rows, rows["queued"], state, load, t, x, a)
        assert int(d) == want, (t, x, a, int(d), want)


# -- invariants on a workload-shaped catalog ----------------------------------------------------
def test_stateful_invariants():
    w = W.make("C3", n_queries=20000)
    rng = np.random.default_rng(4)
    state = _random_states(rng, w.n_variants, (0.75, 0.05, 0.1, 0.1))
    load = rng.integers(1000, 100_000, w.n_variants).astype(np.uint32)
    s = StatefulOracleCatalog(w.rows, w.n_tasks, state, load)
    s.queued[:] = rng.integers(0, 6, w.n_variants)
    d = s.select(w.task, w.slo_us, w.min_acc_bp, 4)
    pred = s.pred_lat().astype(np.int64)
    acc, cost, tk = (w.rows[k].astype(np.int64) for k in ("acc_bp", "cost", "task"))
    eff = np.minimum(2**32 - 1, pred + load)
    by_task = [np.flatnonzero(tk == t) for t in range(w.n_tasks)]
    seen = {"active": 0, "inactive": 0, "miss": 0}
    for q in rng.choice(w.n_queries, 2000, replace=False):
        m = by_task[int(w.task[q])]
        slo, ma = int(w.slo_us[q]), int(w.min_acc_bp[q])
        ok_a = m[(state[m] == ACTIVE) & (pred[m] <= slo) & (acc[m] >= ma)]
        ok_i = m[(state[m] == INACTIVE) & (eff[m] <= slo) & (acc[m] >= ma)]
        v = int(d[q]) & 0x7FFFFFFF
        assert state[v] in (ACTIVE, INACTIVE)                    # never Overloaded / Interfered
        if ok_a.size:                                            # an Active match wins, cheapest
            assert d[q] >> 31 == 0 and v in ok_a and cost[v] == cost[ok_a].min()
            seen["active"] += 1
        elif ok_i.size:                                          # else the quickest Inactive match
            assert d[q] >> 31 == 0 and v in ok_i and eff[v] == eff[ok_i].min()
            seen["inactive"] += 1
        else:
            assert d[q] >> 31 == 1 and v in m
            seen["miss"] += 1
    assert min(seen.values()) > 20, seen
    # what Overloaded / Interfered variants look like is irrelevant; so is dropping them
    rows2 = w.rows.copy()
    off = np.isin(state, (OVERLOADED, INTERFERED))
    rows2["cost"][off] = 1; rows2["lat_us"][off] = 1; rows2["acc_bp"][off] = 10000
    s2 = StatefulOracleCatalog(rows2, w.n_tasks, state, load); s2.queued[:] = s.queued
    assert np.array_equal(d, s2.select(w.task, w.slo_us, w.min_acc_bp, 4))
    keep = np.flatnonzero(~off)
    s3 = StatefulOracleCatalog(w.rows[keep], w.n_tasks, state[keep], load[keep]); s3.queued[:] = s.queued[keep]
    d3 = s3.select(w.task, w.slo_us, w.min_acc_bp, 4)
    assert np.array_equal(d3 & NO_FEASIBLE_BIT, d & NO_FEASIBLE_BIT)
    assert np.array_equal(keep[d3 & 0x7FFFFFFF], d & 0x7FFFFFFF)


# -- equal distance: an Active variant is suggested before an Inactive one ----------------------
def test_suggestion_prefers_active_on_equal_distance():
    rows = rows_from([0, 0], [1, 1], [100, 60], [7000, 7000], [5, 1])
    # id0 Active with latency 100; id1 Inactive with 60 + loading latency
    s = StatefulOracleCatalog(rows, 1, [ACTIVE, INACTIVE], [0, 40])
    assert int(s.select([0], [50], [7000])[0]) == (NO_FEASIBLE_BIT | 0)    # both miss by 50 us
    s = StatefulOracleCatalog(rows, 1, [ACTIVE, INACTIVE], [0, 39])
    assert int(s.select([0], [50], [7000])[0]) == (NO_FEASIBLE_BIT | 1)    # id1 misses by 49
    s = StatefulOracleCatalog(rows, 1, [ACTIVE, INACTIVE], [0, 40])
    assert int(s.select([0], [100], [7000])[0]) == 0                         # Active match first
    assert int(s.select([0], [100], [7001])[0]) == (NO_FEASIBLE_BIT | 0)
    s = StatefulOracleCatalog(rows, 1, [OVERLOADED, INACTIVE], [0, 40])
    assert int(s.select([0], [100], [7000])[0]) == 1                         # the only selectable match
    s = StatefulOracleCatalog(rows, 1, [OVERLOADED, INTERFERED], [0, 40])
    assert int(s.select([0], [100], [7000])[0]) == INVALID


# -- equal distance inside one class: Active by (cost, latency, accuracy, id), Inactive by
#    (combined latency, accuracy, id); every case sets two criteria against each other ---------
def test_suggestion_tie_break_order_inside_a_class():
    def miss(rows, state, load, slo, acc):
        d = int(StatefulOracleCatalog(rows, 1, state, load).select([0], [slo], [acc])[0])
        assert d & NO_FEASIBLE_BIT
        return d & 0x7FFFFFFF
    A, I = ACTIVE, INACTIVE
    # Active pair, both miss the accuracy by 1 bp: slower and cheaper wins (cost before latency)
    rows = rows_from([0, 0], [1, 1], [20, 10], [7000, 7000], [1, 2])
    assert miss(rows, [A, A], [0, 0], 100, 7001) == 0
    # Active pair, one over the SLO by 1 us, one under the accuracy by 100 bp at slo 100
    rows = rows_from([0, 0], [1, 1], [101, 50], [7000, 6900], [1, 2])
    assert miss(rows, [A, A], [0, 0], 100, 7000) == 0
    rows = rows_from([0, 0], [1, 1], [50, 101], [6900, 7000], [2, 1])
    assert miss(rows, [A, A], [0, 0], 100, 7000) == 1
    # the same pair Inactive: the quicker one wins although it is dearer and less accurate
    rows = rows_from([0, 0], [1, 1], [101, 50], [7000, 6900], [1, 2])
    assert miss(rows, [I, I], [0, 0], 100, 7000) == 1
    # ... through the loading latency too: 40 + 61 against 30 + 20
    rows = rows_from([0, 0], [1, 1], [40, 30], [7000, 6900], [1, 2])
    assert miss(rows, [I, I], [61, 20], 100, 7000) == 1
    # Inactive, equal distance and combined latency: higher accuracy before lower id, cost ignored
    rows = rows_from([0, 0, 0], [1, 1, 1], [150, 100, 150], [7100, 7300, 7300], [1, 9, 9])
    assert miss(rows, [I, I, I], [0, 50, 0], 100, 7000) == 1
    # Inactive pair, both miss the accuracy by 1 bp at the same distance: lower combined latency
    # first, although the other one is the more accurate... which would change the distance, so
    # equal accuracy here and the combined latency alone decides (cost the other way round)
    rows = rows_from([0, 0], [1, 1], [20, 10], [7000, 7000], [1, 2])
    assert miss(rows, [I, I], [0, 0], 100, 7001) == 1


# -- state transitions at the end of a window: closed form under constant arrivals --------------
def test_state_transitions_closed_form():
    #         id0        id1       id2         id3
    rows = rows_from([0] * 4, [1] * 4, [1000] * 4, [7000] * 4, [1, 2, 3, 4], [0, 0, 0, 9])
    s = StatefulOracleCatalog(rows, 1, [ACTIVE, INACTIVE, INTERFERED, INACTIVE], [0] * 4)
    window_us = 5000                                             # drain = 5 per window
    arrivals = np.array([0] * 8 + [1] * 3 + [2] * 50, np.uint32)   # 8, 3, 50, 0 per window
    for k in range(1, 4):
        s.load_update(arrivals, window_us)
        # id0: backlog 3k -> Overloaded; id1: loaded by its first queries, keeps up -> Active;
        # id2: Interfered whatever its load; id3: no queries -> stays Inactive, its queue drains
        assert list(s.queued) == [3 * k, 0, 45 * k, max(0, 9 - 5 * k)]
        assert list(s.state) == [OVERLOADED, ACTIVE, INTERFERED, INACTIVE]
    none = np.zeros(0, np.uint32)
    for k in range(1, 4):                                        # arrivals stop: 9 -> 4 -> 0
        s.load_update(none, window_us)
        assert int(s.queued[0]) == max(0, 9 - 5 * k)
        assert int(s.state[0]) == (OVERLOADED if 9 - 5 * k > 0 else ACTIVE)
    # an Inactive variant that is given more than it can drain is Overloaded at once
    s = StatefulOracleCatalog(rows, 1, [INACTIVE] * 4, [0] * 4)
    s.load_update(np.array([1] * 6, np.uint32), window_us)
    assert list(s.state) == [INACTIVE, OVERLOADED, INACTIVE, INACTIVE] and int(s.queued[1]) == 1
    # tallies and counters are those of the plain update
    o = OracleCatalog(rows, 1)
    o.load_update(np.array([1] * 6, np.uint32), window_us)
    assert np.array_equal(o.queued, s.queued) and np.array_equal(o.counters, s.counters)


# -- Inactive ties and the saturating sum -----------------------------------------------------
def test_inactive_ties_and_saturation():
    #                 id0   id1   id2   id3
    rows = rows_from([0] * 4, [1] * 4, [70, 60, 50, 50], [7000, 7200, 7200, 7100], [1, 9, 9, 9])
    s = StatefulOracleCatalog(rows, 1, [INACTIVE] * 4, [30, 40, 50, 50])   # all combine to 100
    assert int(s.select([0], [100], [0])[0]) == 1          # equal latency: accuracy, then id; not cost
    assert int(s.select([0], [100], [7201])[0]) == (NO_FEASIBLE_BIT | 1)
    assert int(s.select([0], [99], [0])[0]) == (NO_FEASIBLE_BIT | 1)
    # 50 + (2^32 - 1) stays at 2^32 - 1 instead of wrapping to 49; id3 sums to 2^32 - 50
    s = StatefulOracleCatalog(rows, 1, [INTERFERED, OVERLOADED, INACTIVE, INACTIVE], [0, 0, 2**32 - 1, 2**32 - 100])
    assert int(s.select([0], [49], [0])[0]) == (NO_FEASIBLE_BIT | 3)
    assert int(s.select([0], [2**32 - 1], [7200])[0]) == 2
    assert int(s.select([0], [2**32 - 2], [7200])[0]) == (NO_FEASIBLE_BIT | 2)
    assert int(s.select([0], [2**32 - 2], [0])[0]) == 3


# -- permuting the catalog rows (ids, states and loading latencies carried along) -----------------
def test_row_permutation_equivariance_stateful():
    w = W.make("C2", n_queries=4000)
    rng = np.random.default_rng(6)
    state = _random_states(rng, w.n_variants, (0.5, 0.3, 0.1, 0.1))
    load = rng.integers(0, 200_000, w.n_variants).astype(np.uint32)
    d0 = StatefulOracleCatalog(w.rows, w.n_tasks, state, load).select(w.task, w.slo_us, w.min_acc_bp, 3)
    perm = rng.permutation(w.n_variants)
    d1 = StatefulOracleCatalog(w.rows[perm], w.n_tasks, state[perm], load[perm]).select(w.task, w.slo_us, w.min_acc_bp)
    assert np.array_equal(d1 == INVALID, d0 == INVALID)
    ok = d0 != INVALID
    assert np.array_equal(d1[ok] & NO_FEASIBLE_BIT, d0[ok] & NO_FEASIBLE_BIT)
    r0, r1 = w.rows[d0[ok] & 0x7FFFFFFF], w.rows[perm][d1[ok] & 0x7FFFFFFF]
    for k in ("cost", "lat_us", "acc_bp", "batch", "queued"):   # the same variant up to id ties
        assert np.array_equal(r0[k], r1[k])
    assert np.array_equal(state[d0[ok] & 0x7FFFFFFF], state[perm][d1[ok] & 0x7FFFFFFF])


# -- loading a variant (Inactive -> Active) never turns a served query into an unserved one ------
def test_activation_is_monotone():
    w = W.make("C2", n_queries=4000)
    rng = np.random.default_rng(7)
    state = _random_states(rng, w.n_variants, (0.7, 0.2, 0.05, 0.05))
    load = rng.integers(1000, 300_000, w.n_variants).astype(np.uint32)
    d0 = StatefulOracleCatalog(w.rows, w.n_tasks, state, load).select(w.task, w.slo_us, w.min_acc_bp, 3)
    state2 = state.copy()
    flip = (state == INACTIVE) & (rng.random(w.n_variants) < 0.5)
    state2[flip] = ACTIVE
    d1 = StatefulOracleCatalog(w.rows, w.n_tasks, state2, load).select(w.task, w.slo_us, w.min_acc_bp, 3)
    served0, served1 = (d0 >> 31) == 0, (d1 >> 31) == 0
    assert np.all(served1[served0]) and served1.sum() > served0.sum()
    # and a query that an Active variant already served is still served by an Active one, no dearer
    was_active = served0 & (state[d0 & 0x7FFFFFFF] == ACTIVE)
    assert np.all(state2[d1[was_active]] == ACTIVE)
    assert np.all(w.rows["cost"][d1[was_active]].astype(np.int64) <= w.rows["cost"][d0[was_active]].astype(np.int64))
