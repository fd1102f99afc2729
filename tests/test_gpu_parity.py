"""GPU parity: the CUDA path, called through the C ABI, against the CPU oracle, element by
element on the same seeded inputs.  Integer work: the bar is bit-exact."""
import numpy as np
import pytest

from oracle import OracleCatalog
from paper_1905_13348_b200 import workloads as W
from tests.helpers import INVALID, NO_FEASIBLE_BIT, rows_from

pytestmark = pytest.mark.gpu


def _torch():
    import torch
    return torch


def _to_dev(a):
    torch = _torch()
    view = {np.dtype("uint16"): np.int16, np.dtype("uint32"): np.int32}[a.dtype]
    return torch.from_numpy(np.ascontiguousarray(a).view(view)).cuda()


def _to_host_u32(t):
    return t.cpu().numpy().view(np.uint32)


def gpu_select(cat, task, slo, acc):
    import paper_1905_13348_b200 as P
    torch = _torch()
    d_task, d_slo, d_acc = _to_dev(task), _to_dev(slo), _to_dev(acc)
    d_dec = torch.full((task.shape[0],), 0x5A5A5A5A, dtype=torch.int32, device="cuda")
    P.infaas_select_batch(cat, d_task, d_slo, d_acc, d_dec)
    torch.cuda.synchronize()
    return d_dec


def assert_state_equal(cat, o):
    import paper_1905_13348_b200 as P
    st = P.infaas_catalog_get_state(cat)
    assert np.array_equal(st["queued"], o.queued)
    assert np.array_equal(st["pred_lat_us"], o.pred_lat())
    assert np.array_equal(st["served_total"], o.served_total)
    assert np.array_equal(st["counters"], o.counters)


def run_both(w, n_threads=8, check_state=True):
    """Whole workload through both sides; windowed if the workload says so."""
    import paper_1905_13348_b200 as P
    cat = P.infaas_catalog_load(w.rows, w.n_tasks)
    o = OracleCatalog(w.rows, w.n_tasks)
    try:
        if check_state:
            assert_state_equal(cat, o)
        step = w.window if w.window else max(1, w.n_queries)
        for lo in range(0, w.n_queries, step):
            s = slice(lo, min(w.n_queries, lo + step))
            want = o.select(w.task[s], w.slo_us[s], w.min_acc_bp[s], n_threads)
            d_dec = gpu_select(cat, w.task[s], w.slo_us[s], w.min_acc_bp[s])
            got = _to_host_u32(d_dec)
            bad = np.flatnonzero(got != want)
            assert bad.size == 0, (w.name, lo, bad[:5], got[bad[:5]], want[bad[:5]])
            if w.window:
                P.infaas_load_update(cat, d_dec, w.window_us)
                o.load_update(want, w.window_us)
                if check_state:
                    assert_state_equal(cat, o)
        if not w.window:
            P.infaas_load_update(cat, d_dec, 1000)
            o.load_update(want, 1000)
            assert_state_equal(cat, o)
    finally:
        cat.free()


@pytest.mark.parametrize("name,kw", [
    ("C1", {}),
    ("C2", {"n_queries": 200_003}),
    ("C3", {"n_queries": 12 * 8192 + 77, "window": 8192}),
    ("C4", {"n_queries": 65_537}),
    ("C5", {"n_windows": 6, "window": 4096}),
])
def test_configs_reduced(name, kw):
    run_both(W.make(name, **kw))


def test_heavy_load_windows_change_the_frontier():
    # few queries' worth of drain per window: queues build up, scan lists change every window
    w = W.make("C3", n_queries=20 * 4096, window=4096)
    w.window_us = 300
    run_both(w)


@pytest.mark.parametrize("n", [0, 1, 2, 3, 4, 5, 7, 8, 511, 2049])
def test_ragged_sizes(n):
    w = W.make("C2", n_queries=4096)
    w.task, w.slo_us, w.min_acc_bp = w.task[:n], w.slo_us[:n], w.min_acc_bp[:n]
    if n == 0:
        import paper_1905_13348_b200 as P
        cat = P.infaas_catalog_load(w.rows, w.n_tasks)
        P.infaas_select_batch(cat, None, None, None, None, n=0)
        P.infaas_load_update(cat, None, 1000, n=0)
        assert_state_equal(cat, _advance(OracleCatalog(w.rows, w.n_tasks), 1000))
        cat.free()
        return
    run_both(w)


def _advance(o, window_us):
    o.load_update(np.zeros(0, np.uint32), window_us)
    return o


def test_invalid_and_extreme_queries():
    # tasks 0 and 2 have variants, task 1 has none, tasks >= 3 do not exist
    rows = rows_from([0, 0, 2, 2, 2], [1, 4, 1, 2, 65535], [100, 2**32 - 1, 50, 1, 7],
                     [7000, 10000, 0, 6500, 9000], [5, 2**32 - 1, 1, 2, 3], [0, 2**32 - 1, 3, 0, 9])
    rng = np.random.default_rng(0)
    n = 5000
    task = rng.integers(0, 6, n).astype(np.uint16)
    task[:4] = [65535, 3, 1, 0]
    slo = rng.choice(np.array([0, 1, 49, 50, 100, 200, 2**32 - 1], np.uint32), n)
    acc = rng.choice(np.array([0, 6500, 7000, 7001, 10000, 10001, 65535], np.uint16), n)
    w = W.Workload("edge", 3, rows, task, slo, acc, 0, 0, "edge cases")
    run_both(w)
    d = OracleCatalog(rows, 3).select(task, slo, acc)
    assert (d == INVALID).any() and ((d >> 31) == 1).any() and ((d >> 31) == 0).any()


def test_ties_everywhere():
    # tiny attribute ranges: many equal costs, latencies and accuracies -> tie-break order
    rng = np.random.default_rng(5)
    nv, T = 600, 3
    rows = rows_from(rng.integers(0, T, nv), rng.choice([1, 2], nv), rng.integers(10, 14, nv),
                     rng.integers(7000, 7004, nv), rng.integers(1, 4, nv), rng.integers(0, 3, nv))
    n = 30000
    w = W.Workload("ties", T, rows, rng.integers(0, T, n).astype(np.uint16),
                   rng.integers(8, 45, n).astype(np.uint32),
                   rng.integers(6998, 7006, n).astype(np.uint16), 6000, 20, "ties")
    run_both(w)


def test_single_task_maximum_size_and_unequal_tasks():
    rng = np.random.default_rng(6)
    sizes = [8192, 1, 0, 37]                        # the per-task limit, a singleton, an empty task
    task = np.repeat(np.arange(4), sizes)
    nv = task.size
    rows = rows_from(task, rng.choice([1, 8, 64], nv), rng.integers(100, 10**6, nv),
                     rng.integers(5000, 9000, nv), rng.integers(1, 5000, nv))
    rows = rows[rng.permutation(nv)]
    n = 20000
    w = W.Workload("big-task", 4, rows, rng.integers(0, 4, n).astype(np.uint16),
                   rng.integers(50, 2 * 10**6, n).astype(np.uint32),
                   rng.integers(5000, 9200, n).astype(np.uint16), 0, 0, "one task at the size limit")
    run_both(w, check_state=True)


def test_load_update_ignores_flagged_and_out_of_range_decisions():
    import paper_1905_13348_b200 as P
    w = W.make("C2", n_queries=16)
    rng = np.random.default_rng(9)
    dec = rng.integers(0, w.n_variants, 40001).astype(np.uint32)
    dec[::7] |= NO_FEASIBLE_BIT
    dec[::11] = INVALID
    dec[::13] = w.n_variants + 5                     # not a variant id: counted as invalid
    dec[5:3000] = 17                                  # one hot variant
    cat = P.infaas_catalog_load(w.rows, w.n_tasks)
    o = OracleCatalog(w.rows, w.n_tasks)
    for _ in range(3):
        P.infaas_load_update(cat, _to_dev(dec), 5000)
        o.load_update(dec, 5000)
        assert_state_equal(cat, o)
    cat.free()


def test_frontier_lists_are_sorted_non_dominated_sets():
    import paper_1905_13348_b200 as P
    w = W.make("C3", n_queries=16)
    cat = P.infaas_catalog_load(w.rows, w.n_tasks)
    o = OracleCatalog(w.rows, w.n_tasks)
    pred = o.pred_lat().astype(np.int64)
    acc, cost = w.rows["acc_bp"].astype(np.int64), w.rows["cost"].astype(np.int64)
    for t in range(0, w.n_tasks, 9):
        ids = P.infaas_catalog_get_frontier(cat, t).astype(np.int64)
        members = np.flatnonzero(w.rows["task"] == t)
        keys = [(cost[v], pred[v], -acc[v], v) for v in ids]
        assert keys == sorted(keys) and set(ids) <= set(members)
        def dominated(b):
            return any(pred[a] <= pred[b] and acc[a] >= acc[b] and cost[a] <= cost[b] and
                       ((pred[a], acc[a], cost[a]) != (pred[b], acc[b], cost[b]) or a < b)
                       for a in members if a != b)
        assert set(ids) == {int(v) for v in members if not dominated(v)}
    cat.free()


def test_alignment_and_null_errors():
    import paper_1905_13348_b200 as P
    from paper_1905_13348_b200 import binding as B
    torch = _torch()
    w = W.make("C1")
    cat = P.infaas_catalog_load(w.rows, w.n_tasks)
    d_task, d_slo, d_acc = _to_dev(w.task), _to_dev(w.slo_us), _to_dev(w.min_acc_bp)
    d_dec = torch.zeros(w.n_queries, dtype=torch.int32, device="cuda")
    with pytest.raises(B.InfaasError) as e:
        P.infaas_select_batch(cat, d_task[1:], d_slo[1:], d_acc[1:], d_dec[1:])
    assert e.value.code == -8
    with pytest.raises(B.InfaasError) as e:
        P.infaas_select_batch(cat, d_task, None, d_acc, d_dec, n=8)
    assert e.value.code == -1
    cat.free()


# -- full sizes, in the launch configuration the benchmark times ----------------------------
def _np_pred(rows, queued):
    lat, q, b = (rows["lat_us"].astype(np.uint64), queued.astype(np.uint64),
                 rows["batch"].astype(np.uint64))
    return np.minimum(lat + q * lat // b, np.uint64(2**32 - 1)).astype(np.uint32)


def _assert_state_fast(cat, o, rows):
    import paper_1905_13348_b200 as P
    st = P.infaas_catalog_get_state(cat)
    assert np.array_equal(st["queued"], o.queued)
    assert np.array_equal(st["pred_lat_us"], _np_pred(rows, o.queued))
    assert np.array_equal(st["served_total"], o.served_total)
    assert np.array_equal(st["counters"], o.counters)


def _threads():
    import os
    return os.cpu_count() or 1


@pytest.mark.parametrize("name", ["C2", "C3", "C4"])
def test_full_size_single_launch_then_update(name):
    """All queries of the configuration in ONE infaas_select_batch (the launch shape the
    benchmark times: one contiguous range per SM), then one load update over all decisions,
    then a second launch against the updated load."""
    import paper_1905_13348_b200 as P
    w = W.make(name)
    window_us = max(1, w.n_queries // max(1, w.window)) * w.window_us if w.window else 1_000_000
    window_us = min(window_us, 2**32 - 1)
    cat = P.infaas_catalog_load(w.rows, w.n_tasks)
    o = OracleCatalog(w.rows, w.n_tasks)
    try:
        for rnd in range(2):
            want = o.select(w.task, w.slo_us, w.min_acc_bp, _threads())
            d_dec = gpu_select(cat, w.task, w.slo_us, w.min_acc_bp)
            got = _to_host_u32(d_dec)
            bad = np.flatnonzero(got != want)
            assert bad.size == 0, (name, rnd, bad[:5], got[bad[:5]], want[bad[:5]])
            P.infaas_load_update(cat, d_dec, window_us)
            o.load_update(want, window_us)
            _assert_state_fast(cat, o, w.rows)
    finally:
        cat.free()


@pytest.mark.parametrize("name,state_every,fused", [("C3", 16, False), ("C3", 32, True), ("C5", 100, False)])
def test_full_size_windowed(name, state_every, fused):
    """The configuration as a stream of windows (select one window, update, repeat): every
    decision of every window is compared; the load state every `state_every` windows and at
    the end."""
    import paper_1905_13348_b200 as P
    torch = _torch()
    w = W.make(name)
    cat = P.infaas_catalog_load(w.rows, w.n_tasks)
    o = OracleCatalog(w.rows, w.n_tasks)
    d_task, d_slo, d_acc = _to_dev(w.task), _to_dev(w.slo_us), _to_dev(w.min_acc_bp)
    d_dec = torch.empty(w.n_queries, dtype=torch.int32, device="cuda")
    nwin = w.n_queries // w.window
    try:
        for k in range(nwin):
            s = slice(k * w.window, (k + 1) * w.window)
            if fused:
                P.infaas_select_update(cat, d_task[s], d_slo[s], d_acc[s], d_dec[s], w.window_us)
            else:
                P.infaas_select_batch(cat, d_task[s], d_slo[s], d_acc[s], d_dec[s])
                P.infaas_load_update(cat, d_dec[s], w.window_us)
            want = o.select(w.task[s], w.slo_us[s], w.min_acc_bp[s], _threads())
            o.load_update(want, w.window_us)
            got = _to_host_u32(d_dec[s])
            bad = np.flatnonzero(got != want)
            assert bad.size == 0, (name, k, bad[:5], got[bad[:5]], want[bad[:5]])
            if (k + 1) % state_every == 0 or k == nwin - 1:
                _assert_state_fast(cat, o, w.rows)
        assert int(o.counters.sum()) == w.n_queries
    finally:
        cat.free()


@pytest.mark.parametrize("name,kw,sizes", [
    ("C3", {"n_queries": 40_000}, [4096, 1, 0, 777, 8192, 130, 2049, 10_000, 14_654]),
    ("C5", {"n_windows": 3, "window": 8192}, [8192, 5, 8187, 8192]),
    ("C4", {"n_queries": 30_000}, [30_000]),
    ("C2", {"n_queries": 300_000}, [100, 299_900]),          # the second window is above the fused limit
])
def test_fused_window_call(name, kw, sizes):
    """infaas_select_update (one call per window; the selection kernel tallies its own decisions
    for small windows) against the oracle: decisions of every window, state after every window.
    Ragged and empty windows, bad tasks in between, heavy load so that the lists move."""
    import paper_1905_13348_b200 as P
    torch = _torch()
    w = W.make(name, **kw)
    assert sum(sizes) <= w.n_queries
    task = w.task.copy()
    task[::97] = w.n_tasks + 3                                   # invalid queries are counted too
    window_us = 500
    cat = P.infaas_catalog_load(w.rows, w.n_tasks)
    o = OracleCatalog(w.rows, w.n_tasks)
    try:
        lo = 0
        for n in sizes:
            s = slice(lo, lo + n)
            d_dec = torch.empty(n, dtype=torch.int32, device="cuda")     # fresh arrays: 16-byte aligned
            if n:
                P.infaas_select_update(cat, _to_dev(task[s]), _to_dev(w.slo_us[s]), _to_dev(w.min_acc_bp[s]),
                                       d_dec, window_us)
            else:
                P.infaas_select_update(cat, None, None, None, None, window_us, n=0)
            want = o.select(task[s], w.slo_us[s], w.min_acc_bp[s], _threads())
            o.load_update(want, window_us)
            got = _to_host_u32(d_dec)
            bad = np.flatnonzero(got != want)
            assert bad.size == 0, (name, lo, n, bad[:5], got[bad[:5]], want[bad[:5]])
            assert_state_equal(cat, o)
            lo += n
    finally:
        cat.free()


@pytest.mark.parametrize("n_tasks,per_task", [(5000, 4), (20000, 3), (65535, 1)])
def test_many_small_tasks(n_tasks, per_task):
    """Thousands of tasks: the fixed tables of the index alone exceed shared memory (5000 tasks)
    or even the range the task word's offset field addresses (20000 tasks: the tasks whose block
    lies beyond it have no index and are answered by walking their lists).  Two windows with an
    update between them."""
    rng = np.random.default_rng(77)
    nv = n_tasks * per_task
    task = np.repeat(np.arange(n_tasks), per_task)
    rows = rows_from(task, rng.choice(np.array([1, 2, 4, 8]), nv), rng.integers(500, 200_000, nv),
                     rng.integers(5600, 8300, nv), rng.integers(1, 2000, nv), rng.integers(0, 3, nv))
    rows = rows[rng.permutation(nv)]
    n = 2 * 30_011
    q_task = rng.integers(0, n_tasks + 2, n).astype(np.uint16)
    q_slo = np.exp(rng.uniform(np.log(300.0), np.log(400_000.0), n)).astype(np.uint32)
    q_acc = rng.integers(5000, 8600, n).astype(np.uint16)
    run_both(W.Workload("many tasks", n_tasks, rows, q_task, q_slo, q_acc, 30_011, 20_000, "many small tasks"))


def test_split_update_with_summed_counts_matches_whole_window():
    """infaas_tally / infaas_pending_counts / infaas_advance: two catalogs on this GPU stand
    in for two ranks; each decides its share of a window, the pending counts are summed and
    handed to both, and both must reach the oracle's state for the whole window."""
    import paper_1905_13348_b200 as P
    from paper_1905_13348_b200 import sharding as S
    torch = _torch()
    w = W.make("C3", n_queries=5 * 8192, window=8192)
    w.window_us = 300
    cats = [P.infaas_catalog_load(w.rows, w.n_tasks) for _ in range(2)]
    o = OracleCatalog(w.rows, w.n_tasks)
    try:
        for k in range(w.n_queries // w.window):
            base = k * w.window
            ws = slice(base, base + w.window)
            want = o.select(w.task[ws], w.slo_us[ws], w.min_acc_bp[ws], 4)
            o.load_update(want, w.window_us)
            exported = []
            for r, cat in enumerate(cats):
                lo, hi = S.shard_bounds(w.window, 2, r)
                sl = slice(base + lo, base + hi)
                d_dec = gpu_select(cat, w.task[sl], w.slo_us[sl], w.min_acc_bp[sl])
                assert np.array_equal(_to_host_u32(d_dec), want[lo:hi])
                P.infaas_tally(cat, d_dec)
                cnt = torch.zeros(w.n_variants, dtype=torch.int32, device="cuda")
                P.infaas_pending_counts(cat, cnt, set=False)
                exported.append(cnt)
            total = exported[0] + exported[1]
            for cat in cats:
                P.infaas_pending_counts(cat, total, set=True)
                P.infaas_advance(cat, w.window_us)
                st = P.infaas_catalog_get_state(cat)
                assert np.array_equal(st["queued"], o.queued)
                assert np.array_equal(st["served_total"], o.served_total)
                assert np.array_equal(st["pred_lat_us"], _np_pred(w.rows, o.queued))
        assert o.queued.max() > 0
    finally:
        for cat in cats:
            cat.free()


def test_large_batch_over_a_catalog_whose_tally_bins_need_two_ranges():
    """65,536 variants: the shared-memory tally splits the ids into two ranges; 2M queries in
    one launch (image read from global memory: it does not fit in shared memory)."""
    import paper_1905_13348_b200 as P
    w = W.make("C5", n_windows=32)
    cat = P.infaas_catalog_load(w.rows, w.n_tasks)
    o = OracleCatalog(w.rows, w.n_tasks)
    try:
        for rnd in range(2):
            want = o.select(w.task, w.slo_us, w.min_acc_bp, _threads())
            d_dec = gpu_select(cat, w.task, w.slo_us, w.min_acc_bp)
            assert np.array_equal(_to_host_u32(d_dec), want), rnd
            P.infaas_load_update(cat, d_dec, 32 * w.window_us)
            o.load_update(want, 32 * w.window_us)
            _assert_state_fast(cat, o, w.rows)
    finally:
        cat.free()


@pytest.mark.parametrize("seed", range(6))
def test_random_catalog_shapes(seed):
    """Catalog shapes around the kernels' internal limits: task sizes on both sides of the
    small-task sort limit and of the index limit, accuracy spans wider than the bitmap
    supports, latencies from 1 us to beyond 2^24 us, many equal values, uneven load."""
    rng = np.random.default_rng(1000 + seed)
    sizes = rng.choice(np.array([1, 2, 3, 31, 32, 33, 200, 255, 256, 257, 511, 512, 513, 700, 1025]),
                       size=int(rng.integers(3, 9)))
    T = sizes.size + 1                               # the last task stays empty
    task = np.repeat(np.arange(sizes.size), sizes)
    nv = task.size
    style = seed % 3
    if style == 0:      # trade-off surface: long non-dominated lists, wide accuracy span
        lat = np.exp(rng.uniform(np.log(1.0), np.log(3.0e7), nv))
        cost = 1.0e6 / lat ** 0.5 * np.exp(0.3 * rng.standard_normal(nv))
        acc = np.clip(10000 * (np.log(lat) / np.log(3.0e7)) + 300 * rng.standard_normal(nv), 0, 10000)
    elif style == 1:    # few distinct values: ties everywhere
        lat = rng.choice(np.array([1, 7, 100, 1000, 20000, 2**24, 2**24 + 1, 2**31]), nv).astype(float)
        cost = rng.integers(1, 6, nv).astype(float)
        acc = rng.choice(np.array([0, 1, 5000, 7000, 7001, 9999, 10000]), nv).astype(float)
    else:               # independent attributes: short lists
        lat = np.exp(rng.uniform(np.log(50.0), np.log(5.0e6), nv))
        cost = rng.integers(1, 100000, nv).astype(float)
        acc = rng.integers(5000, 9000, nv).astype(float)
    rows = rows_from(task, rng.choice(np.array([1, 2, 8, 64, 65535]), nv),
                     np.maximum(1, np.round(lat)).astype(np.uint64).clip(1, 2**32 - 1),
                     np.round(acc).astype(np.int64), np.maximum(1, np.round(cost)).astype(np.uint64).clip(1, 2**32 - 1),
                     rng.choice(np.array([0, 0, 0, 1, 5, 1000, 2**20]), nv))
    rows = rows[rng.permutation(nv)]
    n = 3 * 20011
    q_task = rng.integers(0, T + 1, n).astype(np.uint16)
    q_slo = np.where(rng.random(n) < 0.9, np.exp(rng.uniform(0, np.log(1.0e8), n)),
                     rng.choice(np.array([0, 1, 2**24 - 1, 2**24, 2**32 - 1], dtype=np.float64), n)).astype(np.uint64)
    q_slo = q_slo.clip(0, 2**32 - 1).astype(np.uint32)
    q_acc = np.where(rng.random(n) < 0.9, rng.integers(0, 10001, n), rng.choice(np.array([0, 10001, 65535]), n)).astype(np.uint16)
    w = W.Workload("shapes", T, rows, q_task, q_slo, q_acc, 20011, 50_000, "random shapes")
    run_both(w)


def test_image_somewhat_larger_than_shared_memory():
    # windows short enough for the queues to be noisy: the lists grow until the lookup image no
    # longer fits in shared memory; the kernel then reads it from global memory, first with the
    # shared memory still reserved, then (after the next look at the state) without
    import paper_1905_13348_b200 as P
    win, n_win = 8192, 36
    w = W.make("C3", n_queries=n_win * win, window=win)
    w.window_us = 5000
    cat = P.infaas_catalog_load(w.rows, w.n_tasks)
    o = OracleCatalog(w.rows, w.n_tasks)
    reserved = released = 0
    try:
        for k in range(n_win):
            s = slice(k * win, (k + 1) * win)
            want = o.select(w.task[s], w.slo_us[s], w.min_acc_bp[s], 8)
            d_dec = gpu_select(cat, w.task[s], w.slo_us[s], w.min_acc_bp[s])
            assert np.array_equal(_to_host_u32(d_dec), want), k
            info = P.infaas_catalog_get_info(cat)
            reserved += info["image_smem"] > 0 and info["image_bytes"] > info["image_smem"]
            released += info["image_smem"] == 0
            P.infaas_load_update(cat, d_dec, w.window_us)
            o.load_update(want, w.window_us)
            if k % 4 == 3:
                assert_state_equal(cat, o)        # also lets the library re-plan its shared memory
        assert released >= 10, (reserved, released)
    finally:
        cat.free()
