"""GPU parity of state-aware selection (Section 4, state machine; Section 4.1, Case I) and of
the state transitions at the end of a window: the CUDA path through the C ABI against the
CPU oracle, bit for bit."""
import numpy as np
import pytest

from oracle import (ACTIVE, INACTIVE, INTERFERED, OVERLOADED, OracleCatalog,
                    StatefulOracleCatalog)
from paper_1905_13348_b200 import workloads as W
from tests.helpers import INVALID, NO_FEASIBLE_BIT, rows_from
from tests.test_gpu_parity import _to_host_u32, assert_state_equal, gpu_select

pytestmark = pytest.mark.gpu

STATES = np.array([INACTIVE, ACTIVE, OVERLOADED, INTERFERED], np.uint8)


def run_stateful(w, state, load, n_threads=8, expect=None):
    """Whole workload through both sides with states; windowed if the workload says so.
    Returns how many decisions were Active picks, Inactive picks, suggestions, invalid."""
    import paper_1905_13348_b200 as P
    cat = P.infaas_catalog_load(w.rows, w.n_tasks)
    o = StatefulOracleCatalog(w.rows, w.n_tasks, state, load)
    seen = np.zeros(4, np.int64)
    try:
        assert np.all(P.infaas_catalog_get_states(cat) == ACTIVE)
        P.infaas_catalog_set_states(cat, state, load)
        assert np.array_equal(P.infaas_catalog_get_states(cat), o.state)
        step = w.window if w.window else max(1, w.n_queries)
        for lo in range(0, w.n_queries, step):
            s = slice(lo, min(w.n_queries, lo + step))
            want = o.select(w.task[s], w.slo_us[s], w.min_acc_bp[s], n_threads)
            d_dec = gpu_select(cat, w.task[s], w.slo_us[s], w.min_acc_bp[s])
            got = _to_host_u32(d_dec)
            bad = np.flatnonzero(got != want)
            assert bad.size == 0, (w.name, lo, bad[:5], got[bad[:5]], want[bad[:5]])
            ok = want[(want >> 31) == 0]
            seen += [int((o.state[ok] == ACTIVE).sum()), int((o.state[ok] == INACTIVE).sum()),
                     int(((want >> 31) == 1).sum() - (want == INVALID).sum()), int((want == INVALID).sum())]
            P.infaas_load_update(cat, d_dec, w.window_us if w.window else 1000)
            o.load_update(want, w.window_us if w.window else 1000)
            assert_state_equal(cat, o)
            assert np.array_equal(P.infaas_catalog_get_states(cat), o.state), (w.name, lo)
    finally:
        cat.free()
    return seen


def _states(rng, n, p):
    return rng.choice(STATES, n, p=p)


@pytest.mark.parametrize("name,kw,p,load_hi", [
    ("C1", {}, (0.5, 0.3, 0.1, 0.1), 150_000),
    ("C2", {"n_queries": 100_003}, (0.6, 0.2, 0.1, 0.1), 150_000),
    ("C3", {"n_queries": 12 * 8192 + 77, "window": 8192}, (0.7, 0.1, 0.1, 0.1), 150_000),
    ("C4", {"n_queries": 65_537}, (0.7, 0.2, 0.05, 0.05), 3_000),   # both lists span several segments
    ("C5", {"n_windows": 6, "window": 4096}, (0.8, 0.1, 0.05, 0.05), 150_000),
])
def test_configs_reduced_stateful(name, kw, p, load_hi):
    w = W.make(name, **kw)
    rng = np.random.default_rng(31)
    seen = run_stateful(w, _states(rng, w.n_variants, p),
                        rng.integers(0, load_hi, w.n_variants).astype(np.uint32))
    assert seen[0] > 0 and seen[1] > 0 and seen[2] > 0, seen


def test_full_size_stateful_two_launches():
    """The 16M-query configuration with the benchmark leg's state mix: one launch over all 2^24
    queries, the load update (states move), and a second launch -- every decision of both."""
    import paper_1905_13348_b200 as P
    from tests.test_gpu_parity import _to_dev
    w = W.make("C3")
    state, load = W.variant_states(w.n_variants)
    cat = P.infaas_catalog_load(w.rows, w.n_tasks)
    o = StatefulOracleCatalog(w.rows, w.n_tasks, state, load)
    window_us = 256 * w.window_us
    try:
        P.infaas_catalog_set_states(cat, state, load)
        d_task, d_slo, d_acc = _to_dev(w.task), _to_dev(w.slo_us), _to_dev(w.min_acc_bp)
        for launch in range(2):
            d_dec = gpu_select(cat, w.task, w.slo_us, w.min_acc_bp) if launch == 0 else d_dec
            if launch:
                P.infaas_select_batch(cat, d_task, d_slo, d_acc, d_dec)
            want = o.select(w.task, w.slo_us, w.min_acc_bp, 16)
            got = _to_host_u32(d_dec)
            bad = np.flatnonzero(got != want)
            assert bad.size == 0, (launch, bad[:5], got[bad[:5]], want[bad[:5]])
            P.infaas_load_update(cat, d_dec, window_us)
            o.load_update(want, window_us)
            assert np.array_equal(P.infaas_catalog_get_state(cat)["queued"], o.queued)
            assert np.array_equal(P.infaas_catalog_get_states(cat), o.state)
        assert (o.state != state).any()                       # the update did move states
    finally:
        cat.free()


def test_stateful_catalog_whose_image_exceeds_shared_memory():
    """A state-aware catalog large enough that the selection kernel reads its tables from
    global memory (128 tasks x 512 variants, both lists long): three windows, all decisions."""
    import paper_1905_13348_b200 as P
    w = W.make("C5", n_windows=3)
    rng = np.random.default_rng(35)
    state = _states(rng, w.n_variants, (0.45, 0.45, 0.05, 0.05))
    load = rng.integers(0, 50_000, w.n_variants).astype(np.uint32)
    cat = P.infaas_catalog_load(w.rows, w.n_tasks)
    try:
        P.infaas_catalog_set_states(cat, state, load)
        info = P.infaas_catalog_get_info(cat)
        assert info["image_bytes"] > info["image_smem"], info
    finally:
        cat.free()
    seen = run_stateful(w, state, load, n_threads=16)
    assert seen[0] > 0 and seen[1] > 0


def test_states_follow_the_load_over_many_windows():
    # little drain per window: variants overload, queries move on to Inactive ones, which
    # become Active (and overload in turn), then everything drains
    w = W.make("C3", n_queries=24 * 4096, window=4096)
    w.window_us = 400
    rng = np.random.default_rng(32)
    state = _states(rng, w.n_variants, (0.85, 0.1, 0.0, 0.05))
    seen = run_stateful(w, state, rng.integers(0, 20_000, w.n_variants).astype(np.uint32))
    assert seen[0] > 0 and seen[1] > 0


def test_whole_tasks_in_one_state():
    w = W.make("C2", n_queries=40_000)
    rng = np.random.default_rng(33)
    state = _states(rng, w.n_variants, (0.4, 0.4, 0.1, 0.1))
    tk = w.rows["task"]
    state[tk == 0] = INACTIVE          # the fast path's list is the Inactive one
    state[tk == 1] = OVERLOADED        # nothing selectable: INVALID
    state[tk == 2] = ACTIVE
    state[tk == 3] = INTERFERED
    state[tk == 4] = np.where(np.arange((tk == 4).sum()) % 2, OVERLOADED, INTERFERED)
    load = rng.integers(0, 100_000, w.n_variants).astype(np.uint32)
    load[rng.random(w.n_variants) < 0.05] = 2**32 - 1            # combined latency saturates
    seen = run_stateful(w, state, load)
    assert seen[3] > 0


def test_all_active_equals_stateless_path():
    import paper_1905_13348_b200 as P
    w = W.make("C3", n_queries=50_000)
    a, b = P.infaas_catalog_load(w.rows, w.n_tasks), P.infaas_catalog_load(w.rows, w.n_tasks)
    try:
        P.infaas_catalog_set_states(b, np.full(w.n_variants, ACTIVE, np.uint8), None)
        da = _to_host_u32(gpu_select(a, w.task, w.slo_us, w.min_acc_bp))
        db = _to_host_u32(gpu_select(b, w.task, w.slo_us, w.min_acc_bp))
        assert np.array_equal(da, db)
        assert np.array_equal(da, OracleCatalog(w.rows, w.n_tasks).select(w.task, w.slo_us, w.min_acc_bp, 8))
    finally:
        a.free(); b.free()


def test_tiny_catalog_grid_stateful():
    # every (slo, min_acc) around the catalog's own values, ties everywhere
    rng = np.random.default_rng(34)
    for _ in range(6):
        nv = int(rng.integers(1, 12))
        rows = rows_from(rng.integers(0, 2, nv), rng.choice([1, 2, 4, 7], nv), rng.integers(1, 40, nv),
                         rng.integers(6990, 7010, nv), rng.integers(1, 4, nv), rng.integers(0, 5, nv))
        state = _states(rng, nv, (0.4, 0.4, 0.1, 0.1))
        load = rng.integers(0, 30, nv).astype(np.uint32)
        slos = np.arange(0, 260, dtype=np.uint32)
        accs = np.arange(6985, 7015, dtype=np.uint16)
        task = np.repeat(np.arange(3, dtype=np.uint16), slos.size * accs.size)
        slo = np.tile(np.repeat(slos, accs.size), 3)
        acc = np.tile(accs, 3 * slos.size)
        w = W.Workload("tiny", 2, rows, task, slo, acc, 0, 0, "grid")
        run_stateful(w, state, load, n_threads=2)


def test_set_states_rejects_bad_values_and_keeps_the_catalog():
    import paper_1905_13348_b200 as P
    w = W.make("C1")
    cat = P.infaas_catalog_load(w.rows, w.n_tasks)
    try:
        bad = np.full(w.n_variants, ACTIVE, np.uint8); bad[3] = 4
        with pytest.raises(P.InfaasError) as e:
            P.infaas_catalog_set_states(cat, bad, None)
        assert e.value.code == -10
        got = _to_host_u32(gpu_select(cat, w.task, w.slo_us, w.min_acc_bp))
        assert np.array_equal(got, OracleCatalog(w.rows, w.n_tasks).select(w.task, w.slo_us, w.min_acc_bp))
    finally:
        cat.free()
