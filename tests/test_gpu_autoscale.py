"""GPU parity of the Model-Autoscaler's scaling-up step (Section 4.2.2) against the CPU
oracle: same tallies, instances, loading latencies and SLOs on both sides, bit for bit."""
import numpy as np
import pytest

from oracle import AUTOSCALE_ESCALATE, AUTOSCALE_NONE, OracleCatalog, autoscale_step
from paper_1905_13348_b200 import workloads as W
from tests.helpers import rows_from
from tests.test_gpu_parity import _to_host_u32, gpu_select

pytestmark = pytest.mark.gpu


def gpu_step(cat, window_us, slack, lam):
    import torch
    import paper_1905_13348_b200 as P
    v = torch.full((cat.n_tasks,), 0x5A5A5A5A, dtype=torch.int32, device="cuda")
    d = torch.full((cat.n_tasks,), 0x5A5A5A5A, dtype=torch.int32, device="cuda")
    P.infaas_autoscale_step(cat, window_us, slack, lam, v, d)
    torch.cuda.synchronize()
    return _to_host_u32(v), _to_host_u32(d)


@pytest.mark.parametrize("name,kw", [("C2", {"n_queries": 60_000}), ("C3", {"n_queries": 65_536}),
                                     ("C4", {"n_queries": 30_000}), ("C5", {"n_windows": 1, "window": 65_536})])
def test_step_on_the_tallies_of_a_window(name, kw):
    import paper_1905_13348_b200 as P
    w = W.make(name, **kw)
    rng = np.random.default_rng(51)
    cat = P.infaas_catalog_load(w.rows, w.n_tasks)
    o = OracleCatalog(w.rows, w.n_tasks)
    try:
        want_dec = o.select(w.task, w.slo_us, w.min_acc_bp, 8)
        d_dec = gpu_select(cat, w.task, w.slo_us, w.min_acc_bp)
        assert np.array_equal(_to_host_u32(d_dec), want_dec)
        P.infaas_tally(cat, d_dec)                               # pending counts, not yet advanced
        ok = want_dec[(want_dec >> 31) == 0]
        count = np.bincount(ok, minlength=w.n_variants).astype(np.uint32)
        load = rng.integers(590_000, 11_000_000, w.n_variants).astype(np.uint32)
        P.infaas_catalog_set_states(cat, np.ones(w.n_variants, np.uint8), load)   # all Active: same lists
        P.infaas_tally(cat, d_dec[:0])
        seen = set()
        for trial in range(6):
            inst = (rng.integers(1, 4, w.n_variants) * ((count > 0) & (rng.random(w.n_variants) < 0.7))).astype(np.uint32)
            if trial == 5:
                inst[:] = 0                                      # nothing runs anywhere
            slo = rng.choice(np.array([3_000, 30_000, 300_000, 3_000_000], np.uint32), w.n_tasks)
            window_us = int(rng.choice([2_000, 40_000, 1_000_000]))
            slack, lam = int(rng.choice([100, 105, 200])), int(rng.choice([0, 100, 10_000]))
            P.infaas_autoscale_config(cat, inst, slo)
            gv, gd = gpu_step(cat, window_us, slack, lam)
            ov, od = autoscale_step(w.rows, w.n_tasks, count, inst, load, slo, window_us, slack, lam)
            assert np.array_equal(gv, ov) and np.array_equal(gd, od), (trial, np.flatnonzero(gv != ov)[:5])
            seen |= {"none" if x == AUTOSCALE_NONE else "escalate" if x == AUTOSCALE_ESCALATE else "act" for x in ov}
        assert "act" in seen and len(seen) >= 2, seen
        # the step leaves the pending counts alone: the update still sees them
        P.infaas_advance(cat, 1000)
        o.load_update(want_dec, 1000)
        st = P.infaas_catalog_get_state(cat)
        assert np.array_equal(st["queued"], o.queued) and np.array_equal(st["served_total"], o.served_total)
    finally:
        cat.free()


def test_worked_example_and_saturation_on_gpu():
    import torch
    import paper_1905_13348_b200 as P
    # Tables 2 and 3: A (200 ms, 5/s, cost 1), B (20 ms, 100/s, 3), C (15 ms, 800/s, 16), one architecture
    rows = rows_from([0] * 3, [1, 2, 12], [200_000, 20_000, 15_000], [7600] * 3, [1, 3, 16])
    rows["arch"] = 7
    cat = P.infaas_catalog_load(rows, 1)
    try:
        for qps, slo, running, want in ((10, 300_000, [1, 0, 0], (0, 1)), (10, 50_000, [0, 0, 0], (1, 1)),
                                        (1000, 300_000, [0, 2, 0], (2, 1))):
            served_by = int(np.argmax(running)) if any(running) else 0
            dec = torch.full((qps,), served_by, dtype=torch.int32, device="cuda")
            P.infaas_tally(cat, dec)
            P.infaas_autoscale_config(cat, running, [slo])
            gv, gd = gpu_step(cat, 1_000_000, 100, 0)
            assert (int(gv[0]), int(gd[0])) == want
            P.infaas_advance(cat, 1_000_000)                     # clears the pending counts
    finally:
        cat.free()
    # extreme values: the saturating paths
    rows = rows_from([0, 0, 1], [65535, 1, 1], [1, 2**32 - 1, 10**9], [7000] * 3, [2**32 - 1, 1, 1])
    cat = P.infaas_catalog_load(rows, 2)
    try:
        dec = torch.cat([torch.zeros(70_000, dtype=torch.int32), torch.full((3,), 2, dtype=torch.int32)]).cuda()
        P.infaas_tally(cat, dec)
        count = np.array([70_000, 0, 3], np.uint32)
        load = np.array([2**32 - 1, 0, 5], np.uint32)
        P.infaas_catalog_set_states(cat, np.ones(3, np.uint8), load)
        for inst, window_us, slack, lam in (([2**32 - 1, 0, 0], 1, 2**32 - 1, 0), ([1, 0, 0], 1, 100, 2**32 - 1),
                                            ([0, 1, 336_666_666], 3, 101, 7), ([0, 0, 0], 1, 2**32 - 1, 2**32 - 1)):
            inst = np.array(inst, np.uint32)
            slo = np.array([2**32 - 1, 2**32 - 1], np.uint32)
            P.infaas_autoscale_config(cat, inst, slo)
            gv, gd = gpu_step(cat, window_us, slack, lam)
            ov, od = autoscale_step(rows, 2, count, inst, load, slo, window_us, slack, lam)
            assert np.array_equal(gv, ov) and np.array_equal(gd, od), (inst, gv, ov, gd, od)
    finally:
        cat.free()


def test_step_argument_errors():
    import torch
    import paper_1905_13348_b200 as P
    w = W.make("C1")
    cat = P.infaas_catalog_load(w.rows, w.n_tasks)
    try:
        out = torch.zeros(1, dtype=torch.int32, device="cuda")
        with pytest.raises(P.InfaasError) as e:                  # config never called
            P.infaas_autoscale_step(cat, 1000, 105, 0, out, out.clone())
        assert e.value.code == -11
        P.infaas_autoscale_config(cat, np.zeros(w.n_variants, np.uint32), np.array([1000], np.uint32))
        with pytest.raises(P.InfaasError) as e:
            P.infaas_autoscale_step(cat, 0, 105, 0, out, out.clone())
        assert e.value.code == -11
    finally:
        cat.free()
