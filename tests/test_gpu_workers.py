"""GPU parity of the worker choice (Section 4.1, Case I) against the CPU oracle."""
import numpy as np
import pytest

from oracle import OracleCatalog, assign_workers
from paper_1905_13348_b200 import workloads as W
from tests.helpers import INVALID, NO_FEASIBLE_BIT
from tests.test_gpu_parity import _to_dev, _to_host_u32, gpu_select

pytestmark = pytest.mark.gpu


def gpu_assign(cat, dec):
    import torch
    import paper_1905_13348_b200 as P
    d_dec = _to_dev(dec) if dec.size else torch.empty(0, dtype=torch.int32, device="cuda")
    d_w = torch.full((dec.shape[0],), 0x5A5A5A5A, dtype=torch.int32, device="cuda")
    P.infaas_assign_workers(cat, d_dec, d_w)
    torch.cuda.synchronize()
    return _to_host_u32(d_w)


def tables(rng, w, n_workers, frac_loaded, dup):
    """Instance table: a share of the variants runs on 1..dup workers; some rows point nowhere."""
    loaded = np.flatnonzero(rng.random(w.n_variants) < frac_loaded)
    iv = np.repeat(loaded, rng.integers(1, dup + 1, loaded.size))
    iw = rng.integers(0, n_workers, iv.size)
    il = rng.integers(0, 50, iv.size)                         # equal loads are common
    junk = rng.integers(w.n_variants, 2**32, 7, dtype=np.uint64)          # variants that do not exist
    k = loaded[:3].size                                                   # workers that do not exist
    iv = np.concatenate([iv, junk, loaded[:3]])
    iw = np.concatenate([iw, rng.integers(0, n_workers, 7), rng.integers(n_workers, 2**32, k, dtype=np.uint64)])
    il = np.concatenate([il, np.zeros(7 + k, np.int64)])                  # the lowest load, were they counted
    p = rng.permutation(iv.size)
    hw = rng.integers(0, 5, n_workers).astype(np.uint8)       # the catalogs use codes 0..3: code 4 is never wanted
    ut = rng.integers(0, 100, n_workers).astype(np.uint32)
    return iv[p].astype(np.uint32), iw[p].astype(np.uint32), il[p].astype(np.uint32), hw, ut


@pytest.mark.parametrize("name,kw,n_workers", [("C1", {}, 3), ("C2", {"n_queries": 100_003}, 40),
                                               ("C3", {"n_queries": 300_001}, 500),
                                               ("C5", {"n_windows": 2, "window": 65_536}, 2000)])
def test_workers_for_a_batch_of_decisions(name, kw, n_workers):
    import paper_1905_13348_b200 as P
    w = W.make(name, **kw)
    rng = np.random.default_rng(61)
    cat = P.infaas_catalog_load(w.rows, w.n_tasks)
    try:
        dec = _to_host_u32(gpu_select(cat, w.task, w.slo_us, w.min_acc_bp))
        assert np.array_equal(dec, OracleCatalog(w.rows, w.n_tasks).select(w.task, w.slo_us, w.min_acc_bp, 8))
        dec[:5] = [INVALID, w.n_variants, NO_FEASIBLE_BIT, 0x7FFFFFFF, w.n_variants - 1]
        for frac in (0.0, 0.3, 1.0):
            iv, iw, il, hw, ut = tables(rng, w, n_workers, frac, 4)
            P.infaas_workers_config(cat, iv, iw, il, hw, ut)
            want_per_variant = assign_workers(w.rows, iv, iw, il, hw, ut, np.arange(w.n_variants, dtype=np.uint32))
            want = np.where(dec < w.n_variants, want_per_variant[np.minimum(dec, w.n_variants - 1)], INVALID)
            sample = rng.choice(dec.size, 300, replace=False)    # the oracle itself, query by query
            assert np.array_equal(want[sample], assign_workers(w.rows, iv, iw, il, hw, ut, dec[sample]))
            got = gpu_assign(cat, dec)
            assert np.array_equal(got, want.astype(np.uint32)), np.flatnonzero(got != want)[:5]
        for n in (0, 1, 2, 3, 5, 1023):                          # ragged sizes
            assert np.array_equal(gpu_assign(cat, dec[:n]), want[:n].astype(np.uint32))
        P.infaas_workers_config(cat, [], [], [], [], [])         # no workers at all
        assert np.all(gpu_assign(cat, dec[:1000]) == INVALID)
    finally:
        cat.free()


def test_assign_before_config_is_an_error():
    import torch
    import paper_1905_13348_b200 as P
    w = W.make("C1")
    cat = P.infaas_catalog_load(w.rows, w.n_tasks)
    try:
        d = torch.zeros(4, dtype=torch.int32, device="cuda")
        with pytest.raises(P.InfaasError) as e:
            P.infaas_assign_workers(cat, d, d.clone())
        assert e.value.code == -11
    finally:
        cat.free()
