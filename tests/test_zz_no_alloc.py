"""The allocation-free tally entry point against the regular path (collected last).

Some callers of this library cannot allocate device memory when they need tallies: a
serving process whose memory pool already owns the device's free memory, or a dispatch loop
that must not stall on an allocation.  `infaas_tally_static` counts into a fixed array
inside the library instead.  Here its counts must equal what `infaas_load_update` adds to
the catalog's per-variant totals, bit for bit, on two calls in a row (the second call
finds the first call's numbers in the shared array and has to clear them)."""
import numpy as np
import pytest

from paper_1905_13348_b200 import workloads as W

pytestmark = pytest.mark.gpu


def test_static_tally_matches_load_update_twice():
    import torch

    import paper_1905_13348_b200 as P

    w = W.make("C2", n_queries=16)
    rng = np.random.default_rng(21)
    cat = P.infaas_catalog_load(w.rows, w.n_tasks)
    d_count = torch.full((w.n_variants,), -1, dtype=torch.int32, device="cuda")
    d_counters = torch.full((3,), -1, dtype=torch.int64, device="cuda")
    served_before = np.zeros(w.n_variants, np.uint64)
    counters_before = np.zeros(3, np.uint64)
    for call, n in enumerate((50_003, 7_001)):
        dec = rng.integers(0, w.n_variants, n).astype(np.uint32)
        dec[::5] |= 0x80000000
        dec[::17] = 0xFFFFFFFF
        dec[3::19] = w.n_variants + call
        dec[100:2000] = 42 + call
        d_dec = torch.from_numpy(dec.view(np.int32)).cuda()
        P.infaas_tally_static(d_dec, w.n_variants, d_count, d_counters)
        P.infaas_load_update(cat, d_dec, 1000)
        st = P.infaas_catalog_get_state(cat)
        torch.cuda.synchronize()
        got = d_count.cpu().numpy().view(np.uint32).astype(np.uint64)
        assert np.array_equal(got, st["served_total"] - served_before), call
        assert np.array_equal(d_counters.cpu().numpy().view(np.uint64), st["counters"] - counters_before), call
        assert int(got.sum()) == int((st["counters"] - counters_before)[0])
        served_before, counters_before = st["served_total"].copy(), st["counters"].copy()
    cat.free()


def test_static_tally_large_batch_near_the_size_limit():
    """A batch large enough for the shared-memory histogram kernel over a catalog just below
    the array's limit (the ids are counted in two ranges then), against numpy, twice."""
    import torch

    import paper_1905_13348_b200 as P

    nv = 60_001
    rng = np.random.default_rng(22)
    d_count = torch.full((nv,), -1, dtype=torch.int32, device="cuda")
    d_counters = torch.full((3,), -1, dtype=torch.int64, device="cuda")
    for n in ((1 << 18) + 13, (1 << 19) + 1):
        dec = rng.integers(0, nv, n).astype(np.uint32)
        dec[::7] |= 0x80000000
        dec[::31] = 0xFFFFFFFF
        dec[5::41] = nv + 5
        dec[1000:60000] = nv - 1                     # a hot variant in the upper range
        d_dec = torch.from_numpy(dec.view(np.int32)).cuda()
        P.infaas_tally_static(d_dec, nv, d_count, d_counters)
        torch.cuda.synchronize()
        feas = dec[dec < nv]
        assert np.array_equal(d_count.cpu().numpy().view(np.uint32), np.bincount(feas, minlength=nv).astype(np.uint32))
        flagged = ((dec >> 31) == 1) & (dec != 0xFFFFFFFF)
        want = [feas.size, int(flagged.sum()), int(n - feas.size - flagged.sum())]
        assert d_counters.cpu().numpy().tolist() == want


def test_static_tally_rejects_sizes_beyond_its_array():
    import torch

    import paper_1905_13348_b200 as P
    from paper_1905_13348_b200.binding import InfaasError

    d_dec = torch.zeros(16, dtype=torch.int32, device="cuda")
    d_count = torch.zeros(65537, dtype=torch.int32, device="cuda")
    d_counters = torch.zeros(3, dtype=torch.int64, device="cuda")
    with pytest.raises(InfaasError) as e:
        P.infaas_tally_static(d_dec, 65537, d_count, d_counters)
    assert e.value.code == -6
