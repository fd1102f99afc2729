"""Pins for the worker-choice part of the CPU oracle (Section 4.1, Case I): a restatement by
sorting, library routines for the special cases, invariants, invariance under reordering."""
import numpy as np
import pytest

from oracle import assign_workers
from tests.helpers import INVALID, NO_FEASIBLE_BIT, rows_from


def _rows(nv, hw):
    r = rows_from([0] * nv, [1] * nv, [100] * nv, [7000] * nv, [1] * nv)
    r["hw"] = hw
    return r


def plain(rows, iv, iw, il, hw, ut, d):
    if d & NO_FEASIBLE_BIT or d >= len(rows):
        return INVALID
    mine = sorted((int(l), int(w)) for v, w, l in zip(iv, iw, il) if v == d and w < len(hw))
    if mine:
        return mine[0][1]
    cand = sorted((int(ut[w]), w) for w in range(len(hw)) if hw[w] == rows["hw"][d])
    return cand[0][1] if cand else INVALID


@pytest.mark.parametrize("seed", range(8))
def test_against_sorting(seed):
    rng = np.random.default_rng(400 + seed)
    nv, nw, ni = int(rng.integers(1, 12)), int(rng.integers(1, 7)), int(rng.integers(0, 25))
    if seed % 2:
        nv, nw, ni = int(rng.integers(1, 4)), int(rng.integers(3, 9)), 40      # many instances per variant
    rows = _rows(nv, rng.integers(0, 3, nv))
    iv, iw = rng.integers(0, nv + 1, ni), rng.integers(0, nw + 1, ni)     # some rows point nowhere
    il = rng.integers(0, 4, ni)                                          # many equal loads
    hw, ut = rng.integers(0, 3, nw), rng.integers(0, 3, nw)
    dec = np.concatenate([np.arange(nv + 2), np.arange(nv) | NO_FEASIBLE_BIT, [INVALID]]).astype(np.uint32)
    got = assign_workers(rows, iv, iw, il, hw, ut, dec)
    assert [int(x) for x in got] == [plain(rows, iv, iw, il, hw, ut, int(d)) for d in dec]


@pytest.mark.parametrize("seed", range(6))
def test_against_sorting_mostly_unloaded(seed):
    """Most variants have no instance, so the choice falls to the utilisation rule, with few
    distinct utilisations: equal ones must go to the lower worker id."""
    rng = np.random.default_rng(500 + seed)
    nv, nw = int(rng.integers(6, 20)), int(rng.integers(3, 12))
    rows = _rows(nv, rng.integers(0, 2, nv))
    loaded = rng.choice(nv, 2, replace=False)
    iv, iw, il = np.repeat(loaded, 2), rng.integers(0, nw, 4), rng.integers(0, 3, 4)
    hw, ut = rng.integers(0, 2, nw), rng.integers(0, 2, nw)
    dec = np.arange(nv, dtype=np.uint32)
    got = assign_workers(rows, iv, iw, il, hw, ut, dec)
    assert [int(x) for x in got] == [plain(rows, iv, iw, il, hw, ut, int(d)) for d in dec]


def test_equal_utilisation_goes_to_the_lowest_worker_id():
    rows = _rows(2, [0, 1])
    none = np.zeros(0, np.uint32)
    # three workers with the variant's hardware and the same utilisation -> worker 0
    assert int(assign_workers(rows, none, none, none, [0, 0, 0], [5, 5, 5], [0])[0]) == 0
    # the first two lack the hardware; of the equal rest the lowest id
    assert int(assign_workers(rows, none, none, none, [0, 0, 1, 1, 1], [1, 1, 7, 7, 7], [1])[0]) == 2
    # a lower utilisation later in the table still wins
    assert int(assign_workers(rows, none, none, none, [0, 0, 0], [5, 5, 4], [0])[0]) == 2
    # equal loads of a variant's instances -> lower worker id, whatever the table order
    assert int(assign_workers(rows, [0, 0, 0], [2, 1, 3], [4, 4, 4], [0] * 4, [0] * 4, [0])[0]) == 1


def test_special_cases_reduce_to_argmin():
    rng = np.random.default_rng(42)
    nv, nw = 50, 40
    rows = _rows(nv, np.zeros(nv, np.uint8))
    hw, ut = np.zeros(nw, np.uint8), rng.permutation(nw).astype(np.uint32)
    none = np.zeros(0, np.uint32)
    dec = np.arange(nv, dtype=np.uint32)
    # nothing is loaded and all workers have the hardware: everybody goes to the idlest worker
    assert np.all(assign_workers(rows, none, none, none, hw, ut, dec) == int(np.argmin(ut)))
    # every variant runs on every worker with distinct loads: the least-loaded worker per variant
    load = np.stack([rng.permutation(nw) for _ in range(nv)]).astype(np.uint32)
    iv, iw = np.repeat(np.arange(nv), nw), np.tile(np.arange(nw), nv)
    got = assign_workers(rows, iv, iw, load.ravel(), hw, ut, dec)
    assert np.array_equal(got, np.argmin(load, axis=1).astype(np.uint32))
    # the order of the instance table does not matter
    p = rng.permutation(iv.size)
    assert np.array_equal(got, assign_workers(rows, iv[p], iw[p], load.ravel()[p], hw, ut, dec))
    # a loaded variant goes to its own worker even if an idle worker with its hardware exists
    assert int(assign_workers(rows, [3], [7], [10**9], hw, np.zeros(nw, np.uint32), [3])[0]) == 7
    # no worker has the hardware
    rows["hw"][5] = 9
    assert int(assign_workers(rows, none, none, none, hw, ut, [5])[0]) == INVALID
