"""Windows shared out over ranks: index arithmetic, and a world-size-2 run over gloo on the CPU
in which each rank decides its share with the oracle, the per-variant counts are summed over
the ranks, and every rank must reach the state a single process reaches on the whole window."""
import os
import socket

import numpy as np
import pytest

from paper_1905_13348_b200 import sharding as S


@pytest.mark.parametrize("n", [0, 1, 127, 128, 129, 1000, 65536, 65537, 10**6 + 3])
@pytest.mark.parametrize("world", [1, 2, 3, 4, 8])
def test_shard_bounds_partition_the_range(n, world):
    prev = 0
    sizes = []
    for r in range(world):
        lo, hi = S.shard_bounds(n, world, r)
        assert lo == prev and lo <= hi <= n
        assert lo % S.ALIGN == 0 or lo == n
        sizes.append(hi - lo)
        prev = hi
    assert prev == n and sum(sizes) == n
    assert max(sizes) - min(sizes) <= S.ALIGN
    with pytest.raises(ValueError):
        S.shard_bounds(n, world, world)


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _rank_main(rank, world, port, n_queries, window, out_dir):
    import torch
    import torch.distributed as dist

    from oracle import OracleCatalog
    from paper_1905_13348_b200 import workloads as W

    os.environ["MASTER_ADDR"], os.environ["MASTER_PORT"] = "127.0.0.1", str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        w = W.make("C3", n_queries=n_queries, window=window)
        w.window_us = 400                      # little drain: the queues (and answers) move
        nv = w.n_variants
        mine = OracleCatalog(w.rows, w.n_tasks)            # this rank's copy of the catalog
        whole = OracleCatalog(w.rows, w.n_tasks)           # what one process would do
        for k in range(n_queries // window):
            base = k * window
            lo, hi = S.shard_bounds(window, world, rank)
            sl = slice(base + lo, base + hi)
            pending = np.zeros(nv, np.int64)

            def select():
                return mine.select(w.task[sl], w.slo_us[sl], w.min_acc_bp[sl])

            def tally(d):
                pending[:] += np.bincount(d[d < nv], minlength=nv)

            def advance(window_us):
                # the oracle advances from decisions: one decision per counted query
                mine.load_update(np.repeat(np.arange(nv, dtype=np.uint32), pending), window_us)

            box = {}
            d = S.sharded_window(select, tally, lambda: torch.from_numpy(pending.copy()),
                                 lambda t: pending.__setitem__(slice(None), t.numpy()), advance,
                                 w.window_us)
            box["d"] = d
            ws = slice(base, base + window)
            want = whole.select(w.task[ws], w.slo_us[ws], w.min_acc_bp[ws])
            whole.load_update(want, w.window_us)
            assert np.array_equal(d, want[lo:hi]), (rank, k)
            assert np.array_equal(mine.queued, whole.queued), (rank, k)
            assert np.array_equal(mine.served_total, whole.served_total), (rank, k)
        assert mine.queued.max() > 0
        assert S.max_over_ranks(float(rank)) == float(world - 1)
        open(os.path.join(out_dir, f"ok{rank}"), "w").write("ok")
    finally:
        dist.destroy_process_group()


def test_two_ranks_over_gloo_reach_the_single_process_state(tmp_path):
    import torch.multiprocessing as mp
    world = 2
    mp.spawn(_rank_main, args=(world, _free_port(), 6 * 2048, 2048, str(tmp_path)), nprocs=world, join=True)
    assert all((tmp_path / f"ok{r}").exists() for r in range(world))
