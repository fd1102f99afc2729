"""Host-side logic for windows shared out over several ranks (one process per GPU).

Queries of a window are independent given the load snapshot, so rank r decides a contiguous
share of them against its own copy of the catalog; the one exchange is the sum of the
per-variant counts (the load every worker reports, Section 4.2.2 / Section 5 of the paper),
after which every rank advances its catalog with the same counts.  This module holds only
index arithmetic and the `torch.distributed` calls; it works with any backend (NCCL on GPUs,
gloo in the CPU tests).
"""
from __future__ import annotations

ALIGN = 128   # shares start at multiples of this many queries (16-byte aligned sub-arrays)


def shard_bounds(n: int, world: int, rank: int, align: int = ALIGN) -> tuple[int, int]:
    """[lo, hi) of rank's share of n queries: contiguous, in rank order, disjoint, covering
    0..n, every boundary but the last a multiple of `align`, sizes differing by at most
    `align`."""
    if not (0 <= rank < world) or n < 0:
        raise ValueError("bad rank / world / n")
    blocks = -(-n // align)
    lo_b = blocks * rank // world
    hi_b = blocks * (rank + 1) // world
    return min(n, lo_b * align), min(n, hi_b * align)


def allreduce_sum_(t):
    """In-place sum over all ranks of a tensor of counts (no-op without a process group)."""
    import torch.distributed as dist
    if dist.is_available() and dist.is_initialized() and dist.get_world_size() > 1:
        dist.all_reduce(t, op=dist.ReduceOp.SUM)
    return t


def max_over_ranks(value: float, device=None) -> float:
    """Largest `value` over all ranks (timings are reported as the slowest rank's)."""
    import torch
    import torch.distributed as dist
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return float(value)
    t = torch.tensor([value], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def sharded_window(select, tally, export_counts, import_counts, advance, window_us: int):
    """One window on this rank: decide the share, tally it, sum the counts over the ranks,
    advance.  The five callables wrap the library (or, in the CPU tests, the oracle);
    `export_counts()` returns a tensor of counts that `import_counts(t)` takes back."""
    decisions = select()
    tally(decisions)
    counts = export_counts()
    allreduce_sum_(counts)
    import_counts(counts)
    advance(window_us)
    return decisions
