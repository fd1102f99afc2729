"""Find the accuracy-quantile scale for the C4 query stream at which about 10 % of the
queries have no feasible variant.  Calls only the CPU oracle.  The value it prints is the
constant C4_ACC_QUANTILE_SCALE in the workload module.

    python tests/golden/calibrate_c4.py
"""
import os
import sys

import numpy as np

sys.path.insert(0, os.path.join(os.path.dirname(os.path.abspath(__file__)), "..", ".."))

from oracle import OracleCatalog  # noqa: E402
from paper_1905_13348_b200 import workloads as W  # noqa: E402


def infeasible_fraction(scale: float, n: int = 1 << 17) -> float:
    W.C4_ACC_QUANTILE_SCALE = scale
    w = W.config_c4(n)
    d = OracleCatalog(w.rows, w.n_tasks).select(w.task, w.slo_us, w.min_acc_bp, os.cpu_count())
    return float(np.mean((d >> 31) == 1))


if __name__ == "__main__":
    lo, hi = 0.0, 1.0
    for _ in range(12):
        mid = 0.5 * (lo + hi)
        f = infeasible_fraction(mid)
        print(f"scale {mid:.4f} -> infeasible {f:.4f}")
        if f > 0.10:
            hi = mid
        else:
            lo = mid
    print("C4_ACC_QUANTILE_SCALE =", round(0.5 * (lo + hi), 3))
