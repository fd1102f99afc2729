"""CPU oracle (test infrastructure only; never imported by the CUDA path)."""
from .oracle import (ACTIVE, AUTOSCALE_ESCALATE, AUTOSCALE_NONE, INACTIVE, INTERFERED,  # noqa: F401
                     OVERLOADED, OracleCatalog, StatefulOracleCatalog, assign_workers, autoscale_step,
                     build, pred_lat)
