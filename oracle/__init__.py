"""CPU oracle (test infrastructure only; never imported by the CUDA path)."""
from .oracle import (ACTIVE, INACTIVE, INTERFERED, OVERLOADED, OracleCatalog,  # noqa: F401
                     StatefulOracleCatalog, build, pred_lat)
