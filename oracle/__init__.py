"""CPU oracle (test infrastructure only; never imported by the CUDA path)."""
from .oracle import OracleCatalog, build, pred_lat  # noqa: F401
