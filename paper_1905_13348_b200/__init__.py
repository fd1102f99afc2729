"""Batched model-variant selection and load tallies on B200 (C-ABI CUDA library + binding).

`workloads` (input generators) imports without the CUDA library; the binding's functions
are resolved lazily and raise if the library has not been built.
"""
from . import workloads  # noqa: F401

_BINDING = ("infaas_catalog_load", "infaas_select_batch", "infaas_load_update",
            "infaas_catalog_get_state", "infaas_catalog_get_frontier", "infaas_tally_static", "infaas_catalog_get_info",
            "infaas_intpipe_probe", "infaas_select_update",
            "infaas_tally", "infaas_pending_counts", "infaas_advance", "infaas_catalog_set_states",
            "infaas_catalog_get_states", "STATE_INACTIVE", "STATE_ACTIVE", "STATE_OVERLOADED",
            "STATE_INTERFERED", "infaas_autoscale_config", "infaas_autoscale_step", "AUTOSCALE_NONE",
            "AUTOSCALE_ESCALATE", "infaas_workers_config", "infaas_assign_workers", "Catalog", "InfaasError",
            "NO_FEASIBLE", "INVALID")


def __getattr__(name):
    if name in _BINDING:
        from . import binding
        return getattr(binding, name)
    raise AttributeError(name)
