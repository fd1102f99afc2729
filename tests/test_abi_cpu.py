"""No-GPU checks of the C-ABI library: it builds, loads, exports every symbol the header
declares, and rejects bad catalogs on the host before any CUDA call."""
import ctypes
import os
import re

import numpy as np
import pytest

from paper_1905_13348_b200 import build as B
from paper_1905_13348_b200 import workloads as W
from tests.helpers import rows_from

ROOT = os.path.join(os.path.dirname(__file__), "..")


@pytest.fixture(scope="module")
def lib():
    return ctypes.CDLL(B.build())


def declared_functions():
    text = open(os.path.join(ROOT, "include", "infaas.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(infaas_[a-z_0-9]+)\s*\(", text)))


def test_every_declared_symbol_is_exported(lib):
    names = declared_functions()
    assert {"infaas_catalog_load", "infaas_select_batch", "infaas_load_update"} <= set(names)
    for n in names:
        assert hasattr(lib, n), n


def test_row_struct_is_24_bytes_and_matches_generator_dtype():
    assert W.VARIANT_DTYPE.itemsize == 24
    offs = {k: W.VARIANT_DTYPE.fields[k][1] for k in W.VARIANT_DTYPE.names}
    assert offs == {"task": 0, "arch": 2, "hw": 4, "opt": 5, "batch": 6, "lat_us": 8,
                    "acc_bp": 12, "reserved": 14, "cost": 16, "queued": 20}


def _load(lib, rows, n_tasks):
    out = ctypes.c_void_p(None)
    lib.infaas_catalog_load.argtypes = [ctypes.c_void_p, ctypes.c_uint32, ctypes.c_uint32,
                                        ctypes.c_int, ctypes.POINTER(ctypes.c_void_p)]
    rc = lib.infaas_catalog_load(rows.ctypes.data if rows is not None else None,
                                 0 if rows is None else rows.shape[0], n_tasks, 0, ctypes.byref(out))
    assert rc != 0 and out.value is None
    return rc


def test_host_side_validation_codes(lib):
    good = rows_from([0, 1], [1, 1], [10, 10], [7000, 7000], [1, 1])
    assert _load(lib, None, 1) == -1
    assert _load(lib, good, 0) == -2 and _load(lib, good, 70000) == -2
    assert _load(lib, good, 1) == -2                        # row task 1 >= n_tasks 1
    for field, value, code in (("batch", 0, -3), ("lat_us", 0, -4), ("acc_bp", 10001, -5),
                               ("reserved", 1, -5)):
        bad = good.copy(); bad[field][1] = value
        assert _load(lib, bad, 2) == code, field
    big = rows_from([0] * 8193, [1] * 8193, [10] * 8193, [7000] * 8193, [1] * 8193)
    assert _load(lib, big, 1) == -6                         # above the per-task limit
    lib.infaas_strerror.restype = ctypes.c_char_p
    for code in range(-10, 1):
        assert lib.infaas_strerror(code)
    lib.infaas_catalog_free(None)                           # NULL is allowed


def test_binding_fails_loudly_without_device():
    import torch
    if torch.cuda.is_available():
        pytest.skip("a device is present")
    import paper_1905_13348_b200 as P
    with pytest.raises(P.InfaasError):
        P.infaas_catalog_load(W.make("C1").rows, 1)


def test_binding_constants_match_the_header():
    text = open(os.path.join(ROOT, "include", "infaas.h")).read()
    defs = {m.group(1): int(m.group(2).rstrip("u"), 0)
            for m in re.finditer(r"#define\s+(INFAAS_[A-Z_]+)\s+\(?(-?(?:0x[0-9A-Fa-f]+|\d+)u?)\)?", text)}
    from paper_1905_13348_b200 import binding as b
    assert defs["INFAAS_NO_FEASIBLE"] == b.NO_FEASIBLE and defs["INFAAS_INVALID"] == b.INVALID
    assert [defs[f"INFAAS_STATE_{n}"] for n in ("INACTIVE", "ACTIVE", "OVERLOADED", "INTERFERED")] == \
        [b.STATE_INACTIVE, b.STATE_ACTIVE, b.STATE_OVERLOADED, b.STATE_INTERFERED]
    assert defs["INFAAS_AUTOSCALE_NONE"] == b.AUTOSCALE_NONE and defs["INFAAS_AUTOSCALE_ESCALATE"] == b.AUTOSCALE_ESCALATE
    assert sorted(b.EXPORTS) == sorted(n for n in declared_functions())
    codes = sorted(v for k, v in defs.items() if k.startswith("INFAAS_E_"))
    assert codes == list(range(-11, 0))
