"""CPU-side checks of the boundary: the shared library builds, loads and exports every symbol that
include/sla.h declares, and argument validation that needs no device works."""
import ctypes
import re
from pathlib import Path

from paper_2602_01744_b200 import api, build

ROOT = Path(__file__).resolve().parent.parent


def declared_symbols():
    text = (ROOT / "include" / "sla.h").read_text()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(sla_[a-z_0-9]+)\s*\(", text)))


def test_library_builds_and_exports_every_declared_symbol():
    so = build.build()
    L = ctypes.CDLL(str(so))
    names = declared_symbols()
    assert {"sla_plan_create", "sla_forward", "sla_backward", "sla_decode_step"} <= set(names)
    for name in names:
        assert hasattr(L, name), name
    assert set(api.EXPORTS) <= set(names)


def test_status_strings_and_null_arguments():
    L = api.lib()
    assert L.sla_status_string(0) == b"ok"
    assert b"workspace" in L.sla_status_string(3)
    assert L.sla_plan_create(None, None) == 1
    h = ctypes.c_void_p()
    bad = api.sla_desc(4, 1, 1, 1, 64, 4, 128, 128, 64, 1.0, 0)       # wrong struct_size
    assert L.sla_plan_create(ctypes.byref(h), ctypes.byref(bad)) == 1
    assert L.sla_plan_destroy(None) == 0
    assert L.sla_forward(*([None] * 11), None, 0, None) == 1
