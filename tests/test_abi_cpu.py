"""CPU-side checks of the boundary: the shared library builds for sm_100a,
loads without a GPU, and exports every function include/dscale.h declares.
No compute call is made here."""
import ctypes
import os
import re

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _declared():
    text = open(os.path.join(ROOT, "include", "dscale.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(dscale_[a-z0-9_]+)\s*\(", text)))


def test_library_builds_loads_and_exports_every_declared_symbol():
    from paper_2609_37532_b200.build import build
    path = build()
    lib = ctypes.CDLL(path)
    names = _declared()
    assert {"dscale_alloc_verify", "dscale_verify_attn", "dscale_accept",
            "dscale_workspace_bytes", "dscale_workspace_init"} <= set(names)
    for n in names:
        assert hasattr(lib, n), f"{n} declared in dscale.h but not exported"


def test_workspace_size_is_pure_host_arithmetic():
    from paper_2609_37532_b200.build import build
    lib = ctypes.CDLL(build())
    lib.dscale_workspace_bytes.restype = ctypes.c_size_t
    a = lib.dscale_workspace_bytes(32, 32, 8, 128, 148)
    b = lib.dscale_workspace_bytes(64, 32, 8, 128, 148)
    assert 0 < a < b < (64 << 20)
    assert a % 256 == 0
    assert lib.dscale_workspace_bytes(0, 32, 8, 128, 148) == 0
    assert lib.dscale_workspace_bytes(65, 32, 8, 128, 148) == 0


def test_binding_has_no_cpu_fallback():
    """The product package must not import the oracle."""
    pkg = os.path.join(ROOT, "paper_2609_37532_b200")
    for dirpath, _, files in os.walk(pkg):
        for f in files:
            if f.endswith((".py", ".cu", ".cuh", ".h")):
                src = open(os.path.join(dirpath, f)).read()
                assert "oracle" not in src, f"{f} mentions the oracle"
