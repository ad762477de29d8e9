"""The C-ABI library builds for sm_100a, loads without a GPU and exports every function include/qgemm.h declares."""
import ctypes
import os
import re

from paper_2607_19438_b200 import binding, build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def declared_functions():
    text = open(os.path.join(ROOT, "include", "qgemm.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b((?:qg|qgemm|moe|prefill)_\w+)\s*\(", text)))


def test_library_builds_loads_and_exports_every_declared_symbol():
    path = build.build()
    lib = ctypes.CDLL(path)
    names = declared_functions()
    assert {"qgemm_dense", "moe_route", "moe_grouped_qgemm", "moe_combine"} <= set(names)
    for n in names:
        assert hasattr(lib, n), f"missing export {n}"
    assert set(binding.EXPORTS) <= set(names)


def test_strerror_and_workspace_are_host_only():
    lib = binding.load()
    assert binding.strerror(0) == "ok"
    assert "NULL" in binding.strerror(-1)
    assert binding.route_workspace_bytes(2048, 128, 8) == 64 * 128 * 4
    assert binding.route_workspace_bytes(0, 128, 8) > 0
    assert lib.qg_destroy(None) == -1


def test_product_path_never_touches_the_oracle():
    pkg = os.path.join(ROOT, "paper_2607_19438_b200")
    for dirpath, _, files in os.walk(pkg):
        for f in files:
            if f.endswith((".py", ".cu", ".cuh", ".h")):
                src = open(os.path.join(dirpath, f)).read()
                for needle in ("import oracle", "from oracle", "liboracle", "oracle/", "oracle."):
                    assert needle not in src, f"{f} reaches into the oracle ({needle})"
