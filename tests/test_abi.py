"""The C-ABI library loads and exports every function include/ardiff.h declares (no GPU needed)."""
import ctypes
import os
import re
import subprocess

import paper_2512_08537_b200 as pkg
from paper_2512_08537_b200 import build as pkg_build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def declared_functions():
    text = open(os.path.join(ROOT, "include", "ardiff.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(ardiff_[a-z_0-9]+)\s*\(", text)))


def test_library_builds_loads_and_exports_all_declared_symbols():
    pkg_build.build()
    lib = ctypes.CDLL(pkg.LIB_PATH)
    names = declared_functions()
    assert "ardiff_entropy_gate" in names and "ardiff_head_sample" in names
    missing = [n for n in names if not hasattr(lib, n)]
    assert not missing, f"declared in ardiff.h but not exported: {missing}"


def test_library_exports_nothing_the_header_does_not_declare():
    pkg_build.build()
    out = subprocess.check_output(["nm", "-D", "--defined-only", pkg.LIB_PATH], text=True)
    exported = sorted(set(re.findall(r" T (ardiff_[a-z_0-9]+)$", out, flags=re.M)))
    extra = [n for n in exported if n not in declared_functions()]
    assert not extra, f"exported but not declared in ardiff.h: {extra}"


def test_strerror_and_version_need_no_gpu():
    assert pkg.version() >= 100
    assert pkg.strerror(0) == "ok"
    for code in range(-7, 0):
        assert "unknown" not in pkg.strerror(code)
    assert "unknown" in pkg.strerror(-99)
