"""The C-ABI library loads and exports every entry point the header declares (no GPU needed)."""
import ctypes
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _declared():
    text = open(os.path.join(ROOT, "include", "libra.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(libra_[a-z_]+)\s*\(", text)))


def test_header_declares_the_north_star_calls():
    names = _declared()
    for need in ("libra_plan_tiles", "libra_attn_pool_fwd", "libra_attn_pool_bwd"):
        assert need in names


def test_library_exports_every_declared_symbol():
    from paper_2607_23250_b200 import build
    so = build.build()
    lib = ctypes.CDLL(so)
    for name in _declared():
        assert hasattr(lib, name), name


def test_strerror_and_argument_checks_without_a_device():
    from paper_2607_23250_b200 import build
    lib = ctypes.CDLL(build.build())
    lib.libra_strerror.restype = ctypes.c_char_p
    assert lib.libra_strerror(0) == b"ok"
    assert b"timed out" in lib.libra_strerror(-6)
    # null pointers are rejected before any CUDA call
    h = ctypes.c_void_p()
    assert lib.libra_plan_tiles(None, 1, 1, 128, None, None, ctypes.byref(h)) == -1
    assert lib.libra_attn_pool_fwd(None, None, None, None, None, None, None, None, None) == -1
    assert lib.libra_plan_destroy(None) == 0
    assert lib.libra_launch_count() >= 0


def test_binding_names_match_header():
    src = open(os.path.join(ROOT, "paper_2607_23250_b200", "binding.py")).read()
    for name in _declared():
        assert name in src, name
