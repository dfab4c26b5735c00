"""The C-ABI library loads without a GPU and exports every function include/tlr.h declares."""
import os
import re

import pytest


def declared_functions():
    root = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
    text = open(os.path.join(root, "include", "tlr.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(tlr_[a-z_]+)\s*\(", text)))


def test_header_declares_the_boundary():
    names = declared_functions()
    for must in ("tlr_create", "tlr_route", "tlr_route_host", "tlr_destroy", "tlr_status_string"):
        assert must in names


def test_library_exports_every_declared_symbol():
    from paper_2504_07878_b200 import build
    import paper_2504_07878_b200 as P
    build.build()
    lib = P.load_library()
    for name in declared_functions():
        assert hasattr(lib, name), name
    assert P.status_string(0) == "ok" and "argument" in P.status_string(1)


def test_no_gpu_means_an_error_not_a_fallback():
    import torch
    if torch.cuda.is_available():
        pytest.skip("a GPU is present")
    import ctypes
    import paper_2504_07878_b200 as P
    ctx = ctypes.c_void_p(0)
    code = P.load_library().tlr_create(64, 64, ctypes.c_void_p(256), 1, ctypes.byref(ctx))
    assert code != 0 and not ctx.value
