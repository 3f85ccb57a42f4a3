"""The C-ABI library loads and exports every function include/bi.h declares
(no compute call is made: this runs without a GPU)."""
import ctypes
import os
import re

import paper_2607_17855_b200 as bi

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def declared_functions():
    text = open(os.path.join(ROOT, "include", "bi.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    names = re.findall(r"^\s*(?:const\s+)?(?:int|int64_t|char)\s*\*?\s*(bi_[a-z0-9_]+)\s*\(", text, flags=re.M)
    return sorted(set(names))


def test_header_and_library_agree():
    names = declared_functions()
    assert {"bi_model_create", "bi_model_destroy", "bi_filter", "bi_vmp", "bi_mmp", "bi_status",
            "bi_strerror", "bi_filter_static"} <= set(names)
    lib = ctypes.CDLL(bi.build())
    for name in names:
        assert hasattr(lib, name), f"{name} is declared in bi.h but not exported"
    # the binding names every export too
    assert set(names) == set(bi.EXPORTS)


def test_error_strings_and_null_handling_without_a_device():
    L = bi.lib()
    assert L.bi_strerror(0) == b"ok"
    for code in (-1, -2, -3, -4, -5):
        assert L.bi_strerror(code) not in (b"", b"unknown error")
    assert L.bi_strerror(-99) == b"unknown error"
    assert L.bi_model_destroy(None) == 0
    assert L.bi_model_arith(None) == -1
    assert L.bi_launch_count(None) == 0
    out = ctypes.c_void_p()
    assert L.bi_model_create(None, None, ctypes.byref(out)) == -1 and not out.value


def test_binding_refuses_to_compute_without_cuda():
    import pytest
    import torch
    if torch.cuda.is_available():
        pytest.skip("a GPU is present")
    with pytest.raises(RuntimeError):
        bi.Model([2], [2], [[0]], [1], 1, [], [], [])
