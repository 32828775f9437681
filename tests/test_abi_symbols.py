"""The C-ABI library loads without a GPU and exports every function that
include/flashcache.h declares; host-side argument checks answer without a device."""
import ctypes
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    from paper_2511_16786_b200 import build
    path = build.build()
    return ctypes.CDLL(path)


def _declared():
    names = set()
    for fn in os.listdir(os.path.join(ROOT, "include")):
        if fn.endswith(".h"):
            text = open(os.path.join(ROOT, "include", fn)).read()
            text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
            names |= set(re.findall(r"\b(fc_[a-z_0-9]+)\s*\(", text))
    return names


def test_every_declared_function_is_exported(lib):
    names = _declared()
    assert {"fc_score_layer", "fc_allocate_budgets", "fc_select_compact", "fc_create", "fc_destroy"} <= names
    for n in sorted(names):
        assert hasattr(lib, n), "missing export %s" % n


def test_binding_lists_the_same_entry_points():
    from paper_2511_16786_b200 import binding
    assert set(binding.EXPORTS) == _declared()
    for n in ("fc_score_layer", "fc_allocate_budgets", "fc_select_compact"):
        assert callable(getattr(binding, n))


def test_status_strings(lib):
    lib.fc_status_string.restype = ctypes.c_char_p
    seen = {lib.fc_status_string(i) for i in range(7)}
    assert len(seen) == 7 and lib.fc_status_string(0) == b"ok"
    assert lib.fc_status_string(99) == b"unknown status"


def test_null_arguments_are_rejected_on_the_host(lib):
    lib.fc_score_workspace_bytes.restype = ctypes.c_size_t
    assert lib.fc_score_workspace_bytes(None, None) == 0
    assert lib.fc_create(None, 0, 1024) == 1                     # FC_ERR_INVALID_ARG
    h = ctypes.c_void_p()
    assert lib.fc_create(ctypes.byref(h), 0, 0) == 2             # FC_ERR_UNSUPPORTED, before any CUDA call
    assert lib.fc_score_layer(None, None, ctypes.c_double(0.2), None, None, None, 0, None) == 1
    assert lib.fc_allocate_budgets(None, None, 1, 1, None, ctypes.c_double(0.2), 1, None, None, None) == 1
    assert lib.fc_select_compact(None, None, None, None, None, None, None, None, 0, None, 0, None) == 1
    lib.fc_destroy(None)


def test_oracle_is_not_imported_by_the_product():
    pkg = os.path.join(ROOT, "paper_2511_16786_b200")
    for dirpath, _, files in os.walk(pkg):
        for fn in files:
            if fn.endswith((".py", ".cu", ".cuh", ".h")):
                assert "oracle" not in open(os.path.join(dirpath, fn)).read().replace("CPU oracle", ""), fn
