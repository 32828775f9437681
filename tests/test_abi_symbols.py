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


def test_host_side_queries_and_checks_of_the_new_entry_points(lib):
    # the capacity query is the budget total of Sec. 3.2.2 capped at the sequence length, summed over sequences:
    # checked against the oracle's total_budget on a ragged batch, without a device
    from oracle import flashcache_oracle as O
    lib.fc_layer_capacity_rows.restype = ctypes.c_int64
    lib.fc_layer_capacity_rows.argtypes = [ctypes.c_int32, ctypes.c_int32, ctypes.POINTER(ctypes.c_int32),
                                           ctypes.c_double, ctypes.c_int32]
    for lens, L, rho, mk in (([32768], 28, 0.1, 1), ([1024], 1, 0.2, 1), ([5, 0, 100, 7], 3, 0.9, 4),
                             ([10, 20], 4, 0.0, 2), ([8], 2, 1.0, 1)):
        cu = (ctypes.c_int32 * (len(lens) + 1))(*([0] + [sum(lens[:i + 1]) for i in range(len(lens))]))
        want = sum(min(n, O.total_budget(n, L, rho, mk)) for n in lens if n > 0)
        assert lib.fc_layer_capacity_rows(L, len(lens), cu, rho, mk) == want
    assert lib.fc_layer_capacity_rows(0, 1, cu, 0.5, 1) == -1
    assert lib.fc_layer_capacity_rows(1, 1, None, 0.5, 1) == -1
    # null handles and pointers are refused before any CUDA call
    assert lib.fc_select_compact_layers(None, None, None, 1, None, None, None, None, 0, None) == 1
    assert lib.fc_cutoff_from_spectrum(None, None, 0, None, ctypes.c_double(0.5), None, None, None) == 1
    assert lib.fc_proto_dft16_stage(None, None, None, 8, 0, 1, None) == 1
    assert lib.fc_measure_fp32_peak(None, None) == 1
    assert lib.fc_selftest_bounded_wait(None, None) == 1
    assert lib.fc_set_internal_streams(None, 2) == 1
    assert lib.fc_set_l2_persist(None, 1) == 1
