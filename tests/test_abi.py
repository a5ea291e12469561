"""CPU-side checks of the boundary: the library builds and loads, exports every
symbol the header declares, and rejects malformed arguments without a GPU."""
import ctypes
import os
import re

import numpy as np
import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    from paper_2507_20055_b200 import build
    build.build()
    from paper_2507_20055_b200 import binding
    return binding


def _declared_functions():
    text = open(os.path.join(ROOT, "include", "cert.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(cert_[a-z_0-9]+)\s*\(", text)))


def test_every_declared_symbol_is_exported(lib):
    names = _declared_functions()
    assert {"cert_net_create", "cert_deeppoly_bounds", "cert_net_destroy"} <= set(names)
    for n in names:
        assert hasattr(lib.lib, n), f"{n} declared in cert.h but not exported"
    assert sorted(lib.EXPORTS) == names


def test_struct_layout_matches_header(lib):
    # 12 ints followed by two pointers
    assert ctypes.sizeof(lib.cert_layer_desc_t) == 12 * 4 + 2 * ctypes.sizeof(ctypes.c_void_p)


def test_status_strings(lib):
    assert lib.lib.cert_status_string(0) == b"ok"
    assert b"batch" in lib.lib.cert_status_string(4)


def test_create_rejects_bad_arguments_without_gpu(lib):
    from paper_2507_20055_b200 import workloads as wl
    L = lib.lib
    h = ctypes.c_void_p()
    w = wl.small_fc([4, 5, 3], batch=1, eps=0.1)
    arr, keep = lib.marshal_layers(w.layers)
    assert L.cert_net_create(None, 2, 1, 0.0, 1.0, ctypes.byref(h)) == 1
    assert L.cert_net_create(arr, 0, 1, 0.0, 1.0, ctypes.byref(h)) == 1
    assert L.cert_net_create(arr, 2, 0, 0.0, 1.0, ctypes.byref(h)) == 1
    assert L.cert_net_create(arr, 2, 1, 1.0, 0.0, ctypes.byref(h)) == 1
    assert L.cert_net_create(arr, 2, 1, 0.0, 1.0, None) == 1
    # layer chain mismatch
    bad = wl.small_fc([4, 5, 3], batch=1, eps=0.1).layers
    bad[1].weight = np.zeros((3, 6), np.float32)
    arr2, keep2 = lib.marshal_layers(bad)
    assert L.cert_net_create(arr2, 2, 1, 0.0, 1.0, ctypes.byref(h)) == 1
    # null weights
    arr3, keep3 = lib.marshal_layers(w.layers)
    arr3[0].weight = None
    assert L.cert_net_create(arr3, 2, 1, 0.0, 1.0, ctypes.byref(h)) == 1
    # bad conv geometry
    c = wl.small_conv((1, 4, 4), [(2, 3, 1, 0)], [3], batch=1, eps=0.1).layers
    arr4, keep4 = lib.marshal_layers(c)
    arr4[0].stride = 0
    assert L.cert_net_create(arr4, 2, 1, 0.0, 1.0, ctypes.byref(h)) == 1
    assert h.value is None


def test_null_handles(lib):
    L = lib.lib
    assert L.cert_net_num_neurons(None) == -1
    assert L.cert_net_destroy(None) == 1
    assert L.cert_deeppoly_bounds(None, None, 0.1, 1, None, None, None) == 1
    assert L.cert_net_set_contraction(None, 0) == 1


def test_product_does_not_import_the_oracle():
    pkg = os.path.join(ROOT, "paper_2507_20055_b200")
    for dirpath, _, files in os.walk(pkg):
        for f in files:
            if f.endswith((".py", ".cu", ".cuh", ".h")):
                text = open(os.path.join(dirpath, f)).read()
                assert not re.search(r"(from|import)\s+oracle|oracle[/\\.]|liboracle|deeppoly_oracle", text), \
                    f"{f} reaches into the oracle"
    for f in os.listdir(os.path.join(ROOT, "oracle")):
        if f.endswith((".py", ".c")):
            text = open(os.path.join(ROOT, "oracle", f)).read()
            assert "paper_2507_20055_b200" not in text and "cert.h" not in text


def test_null_handles_of_the_other_entry_points(lib):
    L = lib.lib
    assert L.cert_backsub_bounds(None, None, 0.1, 1, None, None, None, None) == 1
    assert L.cert_backsub_bounds_host(None, None, 0.1, 1, None, None, None, None) == 1
    assert L.cert_reusecert_bounds(None, None, 0.1, 1, None, None, None) == 1
    assert L.cert_reusecert_bounds_host(None, None, 0.1, 1, None, None, None) == 1
    assert L.cert_net_enable_reusecert(None) == 1
    assert L.cert_net_set_conv_patches(None, 1) == 1
    assert b"fp16" in L.cert_status_string(7)


def test_null_handles_and_bad_arguments_of_the_helpers(lib):
    L = lib.lib
    assert L.cert_net_check_guards(None, None) == -1
    assert L.cert_net_auto_contraction(None) == -1
    assert L.cert_net_fp16_coefficient_bound(None, 0) == -1.0
    assert L.cert_net_selftest_checked_store(None, None) == 1
    assert L.cert_built_with_checked_stores() == (1 if os.environ.get("CERT_LIB", "").endswith("_checked.so") else 0)
    # the peak micro-kernels validate their arguments before they touch the device
    out = ctypes.c_double()
    assert L.cert_peak_microbench(4, 5.0, ctypes.byref(out), None, None, None) == 1
    assert L.cert_peak_microbench(0, 0.0, ctypes.byref(out), None, None, None) == 1
    assert L.cert_peak_microbench(0, 5000.0, ctypes.byref(out), None, None, None) == 1
    assert L.cert_peak_microbench(0, 5.0, None, None, None, None) == 1
    assert b"checked store" in L.cert_status_string(8)


def test_the_checking_build_exports_the_same_symbols():
    """The same sources with -DCERT_BOUNDS (paper_2507_20055_b200/build.py --checked) load and export every symbol."""
    from paper_2507_20055_b200 import build
    checked = ctypes.CDLL(build.build_checked())
    for n in _declared_functions():
        assert hasattr(checked, n), f"{n} missing from the checking build"
    checked.cert_built_with_checked_stores.restype = ctypes.c_int
    assert checked.cert_built_with_checked_stores() == 1
