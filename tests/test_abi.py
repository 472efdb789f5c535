"""Host-only checks of the C-ABI boundary: the library loads, exports every symbol the header
declares, and rejects bad shapes before touching a device."""
import ctypes
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def api():
    from paper_1910_02120_b200 import build
    build.build()
    from paper_1910_02120_b200 import api as a
    return a


def test_every_declared_symbol_is_exported(api):
    header = open(os.path.join(ROOT, "include", "ist.h")).read()
    header = re.sub(r"/\*.*?\*/", "", header, flags=re.S)
    declared = set(re.findall(r"\b(ist_[a-z0-9_]+)\s*\(", header))
    assert declared, "no declarations found"
    assert declared == set(api.EXPORTS)
    for name in declared:
        assert hasattr(api.lib, name), name
        getattr(api.lib, name)


def test_workspace_bytes_validates_shapes(api):
    assert api.ist_workspace_bytes([784, 1024, 10], 2, api.IST_FP32, 128) > 0
    assert api.ist_workspace_bytes([784, 1024, 10], 0, api.IST_FP32, 128) == 0      # S < 1
    assert api.ist_workspace_bytes([784, 10], 2, api.IST_FP32, 128) == 0            # no hidden layer, S > 1
    assert api.ist_workspace_bytes([784, 10], 1, api.IST_FP32, 128) > 0
    assert api.ist_workspace_bytes([8, 4, 3], 5, api.IST_FP32, 16) == 0             # S > hidden width
    assert api.ist_workspace_bytes([8, 4, 3], 2, 7, 16) == 0                        # bad precision
    assert api.ist_workspace_bytes([8, 4, 3], 2, api.IST_BF16, 0) == 0              # bad batch
    assert api.ist_workspace_bytes([8, 0, 3], 1, api.IST_BF16, 4) == 0              # zero width


def test_workspace_grows_with_shape_and_holds_the_slices(api):
    small = api.ist_workspace_bytes([1024, 4096, 4096, 35], 4, api.IST_BF16, 256)
    big = api.ist_workspace_bytes([3072, 16384, 16384, 10], 8, api.IST_BF16, 512)
    assert big > small
    # packed fp32 masters + bf16 copies of the wide config: 84.1M elements * 6 bytes at least
    elems = 3072 * 16384 + 16384 * 16384 // 8 + 16384 * 10
    assert big >= elems * 6


def test_create_rejects_bad_workspace_without_a_device(api):
    dims = (ctypes.c_int64 * 3)(8, 4, 3)
    h = ctypes.c_void_p()
    st = api.lib.ist_create(ctypes.byref(h), dims, 3, 2, api.IST_FP32, 4, 0, None, 0, None)
    assert st == api.IST_ERR_WORKSPACE and not h.value
    assert b"workspace" in api.lib.ist_last_error(None)
    st = api.lib.ist_create(ctypes.byref(h), dims, 3, 9, api.IST_FP32, 4, 0, None, 0, None)
    assert st == api.IST_ERR_ARG
    st = api.lib.ist_create(ctypes.byref(h), dims, 3, 2, api.IST_FP32, 4, 0, ctypes.c_void_p(256), 16, None)
    assert st == api.IST_ERR_WORKSPACE
    assert api.lib.ist_partition(None, 1) == api.IST_ERR_ARG


def test_slice_shape_and_static_status_need_no_device_to_refuse(api):
    r, c = ctypes.c_int64(-1), ctypes.c_int64(-1)
    assert api.lib.ist_subnet_slice_shape(None, 1, 0, ctypes.byref(r), ctypes.byref(c)) == api.IST_ERR_ARG
    assert (r.value, c.value) == (-1, -1)
    assert api.ist_workspace_bytes([8, 4, 3], 2, api.IST_FP32, 65536) == 0           # batch beyond a launch grid's rows
    assert api.ist_workspace_bytes([8, 4, 3], 2, api.IST_FP32, 65535) > 0


def test_normalisation_entry_points_reject_null_contexts(api):
    assert api.lib.ist_norm_workspace_bytes(None) == 0
    assert api.lib.ist_enable_normalization(None, ctypes.c_float(1e-5), None, 0) == api.IST_ERR_ARG
    assert api.lib.ist_calibrate(None, None, 1) == api.IST_ERR_ARG


def test_partition_rule_is_validated_and_sizes_the_layout(api):
    dims = [64, 4096, 4096, 10]
    bal = api.ist_workspace_bytes2(dims, 8, api.IST_BF16, 128, False, api.IST_PART_BALANCED)
    iid = api.ist_workspace_bytes2(dims, 8, api.IST_BF16, 128, False, api.IST_PART_IID)
    assert bal == api.ist_workspace_bytes(dims, 8, api.IST_BF16, 128)
    assert iid > bal                                  # room for mean + 7 sigma neurons per subnet
    assert api.ist_workspace_bytes2(dims, 8, api.IST_BF16, 128, False, 7) == 0
    one_iid = api.ist_workspace_bytes2(dims, 1, api.IST_BF16, 128, False, api.IST_PART_IID)
    assert one_iid == api.ist_workspace_bytes2(dims, 1, api.IST_BF16, 128, False, api.IST_PART_BALANCED)   # one group holds all
    dims_c = (ctypes.c_int64 * 3)(8, 4, 3)
    h = ctypes.c_void_p()
    st = api.lib.ist_create2(ctypes.byref(h), dims_c, 3, 2, api.IST_FP32, 4, 0, 5, ctypes.c_void_p(256), 1 << 20, None)
    assert st == api.IST_ERR_ARG and not h.value
