"""The C-ABI library loads without a GPU and exports every symbol the public
header declares; host-side argument checks work without launching anything."""
import ctypes
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def built_lib():
    from paper_1602_06709_b200 import build
    build.build()
    from paper_1602_06709_b200 import binding
    return binding


def test_every_declared_symbol_is_exported(built_lib):
    header = open(os.path.join(ROOT, "include", "pcl_dnn.h")).read()
    header = re.sub(r"/\*.*?\*/", "", header, flags=re.S)
    declared = set(re.findall(r"\b(pcl_[a-z0-9_]+)\s*\(", header))
    assert declared, "no declarations found"
    lib = built_lib.lib()
    for name in sorted(declared):
        assert hasattr(lib, name), f"{name} declared in pcl_dnn.h but not exported"
    assert declared == set(built_lib.EXPORTS)


def test_host_side_checks(built_lib):
    B = built_lib
    d = B.conv_desc(2, 8, 8, 5, 5, 3, 3, 1, 1)
    assert B.conv_out_dims(d) == (5, 5)
    d4 = B.conv_desc(256, 3, 96, 231, 231, 11, 11, 4, 0)
    assert B.conv_out_dims(d4) == (56, 56)
    bad = B.conv_desc(2, 8, 8, 2, 2, 5, 5, 1, 0)       # kernel larger than the padded input
    with pytest.raises(B.PclError) as e:
        B.conv_out_dims(bad)
    assert e.value.code == B.ERR_BAD_ARG
    L = B.lib()
    null = ctypes.c_void_p(0)
    assert L.pcl_conv_fwd(ctypes.byref(d), null, null, null, null, 0, null, 0, null) == B.ERR_BAD_ARG
    assert L.pcl_conv_fwd(ctypes.byref(d), ctypes.c_void_p(4), ctypes.c_void_p(16), null, ctypes.c_void_p(16), 0,
                          null, 0, null) == B.ERR_MISALIGNED
    assert L.pcl_conv_fwd(ctypes.byref(d), ctypes.c_void_p(16), ctypes.c_void_p(16), null, ctypes.c_void_p(16), 7,
                          null, 0, null) == B.ERR_BAD_ARG
    # a pass that needs workspace refuses a missing one before touching the device
    # (C % 32 != 0: backward-data makes a transposed copy of the weights, whose room is mandatory)
    big = B.conv_desc(8, 40, 64, 28, 28, 3, 3, 1, 1)
    # (room for the transposed weights, plus scratch for a split reduction where the layer has few tiles)
    assert B.conv_workspace_bytes(big, B.PASS_BWD_DATA) >= 40 * 64 * 9 * 4
    wide = B.conv_desc(256, 256, 256, 56, 56, 3, 3, 1, 1)      # thousands of tiles: no split, the weights' room only
    assert B.conv_workspace_bytes(wide, B.PASS_BWD_DATA) == 256 * 256 * 9 * 4
    assert B.conv_workspace_bytes(wide, B.PASS_FWD) == 0
    assert L.pcl_conv_bwd_data(ctypes.byref(big), ctypes.c_void_p(16), ctypes.c_void_p(16), null, ctypes.c_void_p(16),
                               null, 0, null) == B.ERR_WORKSPACE
    assert L.pcl_maxpool2x2_fwd(1, 3, 4, 4, ctypes.c_void_p(16), ctypes.c_void_p(16), null) == B.ERR_UNSUPPORTED_SHAPE
    assert L.pcl_sgd_update(null, null, 0, 0.1, null) == B.OK
    assert B.status_string(B.ERR_DEVICE_TIMEOUT) == "device-side wait timed out"
    assert L.pcl_set_path(9) == B.ERR_BAD_ARG
    # launcher choices are pinned through the ABI only; an unknown knob is refused
    assert L.pcl_set_tuning(b"TILING", 1) == B.OK and L.pcl_set_tuning(b"NO_SUCH_KNOB", 1) == B.ERR_BAD_ARG
    assert L.pcl_set_tuning(None, 1) == B.ERR_BAD_ARG and L.pcl_reset_tuning() == B.OK
