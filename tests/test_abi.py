"""Host-side checks of the C ABI (no GPU): the library loads, exports every declared symbol,
the host-only entry points work, and invalid arguments are rejected before any launch."""
import ctypes as C
import os
import re

import pytest

from oracle import unet as oracle_unet
from paper_2006_12575_b200 import binding as B

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def test_library_exports_every_declared_symbol():
    hdr = open(os.path.join(ROOT, "include", "lamp.h")).read()
    hdr = re.sub(r"/\*.*?\*/", "", hdr, flags=re.S)
    declared = sorted(set(re.findall(r"\b(lamp_[a-z0-9_]+)\s*\(", hdr)))
    assert len(declared) >= 20
    L = B.lib()
    for name in declared:
        assert hasattr(L, name), name
    assert sorted(B.EXPORTS) == declared
    assert B.lamp_version().startswith("lamp-b200")


def test_layer_plan_and_param_layout_agree_with_the_oracle_plan():
    for levels, ch, cpl, K in [(3, [8, 16, 32], 2, 4), (5, [32, 64, 128, 256, 512], 2, 10),
                               (5, [64, 128, 256, 512, 1024], 3, 10)]:
        net = B.lamp_unet_create(B.unet_spec(levels, ch, cpl, 1, K))
        lay = oracle_unet.unet_layers(oracle_unet.UNetSpec(levels, ch, cpl, 1, K))
        assert B.lamp_unet_num_layers(net) == len(lay)
        wo_expect, bo_expect = 0, 0
        for i, l in enumerate(lay):
            wo, bo, d = B.lamp_unet_param_layout(net, i)
            assert (d.c_in, d.c_out) == (l.c_in, l.c_out)
            assert d.ksize ** 3 == l.taps
            assert (d.stride, d.transposed) == {"conv": (1, 0), "down": (2, 0), "up": (2, 1), "head": (1, 0)}[l.kind]
            assert wo == wo_expect and bo == bo_expect and wo % 8 == 0
            wo_expect += (l.taps * l.c_in * l.c_out + 7) // 8 * 8
            bo_expect += l.c_out
        assert B.lamp_unet_weight_count(net) == wo_expect and B.lamp_unet_bias_count(net) == bo_expect
        B.lamp_unet_destroy(net)


def test_workspace_queries_scale_with_the_volume():
    net = B.lamp_unet_create(B.unet_spec(5, [32, 64, 128, 256, 512], 2, 1, 10))
    a = B.lamp_unet_workspace_bytes(net, 1, 64, 64, 64, B.MODE_INFER)
    b = B.lamp_unet_workspace_bytes(net, 1, 128, 128, 128, B.MODE_INFER)
    t = B.lamp_unet_workspace_bytes(net, 1, 128, 128, 128, B.MODE_TRAIN)
    assert 0 < a < b < t
    assert 7 * a < b < 9 * a
    # the largest network of the workload list must fit one 180 GB device with room to spare
    big = B.lamp_unet_create(B.unet_spec(5, [64, 128, 256, 512, 1024], 3, 1, 10))
    assert B.lamp_unet_workspace_bytes(big, 1, 192, 192, 64, B.MODE_TRAIN) < 60e9
    sw = B.lamp_sliding_window_workspace_bytes(net, 512, 512, 128, (64, 64, 64), 0.25, 8)
    assert 363 * 64 ** 3 * 10 * 4 < sw < 8e9
    B.lamp_unet_destroy(net)
    B.lamp_unet_destroy(big)


def test_invalid_arguments_are_rejected_on_the_host():
    L = B.lib()
    bad = [B.unet_spec(0, [8]), B.unet_spec(2, [8, 12]), B.unet_spec(2, [8, 16], num_classes=40),
           B.unet_spec(2, [8, 16], in_channels=3), B.unet_spec(1, [256])]
    for spec in bad:
        h = C.c_void_p()
        assert L.lamp_unet_create(C.byref(spec), C.byref(h)) in (1, 2)
    # the widest network of the paper (Sec. 3: 128 filters in the first encoder block) is accepted
    wide = B.lamp_unet_create(B.unet_spec(5, [128, 256, 512, 1024, 2048], 2, 1, 10))
    assert B.lamp_unet_weight_count(wide) > 500e6
    B.lamp_unet_destroy(wide)
    d = B.conv_desc(8, 8, 5, 1, 2)
    t = B.Tensor(16, B.LAMP_BF16, 1, 4, 4, 4, 8, 8, 0)
    assert L.lamp_conv3d_fwd(C.byref(d), C.byref(t), 16, None, C.byref(t), None, None, 0, None) == 2
    d = B.conv_desc(8, 8)
    assert L.lamp_conv3d_fwd(C.byref(d), None, 16, None, C.byref(t), None, None, 0, None) == 1
    t_odd = B.Tensor(8, B.LAMP_BF16, 1, 4, 4, 4, 8, 8, 0)                      # misaligned pointer
    assert L.lamp_conv3d_fwd(C.byref(d), C.byref(t_odd), 16, None, C.byref(t), None, None, 0, None) == 1
    t_c = B.Tensor(16, B.LAMP_BF16, 1, 4, 4, 4, 16, 16, 0)                     # channel mismatch
    assert L.lamp_conv3d_fwd(C.byref(d), C.byref(t_c), 16, None, C.byref(t), None, None, 0, None) == 1
    t_sz = B.Tensor(16, B.LAMP_BF16, 1, 4, 4, 5, 8, 8, 0)                      # output extent mismatch
    assert L.lamp_conv3d_fwd(C.byref(d), C.byref(t), 16, None, C.byref(t_sz), None, None, 0, None) == 1
    t_pitch = B.Tensor(16, B.LAMP_BF16, 1, 4, 4, 4, 8, 4, 0)                   # pitch smaller than the slice
    assert L.lamp_conv3d_fwd(C.byref(d), C.byref(t_pitch), 16, None, C.byref(t), None, None, 0, None) == 1
    net = B.lamp_unet_create(B.unet_spec(3, [8, 16, 32]))
    x = B.Tensor(256, B.LAMP_BF16, 1, 6, 8, 8, 1, 1, 0)                        # 6 not divisible by 4
    assert L.lamp_unet_forward(net, 16, 16, C.byref(x), 16, None, 256, 1 << 30, None) == 2
    x = B.Tensor(256, B.LAMP_BF16, 1, 8, 8, 8, 1, 1, 0)
    assert L.lamp_unet_forward(net, 16, 16, C.byref(x), 16, None, 256, 16, None) == 3       # workspace too small
    assert L.lamp_unet_forward(net, 16, 16, C.byref(x), 16, None, None, 0, None) == 3
    assert B.lamp_unet_workspace_bytes(net, 1, 0, 8, 8, 0) == 0
    B.lamp_unet_destroy(net)
    assert B.lib().lamp_status_string(5) == b"device-side wait timed out"
