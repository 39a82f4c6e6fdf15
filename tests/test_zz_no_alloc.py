"""The allocation-free data-gradient entry point (collected last on purpose).

Some callers cannot allocate device memory when they call the library - a layer inside an engine
that owns all device memory, a loop where cudaMalloc's device-wide synchronisation is not allowed -
so they have no workspace to pass.  lamp_conv3d_dgrad_static_scratch keeps the scratch of the pass
in a fixed array inside the library instead.  Its result must equal lamp_conv3d_dgrad's, also when
the shared array still holds another layer's data from the call before.
"""
import numpy as np
import pytest
import torch

from paper_2006_12575_b200 import binding as B
from paper_2006_12575_b200 import synth

from _util import REL_L2, MAX_ABS, assert_close, dev_bf16, host_f64

pytestmark = pytest.mark.gpu


def _layer(C_in, C_out, dhw, seed, k=3, s=1, p=1):
    D, H, W = dhw
    o = lambda n: (n + 2 * p - k) // s + 1
    dy = dev_bf16(synth.normal_bf16((1, o(D), o(H), o(W), C_out), seed))
    w = dev_bf16(synth.kaiming_bf16(k ** 3, C_out, C_in, k ** 3 * C_in, seed + 1))
    return B.conv_desc(C_in, C_out, k, s, p), dy, w, (1, D, H, W, C_in)


def _reference(desc, dy, w, shape):
    dx = torch.full(shape, float("nan"), dtype=torch.bfloat16, device="cuda")
    # the smallest accepted workspace: the pass then runs exactly as it does on the static array
    nbytes = B.lamp_conv3d_workspace_min_bytes(desc, dx, B.PASS_DGRAD)
    ws = torch.empty(max(nbytes, 256), dtype=torch.uint8, device="cuda")
    B.lamp_conv3d_dgrad(desc, dy, w, dx, ws)
    return dx, nbytes


def test_static_scratch_dgrad_equals_workspace_dgrad_on_consecutive_calls():
    # two different layers back to back: the second call finds the first one's weights in the array
    layers = [_layer(64, 128, (8, 12, 20), 11), _layer(128, 64, (9, 7, 16), 21), _layer(64, 128, (8, 12, 20), 11)]
    for desc, dy, w, shape in layers:
        ref, nbytes = _reference(desc, dy, w, shape)
        assert 0 < nbytes <= B.STATIC_SCRATCH_BYTES          # this layer does use scratch
        dx = torch.full(shape, float("nan"), dtype=torch.bfloat16, device="cuda")
        B.lamp_conv3d_dgrad_static_scratch(desc, dy, w, dx)
        assert B.lamp_get_async_status() == 0
        assert_close(host_f64(dx), host_f64(ref), "static-scratch dgrad", rel=REL_L2, mx=MAX_ABS)
        assert torch.equal(dx, ref)                          # same kernels, same inputs: same bits


def test_static_scratch_dgrad_rejects_layers_beyond_the_limit_and_takes_scratch_free_variants():
    desc, dy, w, shape = _layer(512, 512, (2, 2, 4), 31)     # 27 * 512 * 512 * 2 B = 13.5 MiB of scratch
    dx = torch.zeros(shape, dtype=torch.bfloat16, device="cuda")
    assert B.lamp_conv3d_workspace_min_bytes(desc, dx, B.PASS_DGRAD) > B.STATIC_SCRATCH_BYTES
    with pytest.raises(B.LampError) as e:
        B.lamp_conv3d_dgrad_static_scratch(desc, dy, w, dx)
    assert e.value.status == 7 and "scratch" in str(e.value)
    assert (dx == 0).all()                                   # nothing was launched
    # the 1x1x1 conv's data gradient needs no scratch at all
    desc, dy, w, shape = _layer(16, 32, (8, 6, 10), 41, k=1, s=1, p=0)
    ref, nbytes = _reference(desc, dy, w, shape)
    assert nbytes == 0
    dx = torch.full(shape, float("nan"), dtype=torch.bfloat16, device="cuda")
    B.lamp_conv3d_dgrad_static_scratch(desc, dy, w, dx)
    assert torch.equal(dx, ref)
