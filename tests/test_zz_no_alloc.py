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

from oracle import ops
from paper_2006_12575_b200 import binding as B
from paper_2006_12575_b200 import synth

from _util import REL_L2, MAX_ABS, assert_close, dev_bf16, host_f64

pytestmark = pytest.mark.gpu


def _layer(C_in, C_out, dhw, seed, k=3, s=1, p=1, tr=0):
    D, H, W = dhw
    o = (lambda n: 2 * n) if tr else (lambda n: (n + 2 * p - k) // s + 1)
    dy = dev_bf16(synth.normal_bf16((1, o(D), o(H), o(W), C_out), seed))
    w = dev_bf16(synth.kaiming_bf16(k ** 3, C_out, C_in, (1 if tr else k ** 3) * C_in, seed + 1))
    return B.conv_desc(C_in, C_out, k, s, p, tr), dy, w, (1, D, H, W, C_in)


def _reference(desc, dy, w, shape, dtype=torch.bfloat16):
    dx = torch.full(shape, float("nan"), dtype=dtype, device="cuda")
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


def test_static_scratch_dgrad_matches_the_oracle_for_every_conv_variant():
    """The same entry point against the CPU oracle (not only against the workspace form): 3x3x3 stride 1 and
    stride 2, the 2x2x2 transposed conv, an fp32 dx, and a small layer right after a large one (the array
    then still holds most of the large layer's weights behind the part the small layer rewrites)."""
    cases = [dict(C_in=64, C_out=128, dhw=(8, 12, 20), seed=51),
             dict(C_in=32, C_out=32, dhw=(5, 6, 9), seed=52),                        # small after large
             dict(C_in=32, C_out=64, dhw=(8, 8, 12), seed=53, s=2),                  # stride-2 conv
             dict(C_in=128, C_out=64, dhw=(4, 5, 6), seed=54, k=2, s=2, p=0, tr=1),  # transposed conv
             dict(C_in=64, C_out=64, dhw=(6, 33, 9), seed=55)]
    for c in cases:
        k, st, p, tr = c.get("k", 3), c.get("s", 1), c.get("p", 1), c.get("tr", 0)
        desc, dy, w, shape = _layer(c["C_in"], c["C_out"], c["dhw"], c["seed"], k, st, p, tr)
        dy64, w64 = host_f64(dy), host_f64(w)
        ref = ops.convT3d_dgrad(dy64, w64, c["dhw"], k, st) if tr else ops.conv3d_dgrad(dy64, w64, c["dhw"], k, st, p)
        for dtype in (torch.float32, torch.bfloat16):
            dx = torch.full(shape, float("nan"), dtype=dtype, device="cuda")
            B.lamp_conv3d_dgrad_static_scratch(desc, dy, w, dx)
            assert B.lamp_get_async_status() == 0
            if dtype == torch.float32:
                assert_close(host_f64(dx), ref, f"static-scratch dgrad vs oracle {c}", rel=2e-5, mx=2e-5)
            else:
                assert_close(host_f64(dx), ops.bf16_round(ref), f"static-scratch dgrad (bf16) vs oracle {c}", rel=REL_L2, mx=MAX_ABS)
            again, _ = _reference(desc, dy, w, shape, dtype)
            assert torch.equal(dx, again)


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
