"""ctypes binding of liblamp.so: argument marshalling only.

Every function has the name of the C entry point it wraps (see include/lamp.h)
and does nothing but build descriptors and pass device pointers of torch
tensors; all arithmetic runs in the library's CUDA kernels.  There is no CPU
path: loading fails loudly when the library is missing.
"""
from __future__ import annotations

import ctypes as C
import os

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "liblamp.so")

LAMP_BF16, LAMP_F32 = 0, 1
PASS_FWD, PASS_DGRAD, PASS_WGRAD = 0, 1, 2
MODE_INFER, MODE_TRAIN = 0, 1


class LampError(RuntimeError):
    def __init__(self, status, what):
        self.status = int(status)
        super().__init__(f"{what}: lamp status {int(status)} ({lib().lamp_status_string(int(status)).decode()})")


class Tensor(C.Structure):
    _fields_ = [("ptr", C.c_void_p), ("dtype", C.c_int32), ("n", C.c_int32), ("d", C.c_int32), ("h", C.c_int32),
                ("w", C.c_int32), ("c", C.c_int32), ("c_pitch", C.c_int64), ("c_offset", C.c_int32)]


class ConvDesc(C.Structure):
    _fields_ = [("c_in", C.c_int32), ("c_out", C.c_int32), ("ksize", C.c_int32), ("stride", C.c_int32),
                ("pad", C.c_int32), ("transposed", C.c_int32)]


class UNetSpec(C.Structure):
    _fields_ = [("levels", C.c_int32), ("channels", C.c_int32 * 8), ("convs_per_level", C.c_int32),
                ("in_channels", C.c_int32), ("num_classes", C.c_int32), ("in_eps", C.c_float), ("se_ratio", C.c_int32)]


_lib = None


def lib():
    """Loads liblamp.so (built in-tree by build.py).  Raises if it is absent."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise RuntimeError(f"{LIB_PATH} not found: build it with `python -m paper_2006_12575_b200.build`")
        L = C.CDLL(LIB_PATH)
        vp, sz, i32, f32 = C.c_void_p, C.c_size_t, C.c_int32, C.c_float
        TP, DP, SP = C.POINTER(Tensor), C.POINTER(ConvDesc), C.POINTER(UNetSpec)
        I3 = C.POINTER(C.c_int32)
        sig = {
            "lamp_conv3d_workspace_bytes": (sz, [DP, TP, C.c_int]),
            "lamp_conv3d_workspace_min_bytes": (sz, [DP, TP, C.c_int]),
            "lamp_conv3d_fwd": (C.c_int, [DP, TP, vp, vp, TP, vp, vp, sz, vp]),
            "lamp_conv3d_dgrad": (C.c_int, [DP, TP, vp, TP, vp, sz, vp]),
            "lamp_conv3d_dgrad_static_scratch": (C.c_int, [DP, TP, vp, TP, vp]),
            "lamp_conv3d_wgrad": (C.c_int, [DP, TP, TP, vp, vp, vp, sz, vp]),
            "lamp_instnorm_relu_fwd": (C.c_int, [TP, vp, f32, vp, TP, vp]),
            "lamp_instnorm_relu_bwd": (C.c_int, [TP, TP, TP, vp, vp, TP, vp]),
            "lamp_se_squeeze": (C.c_int, [TP, vp, vp, vp]),
            "lamp_se_excite": (C.c_int, [vp, C.c_int64, i32, i32, i32, vp, vp, vp, vp, vp, vp, vp, vp]),
            "lamp_se_apply_fwd": (C.c_int, [TP, vp, vp, TP, TP, vp]),
            "lamp_se_bwd_reduce": (C.c_int, [TP, TP, vp, vp, vp]),
            "lamp_se_excite_bwd": (C.c_int, [vp, C.c_int64, i32, i32, i32, vp, vp, vp, vp, vp, vp, vp, vp, vp, vp, vp]),
            "lamp_se_apply_bwd": (C.c_int, [TP, vp, vp, TP, vp]),
            "lamp_unet_create": (C.c_int, [SP, C.POINTER(vp)]),
            "lamp_unet_se_layout": (C.c_int, [vp, i32, C.POINTER(sz), C.POINTER(i32)]),
            "lamp_unet_destroy": (None, [vp]),
            "lamp_unet_num_layers": (i32, [vp]),
            "lamp_unet_weight_count": (sz, [vp]),
            "lamp_unet_bias_count": (sz, [vp]),
            "lamp_unet_param_layout": (C.c_int, [vp, i32, C.POINTER(sz), C.POINTER(sz), DP]),
            "lamp_unet_workspace_bytes": (sz, [vp, i32, i32, i32, i32, i32]),
            "lamp_unet_tensor_layout": (C.c_int, [vp, i32, i32, i32, i32, i32, i32, i32, TP, C.POINTER(sz)]),
            "lamp_unet_forward": (C.c_int, [vp, vp, vp, TP, vp, vp, vp, sz, vp]),
            "lamp_unet_forward_layers": (C.c_int, [vp, vp, vp, TP, i32, i32, vp, vp, vp, sz, vp]),
            "lamp_unet_train_step": (C.c_int, [vp, vp, vp, TP, vp, vp, vp, vp, vp, vp, sz, vp]),
            "lamp_unet_train_step_buckets": (C.c_int, [vp, vp, vp, TP, vp, vp, vp, vp, vp, vp, sz, vp,
                                                       C.POINTER(C.c_int64), i32, C.POINTER(vp)]),
            "lamp_sliding_window_num_patches": (i32, [i32, i32, i32, I3, f32]),
            "lamp_sliding_window_partial": (C.c_int, [vp, vp, vp, TP, I3, f32, i32, i32, i32, i32, vp, vp, vp, sz, vp]),
            "lamp_sliding_window_finish": (C.c_int, [vp, vp, i32, C.c_int64, i32, vp, vp]),
            "lamp_sliding_window_workspace_bytes": (sz, [vp, i32, i32, i32, I3, f32, i32]),
            "lamp_sliding_window_infer": (C.c_int, [vp, vp, vp, TP, I3, f32, i32, i32, vp, vp, vp, sz, vp]),
            "lamp_overlap_add": (C.c_int, [vp, i32, i32, i32, i32, I3, f32, i32, vp, vp, vp]),
            "lamp_rmsprop_step": (C.c_int, [C.c_int64, vp, vp, vp, vp, f32, f32, f32, vp]),
            "lamp_get_async_status": (C.c_int, [vp]),
            "lamp_selftest_wait_timeout": (C.c_int, [vp]),
            "lamp_status_string": (C.c_char_p, [C.c_int]),
            "lamp_version": (C.c_char_p, []),
        }
        for name, (res, args) in sig.items():
            fn = getattr(L, name)
            fn.restype = res
            fn.argtypes = args
        _lib = L
    return _lib


EXPORTS = ["lamp_conv3d_workspace_bytes", "lamp_conv3d_workspace_min_bytes", "lamp_conv3d_fwd", "lamp_conv3d_dgrad", "lamp_conv3d_dgrad_static_scratch",
           "lamp_conv3d_wgrad",
           "lamp_instnorm_relu_fwd", "lamp_instnorm_relu_bwd",
           "lamp_se_squeeze", "lamp_se_excite", "lamp_se_apply_fwd", "lamp_se_bwd_reduce", "lamp_se_excite_bwd", "lamp_se_apply_bwd",
           "lamp_unet_create", "lamp_unet_se_layout", "lamp_unet_destroy",
           "lamp_unet_num_layers", "lamp_unet_weight_count", "lamp_unet_bias_count", "lamp_unet_param_layout",
           "lamp_unet_workspace_bytes", "lamp_unet_tensor_layout", "lamp_unet_forward", "lamp_unet_forward_layers", "lamp_unet_train_step",
           "lamp_unet_train_step_buckets", "lamp_sliding_window_num_patches", "lamp_sliding_window_partial",
           "lamp_sliding_window_finish",
           "lamp_sliding_window_workspace_bytes", "lamp_sliding_window_infer", "lamp_overlap_add",
           "lamp_rmsprop_step", "lamp_get_async_status", "lamp_selftest_wait_timeout", "lamp_status_string", "lamp_version"]


def _check(st, what):
    if st != 0:
        raise LampError(st, what)


def _stream():
    return C.c_void_p(torch.cuda.current_stream().cuda_stream)


def _ptr(t):
    return C.c_void_p(t.data_ptr()) if t is not None else None


def tensor(t: torch.Tensor, c=None, c_offset=0) -> Tensor:
    """Descriptor of a channel slice [c_offset, c_offset + c) of an NDHWC torch tensor [n,d,h,w,pitch]."""
    assert t.dim() == 5 and t.is_contiguous()
    dt = {torch.bfloat16: LAMP_BF16, torch.float32: LAMP_F32}[t.dtype]
    n, d, h, w, pitch = t.shape
    return Tensor(t.data_ptr(), dt, n, d, h, w, pitch - c_offset if c is None else c, pitch, c_offset)


def _td(x):
    return x if isinstance(x, Tensor) else tensor(x)


def conv_desc(c_in, c_out, ksize=3, stride=1, pad=1, transposed=0) -> ConvDesc:
    return ConvDesc(c_in, c_out, ksize, stride, pad, transposed)


def lamp_conv3d_workspace_bytes(desc, x, pass_):
    return lib().lamp_conv3d_workspace_bytes(C.byref(desc), C.byref(_td(x)), pass_)


def lamp_conv3d_workspace_min_bytes(desc, x, pass_):
    return lib().lamp_conv3d_workspace_min_bytes(C.byref(desc), C.byref(_td(x)), pass_)


def _ws(ws):
    return (_ptr(ws), ws.numel() * ws.element_size()) if ws is not None else (None, 0)


def lamp_conv3d_fwd(desc, x, w, bias, y, stats=None, ws=None):
    p, nbytes = _ws(ws)
    _check(lib().lamp_conv3d_fwd(C.byref(desc), C.byref(_td(x)), _ptr(w), _ptr(bias), C.byref(_td(y)), _ptr(stats),
                                 p, nbytes, _stream()), "lamp_conv3d_fwd")


def lamp_conv3d_dgrad(desc, dy, w, dx, ws=None):
    p, nbytes = _ws(ws)
    _check(lib().lamp_conv3d_dgrad(C.byref(desc), C.byref(_td(dy)), _ptr(w), C.byref(_td(dx)), p, nbytes, _stream()),
           "lamp_conv3d_dgrad")


STATIC_SCRATCH_BYTES = 4 * 1024 * 1024


def lamp_conv3d_dgrad_static_scratch(desc, dy, w, dx):
    """lamp_conv3d_dgrad without a caller workspace: the scratch is a fixed array inside the library
    (for callers that cannot allocate device memory at call time).  Raises LampError with status 7
    when the layer needs more than STATIC_SCRATCH_BYTES."""
    _check(lib().lamp_conv3d_dgrad_static_scratch(C.byref(desc), C.byref(_td(dy)), _ptr(w), C.byref(_td(dx)), _stream()),
           "lamp_conv3d_dgrad_static_scratch")


def lamp_conv3d_wgrad(desc, x, dy, dw, dbias=None, ws=None):
    p, nbytes = _ws(ws)
    _check(lib().lamp_conv3d_wgrad(C.byref(desc), C.byref(_td(x)), C.byref(_td(dy)), _ptr(dw), _ptr(dbias), p, nbytes,
                                   _stream()), "lamp_conv3d_wgrad")


def lamp_instnorm_relu_fwd(y, stats, eps, mu_rstd, z):
    _check(lib().lamp_instnorm_relu_fwd(C.byref(_td(y)), _ptr(stats), eps, _ptr(mu_rstd), C.byref(_td(z)), _stream()),
           "lamp_instnorm_relu_fwd")


def lamp_instnorm_relu_bwd(dz_a, dz_b, y, mu_rstd, sums, dy):
    b = C.byref(_td(dz_b)) if dz_b is not None else None
    _check(lib().lamp_instnorm_relu_bwd(C.byref(_td(dz_a)), b, C.byref(_td(y)), _ptr(mu_rstd), _ptr(sums),
                                        C.byref(_td(dy)), _stream()), "lamp_instnorm_relu_bwd")


def unet_spec(levels, channels, convs_per_level=2, in_channels=1, num_classes=4, eps=1e-5, se_ratio=0) -> UNetSpec:
    ch = (C.c_int32 * 8)(*(list(channels) + [0] * (8 - len(channels))))
    return UNetSpec(levels, ch, convs_per_level, in_channels, num_classes, eps, se_ratio)


def lamp_unet_create(spec: UNetSpec):
    h = C.c_void_p()
    _check(lib().lamp_unet_create(C.byref(spec), C.byref(h)), "lamp_unet_create")
    return h


def lamp_unet_destroy(net):
    lib().lamp_unet_destroy(net)


def lamp_unet_num_layers(net):
    return lib().lamp_unet_num_layers(net)


def lamp_unet_weight_count(net):
    return lib().lamp_unet_weight_count(net)


def lamp_unet_bias_count(net):
    return lib().lamp_unet_bias_count(net)


def lamp_unet_param_layout(net, layer):
    wo, bo, d = C.c_size_t(), C.c_size_t(), ConvDesc()
    _check(lib().lamp_unet_param_layout(net, layer, C.byref(wo), C.byref(bo), C.byref(d)), "lamp_unet_param_layout")
    return wo.value, bo.value, d


def lamp_unet_se_layout(net, layer):
    off, cr = C.c_size_t(), C.c_int32()
    _check(lib().lamp_unet_se_layout(net, layer, C.byref(off), C.byref(cr)), "lamp_unet_se_layout")
    return off.value, cr.value


def lamp_unet_workspace_bytes(net, n, d, h, w, mode):
    return lib().lamp_unet_workspace_bytes(net, n, d, h, w, mode)


T_IN, T_Y, T_OUT, T_STATS, T_MU_RSTD, T_DY, T_DIN, T_DOUT, T_DOUT2, T_PROBS = range(10)


def lamp_unet_tensor_layout(net, n, d, h, w, mode, layer, which):
    """Returns (descriptor, byte offset into the workspace), or None if the layer has no such tensor."""
    t, off = Tensor(), C.c_size_t()
    st = lib().lamp_unet_tensor_layout(net, n, d, h, w, mode, layer, which, C.byref(t), C.byref(off))
    if st == 2:
        return None
    _check(st, "lamp_unet_tensor_layout")
    return t, off.value


def lamp_unet_forward(net, weights, biases, x, probs, argmax, ws):
    p, nbytes = _ws(ws)
    _check(lib().lamp_unet_forward(net, _ptr(weights), _ptr(biases), C.byref(_td(x)), _ptr(probs), _ptr(argmax),
                                   p, nbytes, _stream()), "lamp_unet_forward")


def lamp_unet_forward_layers(net, weights, biases, x, first_layer, last_layer, probs, argmax, ws):
    p, nbytes = _ws(ws)
    _check(lib().lamp_unet_forward_layers(net, _ptr(weights), _ptr(biases), C.byref(_td(x)), first_layer, last_layer,
                                          _ptr(probs), _ptr(argmax), p, nbytes, _stream()), "lamp_unet_forward_layers")


def lamp_unet_train_step(net, weights, biases, x, labels, loss, grad_w, grad_b, probs, ws):
    p, nbytes = _ws(ws)
    _check(lib().lamp_unet_train_step(net, _ptr(weights), _ptr(biases), C.byref(_td(x)), _ptr(labels), _ptr(loss),
                                      _ptr(grad_w), _ptr(grad_b), _ptr(probs), p, nbytes, _stream()),
           "lamp_unet_train_step")


def lamp_unet_train_step_buckets(net, weights, biases, x, labels, loss, grad_w, grad_b, probs, ws, bucket_start, bucket_events):
    """bucket_start: ascending element offsets into grad_w (first 0); bucket_events: one torch.cuda.Event per bucket,
    recorded by the library when that range of grad_w is final."""
    p, nbytes = _ws(ws)
    n = len(bucket_start)
    for e in bucket_events:
        if not e.cuda_event:                 # torch creates the CUDA event lazily, on the first record
            e.record()
    starts = (C.c_int64 * n)(*[int(v) for v in bucket_start])
    events = (C.c_void_p * n)(*[int(e.cuda_event) for e in bucket_events])
    _check(lib().lamp_unet_train_step_buckets(net, _ptr(weights), _ptr(biases), C.byref(_td(x)), _ptr(labels), _ptr(loss),
                                              _ptr(grad_w), _ptr(grad_b), _ptr(probs), p, nbytes, _stream(), starts, n, events),
           "lamp_unet_train_step_buckets")


def _i3(v):
    return (C.c_int32 * 3)(*v)


def lamp_sliding_window_num_patches(d, h, w, patch, overlap):
    return lib().lamp_sliding_window_num_patches(d, h, w, _i3(patch), overlap)


def lamp_sliding_window_partial(net, weights, biases, volume, patch, overlap, sw_batch, window, first_patch, num_patches,
                                sums_planar, weight_sums, ws):
    p, nbytes = _ws(ws)
    _check(lib().lamp_sliding_window_partial(net, _ptr(weights), _ptr(biases), C.byref(_td(volume)), _i3(patch), overlap,
                                             sw_batch, window, first_patch, num_patches, _ptr(sums_planar),
                                             _ptr(weight_sums), p, nbytes, _stream()), "lamp_sliding_window_partial")


def lamp_sliding_window_finish(sums_planar, weight_sums, k, voxels, write_probs, argmax):
    _check(lib().lamp_sliding_window_finish(_ptr(sums_planar), _ptr(weight_sums), k, voxels, 1 if write_probs else 0,
                                            _ptr(argmax), _stream()), "lamp_sliding_window_finish")


def lamp_sliding_window_workspace_bytes(net, d, h, w, patch, overlap, sw_batch):
    return lib().lamp_sliding_window_workspace_bytes(net, d, h, w, _i3(patch), overlap, sw_batch)


def lamp_sliding_window_infer(net, weights, biases, volume, patch, overlap, sw_batch, window, probs_planar, argmax, ws):
    p, nbytes = _ws(ws)
    _check(lib().lamp_sliding_window_infer(net, _ptr(weights), _ptr(biases), C.byref(_td(volume)), _i3(patch), overlap,
                                           sw_batch, window, _ptr(probs_planar), _ptr(argmax), p, nbytes, _stream()),
           "lamp_sliding_window_infer")


def lamp_overlap_add(patch_probs, k, d, h, w, patch, overlap, window, probs_planar, argmax):
    _check(lib().lamp_overlap_add(_ptr(patch_probs), k, d, h, w, _i3(patch), overlap, window, _ptr(probs_planar),
                                  _ptr(argmax), _stream()), "lamp_overlap_add")


def lamp_se_squeeze(y, mu_rstd, sums):
    _check(lib().lamp_se_squeeze(C.byref(_td(y)), _ptr(mu_rstd), _ptr(sums), _stream()), "lamp_se_squeeze")


def lamp_se_excite(sums, voxels_per_sample, n, c, cr, w1, b1, w2, b2, e, hidden, mean):
    _check(lib().lamp_se_excite(_ptr(sums), voxels_per_sample, n, c, cr, _ptr(w1), _ptr(b1), _ptr(w2), _ptr(b2), _ptr(e),
                                _ptr(hidden), _ptr(mean), _stream()), "lamp_se_excite")


def lamp_se_apply_fwd(y, mu_rstd, e, residual, out):
    _check(lib().lamp_se_apply_fwd(C.byref(_td(y)), _ptr(mu_rstd), _ptr(e), C.byref(_td(residual)) if residual is not None else None,
                                   C.byref(_td(out)), _stream()), "lamp_se_apply_fwd")


def lamp_se_bwd_reduce(dout, y, mu_rstd, de_sums):
    _check(lib().lamp_se_bwd_reduce(C.byref(_td(dout)), C.byref(_td(y)), _ptr(mu_rstd), _ptr(de_sums), _stream()),
           "lamp_se_bwd_reduce")


def lamp_se_excite_bwd(de_sums, voxels_per_sample, n, c, cr, e, hidden, mean, w1, w2, ds_over_v, dw1, db1, dw2, db2):
    _check(lib().lamp_se_excite_bwd(_ptr(de_sums), voxels_per_sample, n, c, cr, _ptr(e), _ptr(hidden), _ptr(mean), _ptr(w1),
                                    _ptr(w2), _ptr(ds_over_v), _ptr(dw1), _ptr(db1), _ptr(dw2), _ptr(db2), _stream()),
           "lamp_se_excite_bwd")


def lamp_se_apply_bwd(dout, e, ds_over_v, dz):
    _check(lib().lamp_se_apply_bwd(C.byref(_td(dout)), _ptr(e), _ptr(ds_over_v), C.byref(_td(dz)), _stream()), "lamp_se_apply_bwd")


def lamp_rmsprop_step(grad, master, v, param_bf16=None, lr=1e-3, alpha=0.99, eps=1e-8):
    _check(lib().lamp_rmsprop_step(grad.numel(), _ptr(grad), _ptr(master), _ptr(v), _ptr(param_bf16), lr, alpha, eps,
                                   _stream()), "lamp_rmsprop_step")


def lamp_get_async_status():
    return lib().lamp_get_async_status(_stream())


def lamp_selftest_wait_timeout():
    _check(lib().lamp_selftest_wait_timeout(_stream()), "lamp_selftest_wait_timeout")


def lamp_version():
    return lib().lamp_version().decode()
