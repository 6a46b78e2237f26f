"""Thin ctypes binding of libebs.so: argument marshalling only.

Every function has the name and argument order of its C entry point in ``include/ebs.h`` and
does no arithmetic of its own.  Tensors are ``torch.Tensor`` objects used purely as device (or
pinned host) memory: the binding passes ``tensor.data_ptr()`` and the current CUDA stream.
There is no CPU fallback: if the shared library is missing, loading raises.
"""
from __future__ import annotations

import ctypes
import os
from typing import Optional

import torch

_PKG = os.path.dirname(os.path.abspath(__file__))
# EBS_LIBRARY=checked selects the range-checked build of the same sources (libebs_checked.so); default: libebs.so
LIB_PATH = os.path.join(_PKG, "libebs_checked.so" if os.environ.get("EBS_LIBRARY") == "checked" else "libebs.so")

EBS_OK, EBS_ERR_INVALID_ARG, EBS_ERR_UNSUPPORTED, EBS_ERR_OVERFLOW, EBS_ERR_CUDA, EBS_ERR_TIMEOUT = 0, -1, -2, -3, -4, -5
EBS_ERR_SCRATCH_TOO_SMALL = -6
EBS_NCHW, EBS_NHWC = 0, 1
EBS_F32, EBS_I8_CODES, EBS_U8_CODES = 0, 1, 2

EXPORTS = [
    "ebs_version", "ebs_status_string", "ebs_last_cuda_error", "ebs_conv_out_shape", "ebs_packed_weight_bytes",
    "ebs_packed_act_bytes", "ebs_pack_weights", "ebs_pack_acts", "ebs_conv2d_mixed", "ebs_num_conv_variants",
    "ebs_conv2d_mixed_variant", "ebs_dequant", "ebs_host_workspace_bytes", "ebs_conv2d_mixed_host",
    "ebs_probe_pipe", "ebs_device_wait_timeouts", "ebs_global_avgpool", "ebs_packed_weight_plane_bytes", "ebs_search_weight_forward",
    "ebs_search_act_forward", "ebs_expected_flops", "ebs_fused_plan_upload", "ebs_resnet_cifar_forward", "ebs_noalloc_scratch_bytes", "ebs_conv2d_mixed_host_noalloc",
    "ebs_conv_variant_family", "ebs_conv_variant_applies", "ebs_check_device_status", "ebs_test_set_device_wait",
    "ebs_conv2d_i8", "ebs_maxpool_packed", "ebs_combined_scale", "ebs_reciprocal_step",
    "ebs_checked_build", "ebs_checked_status", "ebs_test_checked_shrink", "ebs_pack_acts_s2d",
]


class ebs_conv_desc(ctypes.Structure):
    _fields_ = [("c_in", ctypes.c_int), ("c_out", ctypes.c_int), ("kh", ctypes.c_int), ("kw", ctypes.c_int),
                ("stride_h", ctypes.c_int), ("stride_w", ctypes.c_int), ("pad_h", ctypes.c_int),
                ("pad_w", ctypes.c_int), ("w_bits", ctypes.c_int), ("a_bits", ctypes.c_int),
                ("w_scale", ctypes.c_float), ("a_scale", ctypes.c_float), ("w_levels", ctypes.c_int)]


class ebs_epilogue(ctypes.Structure):
    _fields_ = [("ch_scale_dev", ctypes.c_void_p), ("ch_bias_dev", ctypes.c_void_p),
                ("residual_dev", ctypes.c_void_p), ("relu", ctypes.c_int), ("next_a_bits", ctypes.c_int),
                ("next_a_scale", ctypes.c_float), ("y_layout", ctypes.c_int), ("res_packed_dev", ctypes.c_void_p),
                ("res_bits", ctypes.c_int), ("res_scale", ctypes.c_float)]


class EbsError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        text = lib().ebs_status_string(status).decode()
        cuda = lib().ebs_last_cuda_error().decode() if status == EBS_ERR_CUDA else ""
        super().__init__(f"{where}: {text} ({status})" + (f": {cuda}" if cuda else ""))


_lib = None


def lib() -> ctypes.CDLL:
    """Loads libebs.so (built by ``paper_2003_07577_b200.build``); raises if it is not there."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise ImportError(f"{LIB_PATH} not found: build it with `python -m paper_2003_07577_b200.build` "
                              "(there is no fallback path)")
        L = ctypes.CDLL(LIB_PATH)
        i, f, p, z = ctypes.c_int, ctypes.c_float, ctypes.c_void_p, ctypes.c_size_t
        D, E = ctypes.POINTER(ebs_conv_desc), ctypes.POINTER(ebs_epilogue)
        L.ebs_version.restype = i
        L.ebs_status_string.argtypes = [i]
        L.ebs_status_string.restype = ctypes.c_char_p
        L.ebs_last_cuda_error.restype = ctypes.c_char_p
        L.ebs_conv_out_shape.argtypes = [D, i, i, ctypes.POINTER(i), ctypes.POINTER(i)]
        L.ebs_packed_weight_bytes.argtypes = [D]
        L.ebs_packed_weight_bytes.restype = z
        L.ebs_packed_weight_plane_bytes.argtypes = [D]
        L.ebs_packed_weight_plane_bytes.restype = z
        L.ebs_packed_act_bytes.argtypes = [i, i, i, i, i]
        L.ebs_packed_act_bytes.restype = z
        L.ebs_pack_weights.argtypes = [p, i, i, D, p, p]
        L.ebs_pack_acts.argtypes = [p, i, i, i, i, i, i, i, f, p, p]
        L.ebs_conv2d_mixed.argtypes = [p, i, i, i, p, D, E, p, p, p, p]
        L.ebs_num_conv_variants.restype = i
        L.ebs_conv2d_mixed_variant.argtypes = [p, i, i, i, p, D, E, p, p, p, p, i]
        L.ebs_dequant.argtypes = [p, z, i, f, p, p, i, p, p]
        L.ebs_host_workspace_bytes.argtypes = [D, i, i, i, i, i]
        L.ebs_host_workspace_bytes.restype = z
        L.ebs_conv2d_mixed_host.argtypes = [p, i, i, i, i, i, p, D, E, p, z, p, p, p, p]
        L.ebs_probe_pipe.argtypes = [i, i, ctypes.POINTER(ctypes.c_double)]
        L.ebs_global_avgpool.argtypes = [p, i, i, i, p, p]
        ip, fp = ctypes.POINTER(ctypes.c_int), ctypes.POINTER(ctypes.c_float)
        L.ebs_search_weight_forward.argtypes = [p, z, ip, fp, i, p, p, p]
        L.ebs_search_act_forward.argtypes = [p, z, ctypes.c_float, ip, fp, i, p, p]
        L.ebs_expected_flops.argtypes = [ctypes.c_double, ip, fp, i, ip, fp, i]
        L.ebs_expected_flops.restype = ctypes.c_double
        L.ebs_fused_plan_upload.argtypes = [ctypes.c_void_p, i, p, p]
        L.ebs_resnet_cifar_forward.argtypes = [p, i, i, i, p, i, ctypes.c_void_p, p, p, ctypes.c_longlong, p]
        L.ebs_noalloc_scratch_bytes.restype = z
        L.ebs_device_wait_timeouts.restype = ctypes.c_longlong
        L.ebs_conv2d_mixed_host_noalloc.argtypes = [p, i, i, i, i, i, p, D, E, p, p, p, p]
        L.ebs_conv2d_i8.argtypes = [p, i, i, i, p, D, E, p, p, p, p]
        L.ebs_maxpool_packed.argtypes = [p, i, i, i, i, i, i, i, i, p, p]
        L.ebs_combined_scale.argtypes = [f, f]
        L.ebs_combined_scale.restype = f
        L.ebs_reciprocal_step.argtypes = [f]
        L.ebs_reciprocal_step.restype = f
        L.ebs_checked_status.argtypes = [ctypes.POINTER(i), ctypes.POINTER(ctypes.c_longlong),
                                         ctypes.POINTER(ctypes.c_longlong), i]
        L.ebs_test_checked_shrink.argtypes = [ctypes.c_longlong]
        L.ebs_pack_acts_s2d.argtypes = [p, i, i, i, i, i, i, p, p]
        L.ebs_conv_variant_family.argtypes = [i]
        L.ebs_conv_variant_family.restype = ctypes.c_char_p
        L.ebs_conv_variant_applies.argtypes = [D, i, i, i, E, i, i, i, i]
        L.ebs_check_device_status.restype = i
        L.ebs_test_set_device_wait.argtypes = [ctypes.c_uint, i]
        _lib = L
    return _lib


def _ptr(t: Optional[torch.Tensor]):
    return None if t is None else ctypes.c_void_p(t.data_ptr())


def _stream(stream=None):
    if stream is None:
        stream = torch.cuda.current_stream()
    return ctypes.c_void_p(stream.cuda_stream)


def _check(rc: int, where: str):
    if rc != EBS_OK:
        raise EbsError(rc, where)


def conv_desc(c_in, c_out, kh, kw, stride_h, stride_w, pad_h, pad_w, w_bits, a_bits, w_scale, a_scale,
              w_levels=0) -> ebs_conv_desc:
    return ebs_conv_desc(c_in, c_out, kh, kw, stride_h, stride_w, pad_h, pad_w, w_bits, a_bits, w_scale, a_scale,
                         int(w_levels))


def epilogue(ch_scale=None, ch_bias=None, residual=None, relu=False, next_a_bits=0, next_a_scale=1.0,
             y_layout=EBS_NHWC, res_packed=None, res_bits=0, res_scale=0.0) -> ebs_epilogue:
    e = ebs_epilogue(None if ch_scale is None else ch_scale.data_ptr(),
                     None if ch_bias is None else ch_bias.data_ptr(),
                     None if residual is None else residual.data_ptr(),
                     int(bool(relu)), int(next_a_bits), float(next_a_scale), int(y_layout),
                     None if res_packed is None else res_packed.data_ptr(), int(res_bits), float(res_scale))
    e._keepalive = (ch_scale, ch_bias, residual, res_packed)
    return e


def ebs_version() -> int:
    return lib().ebs_version()


def ebs_status_string(status: int) -> str:
    return lib().ebs_status_string(status).decode()


def ebs_conv_out_shape(desc: ebs_conv_desc, h: int, w: int):
    ho, wo = ctypes.c_int(0), ctypes.c_int(0)
    _check(lib().ebs_conv_out_shape(ctypes.byref(desc), h, w, ctypes.byref(ho), ctypes.byref(wo)), "ebs_conv_out_shape")
    return ho.value, wo.value


def ebs_packed_weight_bytes(desc: ebs_conv_desc) -> int:
    return lib().ebs_packed_weight_bytes(ctypes.byref(desc))


def ebs_packed_weight_plane_bytes(desc: ebs_conv_desc) -> int:
    return lib().ebs_packed_weight_plane_bytes(ctypes.byref(desc))


def ebs_packed_act_bytes(n: int, h: int, w: int, c: int, a_bits: int) -> int:
    return lib().ebs_packed_act_bytes(n, h, w, c, a_bits)


def ebs_pack_weights(w_dev: torch.Tensor, dtype: int, layout: int, desc: ebs_conv_desc, packed_w_dev: torch.Tensor,
                     stream=None) -> None:
    _check(lib().ebs_pack_weights(_ptr(w_dev), dtype, layout, ctypes.byref(desc), _ptr(packed_w_dev), _stream(stream)),
           "ebs_pack_weights")


def ebs_pack_acts(x_dev: torch.Tensor, dtype: int, layout: int, n: int, c: int, h: int, w: int, a_bits: int,
                  a_scale: float, packed_x_dev: torch.Tensor, stream=None) -> None:
    _check(lib().ebs_pack_acts(_ptr(x_dev), dtype, layout, n, c, h, w, a_bits, a_scale, _ptr(packed_x_dev),
                               _stream(stream)), "ebs_pack_acts")


def ebs_conv2d_mixed(packed_x_dev, n, h, w, packed_w_dev, desc, epi=None, acc_out_dev=None, y_out_dev=None,
                     packed_next_dev=None, stream=None, variant: int = -1) -> None:
    e = None if epi is None else ctypes.byref(epi)
    if variant == -1:
        rc = lib().ebs_conv2d_mixed(_ptr(packed_x_dev), n, h, w, _ptr(packed_w_dev), ctypes.byref(desc), e,
                                    _ptr(acc_out_dev), _ptr(y_out_dev), _ptr(packed_next_dev), _stream(stream))
    else:
        rc = lib().ebs_conv2d_mixed_variant(_ptr(packed_x_dev), n, h, w, _ptr(packed_w_dev), ctypes.byref(desc), e,
                                            _ptr(acc_out_dev), _ptr(y_out_dev), _ptr(packed_next_dev),
                                            _stream(stream), variant)
    _check(rc, "ebs_conv2d_mixed")


def ebs_num_conv_variants() -> int:
    return lib().ebs_num_conv_variants()


def ebs_dequant(acc_dev, n_pixels: int, c_out: int, scale: float, ch_scale_dev=None, ch_bias_dev=None,
                relu=False, y_dev=None, stream=None) -> None:
    _check(lib().ebs_dequant(_ptr(acc_dev), n_pixels, c_out, scale, _ptr(ch_scale_dev), _ptr(ch_bias_dev),
                             int(bool(relu)), _ptr(y_dev), _stream(stream)), "ebs_dequant")


def ebs_host_workspace_bytes(desc, n, h, w, dtype, next_a_bits=0) -> int:
    return lib().ebs_host_workspace_bytes(ctypes.byref(desc), n, h, w, dtype, next_a_bits)


def ebs_conv2d_mixed_host(x_host, dtype, layout, n, h, w, packed_w_dev, desc, epi, workspace_dev,
                          acc_out_host=None, y_out_host=None, packed_next_host=None, stream=None) -> None:
    e = None if epi is None else ctypes.byref(epi)
    rc = lib().ebs_conv2d_mixed_host(_ptr(x_host), dtype, layout, n, h, w, _ptr(packed_w_dev), ctypes.byref(desc), e,
                                     _ptr(workspace_dev), workspace_dev.numel() * workspace_dev.element_size(),
                                     _ptr(acc_out_host), _ptr(y_out_host), _ptr(packed_next_host), _stream(stream))
    _check(rc, "ebs_conv2d_mixed_host")


def ebs_probe_pipe(kind: int, iters: int = 2000) -> float:
    out = ctypes.c_double(0.0)
    _check(lib().ebs_probe_pipe(kind, iters, ctypes.byref(out)), "ebs_probe_pipe")
    return out.value


def ebs_global_avgpool(y_dev, n: int, hw: int, c: int, out_dev, stream=None) -> None:
    _check(lib().ebs_global_avgpool(_ptr(y_dev), n, hw, c, _ptr(out_dev), _stream(stream)), "ebs_global_avgpool")


class ebs_fused_layer(ctypes.Structure):
    _fields_ = [("w8", ctypes.c_void_p), ("ch_scale", ctypes.c_void_p), ("ch_bias", ctypes.c_void_p),
                ("c_in", ctypes.c_int), ("c_out", ctypes.c_int), ("k", ctypes.c_int), ("stride", ctypes.c_int),
                ("h_in", ctypes.c_int), ("w_in", ctypes.c_int), ("src", ctypes.c_int), ("dst", ctypes.c_int),
                ("res", ctypes.c_int), ("relu", ctypes.c_int), ("out_bits", ctypes.c_int), ("hold", ctypes.c_int),
                ("zero_dst", ctypes.c_int), ("trace_off", ctypes.c_int), ("S", ctypes.c_float),
                ("out_inv_step", ctypes.c_float), ("res_step", ctypes.c_float), ("res_buf", ctypes.c_int)]


class ebs_fused_head(ctypes.Structure):
    _fields_ = [("w8", ctypes.c_void_p), ("ch_scale", ctypes.c_void_p), ("ch_bias", ctypes.c_void_p),
                ("c_in", ctypes.c_int), ("c_out", ctypes.c_int), ("a_inv_step", ctypes.c_float), ("S", ctypes.c_float)]


def ebs_fused_plan_upload(layers, layers_dev: torch.Tensor, stream=None) -> None:
    """layers: list of ebs_fused_layer; layers_dev: uint8 device tensor of len(layers) * sizeof(ebs_fused_layer) bytes."""
    arr = (ebs_fused_layer * len(layers))(*layers)
    _check(lib().ebs_fused_plan_upload(arr, len(layers), _ptr(layers_dev), _stream(stream)), "ebs_fused_plan_upload")
    torch.cuda.current_stream().synchronize()          # the host array may be released after the copy


def ebs_resnet_cifar_forward(images_dev, n, img_h, img_w, layers_dev, n_layers, head: ebs_fused_head, logits_dev,
                             trace_dev=None, trace_stride: int = 0, stream=None) -> None:
    _check(lib().ebs_resnet_cifar_forward(_ptr(images_dev), n, img_h, img_w, _ptr(layers_dev), n_layers,
                                          ctypes.byref(head), _ptr(logits_dev), _ptr(trace_dev), trace_stride,
                                          _stream(stream)), "ebs_resnet_cifar_forward")


def _cand(bits, coeff):
    n = len(bits)
    return (ctypes.c_int * n)(*[int(b) for b in bits]), (ctypes.c_float * n)(*[float(c) for c in coeff]), n


def ebs_search_weight_forward(w_dev, bits, coeff, w_hat_dev, scratch_dev, stream=None) -> None:
    b, c, n = _cand(bits, coeff)
    _check(lib().ebs_search_weight_forward(_ptr(w_dev), w_dev.numel(), b, c, n, _ptr(w_hat_dev), _ptr(scratch_dev),
                                           _stream(stream)), "ebs_search_weight_forward")


def ebs_search_act_forward(x_dev, alpha: float, bits, coeff, x_hat_dev, stream=None) -> None:
    b, c, n = _cand(bits, coeff)
    _check(lib().ebs_search_act_forward(_ptr(x_dev), x_dev.numel(), alpha, b, c, n, _ptr(x_hat_dev), _stream(stream)),
           "ebs_search_act_forward")


def ebs_expected_flops(macs: float, bits_w, coeff_w, bits_x, coeff_x) -> float:
    bw, cw, nw = _cand(bits_w, coeff_w)
    bx, cx, nx = _cand(bits_x, coeff_x)
    return lib().ebs_expected_flops(float(macs), bw, cw, nw, bx, cx, nx)


def ebs_device_wait_timeouts() -> int:
    return int(lib().ebs_device_wait_timeouts())


def ebs_noalloc_scratch_bytes() -> int:
    return lib().ebs_noalloc_scratch_bytes()


def ebs_conv2d_mixed_host_noalloc(x_host, dtype, layout, n, h, w, packed_w_dev, desc, epi, acc_out_host=None,
                                  y_out_host=None, packed_next_host=None, stream=None) -> None:
    """Same as ebs_conv2d_mixed_host, for callers that may not allocate device memory: no workspace argument."""
    e = None if epi is None else ctypes.byref(epi)
    rc = lib().ebs_conv2d_mixed_host_noalloc(_ptr(x_host), dtype, layout, n, h, w, _ptr(packed_w_dev),
                                             ctypes.byref(desc), e, _ptr(acc_out_host), _ptr(y_out_host),
                                             _ptr(packed_next_host), _stream(stream))
    _check(rc, "ebs_conv2d_mixed_host_noalloc")


def ebs_conv_variant_family(variant: int) -> str:
    return lib().ebs_conv_variant_family(int(variant)).decode()


def ebs_conv_variant_applies(desc, n, h, w, epi=None, want_acc=True, want_y=False, want_packed_next=False,
                             variant: int = -1) -> int:
    """Status the forced-variant call would return for this request (EBS_OK / EBS_ERR_UNSUPPORTED / ...); launches nothing."""
    e = None if epi is None else ctypes.byref(epi)
    return lib().ebs_conv_variant_applies(ctypes.byref(desc), n, h, w, e, int(bool(want_acc)), int(bool(want_y)),
                                          int(bool(want_packed_next)), int(variant))


def ebs_check_device_status() -> int:
    return int(lib().ebs_check_device_status())


def ebs_checked_build() -> bool:
    return bool(lib().ebs_checked_build())


def ebs_checked_status(clear: bool = True):
    """(recorded, site, index, limit) of the range-checked build; raises in the normal build."""
    site, index, limit = ctypes.c_int(0), ctypes.c_longlong(0), ctypes.c_longlong(0)
    rc = lib().ebs_checked_status(ctypes.byref(site), ctypes.byref(index), ctypes.byref(limit), int(bool(clear)))
    if rc < 0:
        _check(rc, "ebs_checked_status")
    return bool(rc), site.value, index.value, limit.value


def ebs_pack_acts_s2d(x_dev, n, c, h, w, offset, a_bits, packed_x_dev, stream=None) -> None:
    _check(lib().ebs_pack_acts_s2d(_ptr(x_dev), int(n), int(c), int(h), int(w), int(offset), int(a_bits),
                                   _ptr(packed_x_dev), _stream(stream)), "ebs_pack_acts_s2d")


def ebs_test_checked_shrink(elements: int) -> None:
    _check(lib().ebs_test_checked_shrink(int(elements)), "ebs_test_checked_shrink")


def ebs_test_set_device_wait(limit: int, skip_mma: bool) -> None:
    _check(lib().ebs_test_set_device_wait(int(limit), int(bool(skip_mma))), "ebs_test_set_device_wait")


def ebs_conv2d_i8(x_codes_dev, n, h, w, packed_w_dev, desc, epi=None, acc_out_dev=None, y_out_dev=None,
                  packed_next_dev=None, stream=None) -> None:
    """The context path: activations as unpacked u8 NHWC codes (not the paper's method; see include/ebs.h)."""
    e = None if epi is None else ctypes.byref(epi)
    _check(lib().ebs_conv2d_i8(_ptr(x_codes_dev), n, h, w, _ptr(packed_w_dev), ctypes.byref(desc), e, _ptr(acc_out_dev),
                               _ptr(y_out_dev), _ptr(packed_next_dev), _stream(stream)), "ebs_conv2d_i8")


def ebs_maxpool_packed(packed_x_dev, n, h, w, c, a_bits, k, stride, pad, packed_out_dev, stream=None) -> None:
    _check(lib().ebs_maxpool_packed(_ptr(packed_x_dev), n, h, w, c, a_bits, k, stride, pad, _ptr(packed_out_dev),
                                    _stream(stream)), "ebs_maxpool_packed")


def ebs_combined_scale(w_scale: float, a_scale: float) -> float:
    return float(lib().ebs_combined_scale(w_scale, a_scale))


def ebs_reciprocal_step(step: float) -> float:
    return float(lib().ebs_reciprocal_step(step))
