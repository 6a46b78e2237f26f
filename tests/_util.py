"""Helpers for the GPU parity tests: move codes to the device, call the C ABI through the binding,
bring results back in the oracle's [N, C, H, W] order.  No arithmetic of the method here."""
from __future__ import annotations

import numpy as np
import torch

from paper_2003_07577_b200 import binding as ebs


def dev():
    return torch.device("cuda:0")


def desc_for(c_in, c_out, k, stride, pad, w_bits, a_bits, w_scale=0.05, a_scale=0.05, kw=None, stride_w=None,
             pad_w=None):
    return ebs.conv_desc(c_in, c_out, k, k if kw is None else kw, stride, stride if stride_w is None else stride_w,
                         pad, pad if pad_w is None else pad_w, w_bits, a_bits, w_scale, a_scale)


def pack_acts_codes(qa: np.ndarray, a_bits: int, layout=ebs.EBS_NCHW) -> torch.Tensor:
    """uint8 codes [N,C,H,W] -> packed planes on the device (int32 storage)."""
    n, c, h, w = qa.shape
    src = qa.astype(np.uint8)
    if layout == ebs.EBS_NHWC:
        src = np.ascontiguousarray(src.transpose(0, 2, 3, 1))
    x = torch.from_numpy(src).to(dev())
    out = torch.empty(ebs.ebs_packed_act_bytes(n, h, w, c, a_bits) // 4, dtype=torch.int32, device=dev())
    ebs.ebs_pack_acts(x, ebs.EBS_U8_CODES, layout, n, c, h, w, a_bits, 1.0, out)
    return out


def pack_weight_codes(qw: np.ndarray, d, layout=ebs.EBS_NCHW) -> torch.Tensor:
    src = qw.astype(np.int8)
    if layout == ebs.EBS_NHWC:
        src = np.ascontiguousarray(src.transpose(0, 2, 3, 1))
    wt = torch.from_numpy(src).to(dev())
    out = torch.empty(ebs.ebs_packed_weight_bytes(d) // 4, dtype=torch.int32, device=dev())
    ebs.ebs_pack_weights(wt, ebs.EBS_I8_CODES, layout, d, out)
    return out


def as_u32(t: torch.Tensor) -> np.ndarray:
    return t.cpu().numpy().view(np.uint32)


def run_conv(qa, qw, d, epi=None, want_acc=True, want_y=False, next_bits=0, variant=-1, px=None, pw=None):
    """Runs ebs_conv2d_mixed on codes; returns dict with acc / y as [N,Co,Ho,Wo] and packed as u32 array."""
    n, c, h, w = qa.shape
    co = qw.shape[0]
    px = pack_acts_codes(qa, d.a_bits) if px is None else px
    pw = pack_weight_codes(qw, d) if pw is None else pw
    ho, wo = ebs.ebs_conv_out_shape(d, h, w)
    acc = torch.empty((n, ho, wo, co), dtype=torch.int32, device=dev()) if want_acc else None
    y = None
    if want_y:
        nchw = epi is not None and epi.y_layout == ebs.EBS_NCHW
        y = torch.empty((n, co, ho, wo) if nchw else (n, ho, wo, co), dtype=torch.float32, device=dev())
    pn = None
    if next_bits:
        pn = torch.full((ebs.ebs_packed_act_bytes(n, ho, wo, co, next_bits) // 4,), -1, dtype=torch.int32, device=dev())
    ebs.ebs_conv2d_mixed(px, n, h, w, pw, d, epi, acc, y, pn, variant=variant)
    torch.cuda.synchronize()
    out = {}
    if acc is not None:
        out["acc"] = acc.cpu().numpy().transpose(0, 3, 1, 2)
    if y is not None:
        yy = y.cpu().numpy()
        out["y"] = yy if (epi is not None and epi.y_layout == ebs.EBS_NCHW) else yy.transpose(0, 3, 1, 2)
    if pn is not None:
        out["packed"] = as_u32(pn).reshape(n, ho, wo, (co + 31) // 32, next_bits)
    return out


def rand_codes(rng, shape, bits, signed):
    if signed:
        return rng.integers(-(1 << (bits - 1)), (1 << (bits - 1)), size=shape, dtype=np.int32)
    return rng.integers(0, 1 << bits, size=shape, dtype=np.int32)


def spec_desc(spec):
    L = spec.layer
    return ebs.conv_desc(L.c_in, L.c_out, L.k, L.k, L.stride, L.stride, L.pad, L.pad, spec.w_bits, spec.a_bits,
                         spec.w_scale, spec.a_scale)


def conv_on_device(px, n, h, w, pw, d, epi=None, want_acc=True, want_y=False, next_bits=0):
    """ebs_conv2d_mixed on already packed device operands; returns device tensors (acc NHWC, y, packed_next)."""
    ho, wo = ebs.ebs_conv_out_shape(d, h, w)
    acc = torch.empty((n, ho, wo, d.c_out), dtype=torch.int32, device=dev()) if want_acc else None
    y = torch.empty((n, ho, wo, d.c_out), dtype=torch.float32, device=dev()) if want_y else None
    pn = None
    if next_bits:
        pn = torch.empty(ebs.ebs_packed_act_bytes(n, ho, wo, d.c_out, next_bits) // 4, dtype=torch.int32, device=dev())
    ebs.ebs_conv2d_mixed(px, n, h, w, pw, d, epi, acc, y, pn)
    return acc, y, pn


def images_nchw(t: torch.Tensor, idx):
    """Selected images of an NHWC device tensor as a numpy [len(idx), C, H, W] array."""
    return t[idx].cpu().numpy().transpose(0, 3, 1, 2)


def packed_images(pn: torch.Tensor, n, ho, wo, co, bits, idx):
    """Selected images of a packed activation tensor as uint32 [len(idx), ho, wo, CW, bits]."""
    v = pn.view(n, ho, wo, (co + 31) // 32, bits)
    return v[idx].cpu().numpy().view(np.uint32)
