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


def weight_planes(buf: torch.Tensor, d) -> np.ndarray:
    """First part of a packed weight buffer: the plane words [kh][kw][CW][c_out][w_bits]."""
    cw = (d.c_in + 31) // 32
    n = d.kh * d.kw * cw * d.c_out * d.w_bits
    return as_u32(buf)[:n].reshape(d.kh, d.kw, cw, d.c_out, d.w_bits)


def weight_byte_image(buf: torch.Tensor, d) -> np.ndarray:
    """Second part of a packed weight buffer decoded back to signed codes [c_out16, CW*32, kh, kw]:
    undoes the half swap of rows with (co >> 2) & 1 and the byte order 4b + i <- channel 8i + b."""
    cw = (d.c_in + 31) // 32
    co16 = (d.c_out + 15) // 16 * 16
    raw = buf.cpu().numpy().view(np.uint8)[ebs.ebs_packed_weight_plane_bytes(d):]
    rows = raw[: d.kh * d.kw * cw * co16 * 32].reshape(d.kh, d.kw, cw, co16, 2, 16).copy()
    swap = ((np.arange(co16) >> 2) & 1).astype(bool)
    rows[:, :, :, swap] = rows[:, :, :, swap][..., ::-1, :]
    rows = rows.reshape(d.kh, d.kw, cw, co16, 32)
    j = np.arange(32)
    chan = 8 * (j % 4) + j // 4                       # byte j = 4b + i holds channel 8i + b
    out = np.zeros((d.kh, d.kw, cw, co16, 32), np.int8)
    out[..., chan] = rows.view(np.int8)
    return out.transpose(3, 2, 4, 0, 1).reshape(co16, cw * 32, d.kh, d.kw)


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


def variants_of(family):
    """Variant numbers of a kernel family, as the library names them ("popc", "mma", "umma", "umma_strip",
    "umma_resident", "mma_strip", "umma_pipe")."""
    return [v for v in range(ebs.ebs_num_conv_variants()) if ebs.ebs_conv_variant_family(v) == family]


def applies(d, h, w, variant, n=1, epi=None, want_acc=True, want_y=False, want_packed=False):
    """Asks the library whether a forced variant can run this request (its own rules: nothing is restated here).
    EBS_ERR_UNSUPPORTED means no; any other error is a bug in the test's request."""
    rc = ebs.ebs_conv_variant_applies(d, n, h, w, epi, want_acc, want_y, want_packed, variant)
    if rc == ebs.EBS_OK:
        return True
    assert rc == ebs.EBS_ERR_UNSUPPORTED, f"variant {variant}: {ebs.ebs_status_string(rc)}"
    return False


def all_variants(d, w=16, h=None, n=1, epi=None, want_y=False, want_packed=False, min_count=3):
    """Every kernel variant the library accepts for this request (-1 = its own choice comes first)."""
    h = w if h is None else h
    out = [-1] + [v for v in range(ebs.ebs_num_conv_variants())
                  if applies(d, h, w, v, n, epi, True, want_y, want_packed)]
    assert len(out) >= min_count, f"only {len(out)} variants apply: the test would cover too little"
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
