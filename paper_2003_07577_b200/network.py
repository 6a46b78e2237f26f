"""Chains the C-ABI entry points over a basic-block residual network (the CIFAR ResNets and the ImageNet ResNet-18 of
Sec. 5; the ImageNet form has a max pooling between the first convolution and the first block).

Plumbing only: this module owns device buffers and the order of the calls.  Every arithmetic step
(quantize + pack, the plane-pair convolution, scale / bias / shortcut / ReLU / requantize, average
pooling) runs inside the library's kernels.

Data flow for one batch of 8-bit images (NHWC):

    pack(8 bit) -> conv1 [-> max pool] -> x                   x: packed planes of the block input
    per block:   c1(x) -> t ; c2(t) + shortcut -> x'          t, x': packed planes
       identity shortcut:  the packed codes of x, times their step, added inside c2's epilogue
       projection shortcut: ds(x) as fp32, added inside c2's epilogue
    last block also writes fp32 -> global average pool -> pack(8 bit) -> classifier (1x1 conv) -> logits
"""
from __future__ import annotations

from dataclasses import dataclass
from typing import Dict, List, Optional

import torch

from . import binding as ebs


@dataclass
class ConvPlan:
    """One convolution with everything its call needs.  ``desc.a_scale`` must be the step of the
    tensor the layer reads (the producer's ``out_step``)."""
    name: str
    role: str                     # "first" | "conv" | "shortcut" | "fc"
    desc: "ebs.ebs_conv_desc"
    h_in: int
    w_in: int
    packed_w: torch.Tensor
    ch_bias: Optional[torch.Tensor] = None
    ch_scale: Optional[torch.Tensor] = None
    out_bits: int = 0             # bitwidth of the packed output (0: fp32 output only)
    out_step: float = 0.0         # quantization step of the packed output
    # first layer in space-to-depth form (space_to_depth_stem): block offset, and the image the packing reads
    s2d_offset: int = -1
    src_c: int = 0
    src_h: int = 0
    src_w: int = 0


def space_to_depth_weights(weight_codes: torch.Tensor) -> torch.Tensor:
    """[c_out, c, k, k] -> [c_out, 4 c, ceil(k/2), ceil(k/2)]: w2[co][(2 dy + dx) c + ch][bi][bj] = w[co][ch][2 bi + dy][2 bj + dx],
    zero where 2 bi + dy or 2 bj + dx reaches k (slices only)."""
    co, c, k, _ = weight_codes.shape
    k2 = (k + 1) // 2
    w2 = torch.zeros((co, 4 * c, k2, k2), dtype=weight_codes.dtype, device=weight_codes.device)
    for dy in (0, 1):
        for dx in (0, 1):
            sub = weight_codes[:, :, dy::2, dx::2]
            w2[:, (2 * dy + dx) * c:(2 * dy + dx + 1) * c, :sub.shape[2], :sub.shape[3]] = sub
    return w2.contiguous()


def space_to_depth_stem(plan: ConvPlan, weight_codes: torch.Tensor) -> ConvPlan:
    """The first layer of an ImageNet network (k x k, k odd, stride 2, few input channels, even image sides) as the
    equivalent stride-1 layer over the space-to-depth image that ebs_pack_acts_s2d writes: ceil(k/2)-square kernel, four
    times the channels, weights regrouped as w2[co][(2 dy + dx) c + ch][bi][bj] = w[co][ch][2 bi + dy][2 bj + dx]
    (slices of the code tensor: no arithmetic).  Returns `plan` itself when the layer does not have that shape.
    weight_codes: int8 [c_out, c_in, k, k] on the device."""
    d = plan.desc
    c, k = d.c_in, d.kh
    if not (plan.role == "first" and d.kh == d.kw and k % 2 == 1 and d.stride_h == 2 and d.stride_w == 2 and
            d.pad_h == d.pad_w and 4 * c <= 32 and plan.h_in % 2 == 0 and plan.w_in % 2 == 0):
        return plan
    off, k2 = d.pad_h & 1, (k + 1) // 2
    pb = (d.pad_h - off) // 2
    hs, ws = (plan.h_in + off) // 2 + off, (plan.w_in + off) // 2 + off
    w2 = space_to_depth_weights(weight_codes)
    d2 = ebs.conv_desc(4 * c, d.c_out, k2, k2, 1, 1, pb, pb, d.w_bits, d.a_bits, d.w_scale, d.a_scale)
    assert ebs.ebs_conv_out_shape(d2, hs, ws) == ebs.ebs_conv_out_shape(d, plan.h_in, plan.w_in)
    pw2 = torch.empty(ebs.ebs_packed_weight_bytes(d2) // 4, dtype=torch.int32, device=weight_codes.device)
    ebs.ebs_pack_weights(w2, ebs.EBS_I8_CODES, ebs.EBS_NCHW, d2, pw2)
    return ConvPlan(plan.name, plan.role, d2, hs, ws, pw2, plan.ch_bias, plan.ch_scale, plan.out_bits, plan.out_step,
                    s2d_offset=off, src_c=c, src_h=plan.h_in, src_w=plan.w_in)


class BasicBlockNet:
    """conv1, basic blocks named ``<block>c1`` / ``<block>c2`` (/ ``<block>ds``), average pool, classifier."""

    def __init__(self, plans: List[ConvPlan], device=None, pool=None):
        """pool: None, or (k, stride, pad) of the max pooling after the first convolution (ImageNet ResNets: (3, 2, 1))."""
        self.plans = plans
        self.pool = pool
        self.device = torch.device("cuda:0") if device is None else device
        self.first = plans[0]
        self.fc = plans[-1]
        assert self.first.role == "first" and self.fc.role == "fc"
        self.blocks = []
        by_name = {p.name: p for p in plans}
        for p in plans[1:-1]:
            if p.name.endswith("c1"):
                tag = p.name[:-2]
                self.blocks.append((p, by_name[tag + "c2"], by_name.get(tag + "ds")))
        self._buf: Dict[tuple, torch.Tensor] = {}

    # ------------------------------------------------------------------ buffers (allocated once per batch size)
    def _get(self, key, numel, dtype):
        t = self._buf.get(key)
        if t is None or t.numel() != numel:
            t = torch.empty(numel, dtype=dtype, device=self.device)
            self._buf[key] = t
        return t

    def _planes(self, key, n, h, w, c, bits):
        return self._get(key, ebs.ebs_packed_act_bytes(n, h, w, c, bits) // 4, torch.int32)

    def _conv(self, p: ConvPlan, src, n, *, residual=None, res_packed=None, res_bits=0, res_step=0.0, relu=True,
              want_y=False, stream=None):
        d = p.desc
        ho, wo = ebs.ebs_conv_out_shape(d, p.h_in, p.w_in)
        y = self._get((p.name, "y"), n * ho * wo * d.c_out, torch.float32) if want_y else None
        out = self._planes((p.name, "q"), n, ho, wo, d.c_out, p.out_bits) if p.out_bits else None
        epi = ebs.epilogue(p.ch_scale, p.ch_bias, residual, relu, p.out_bits, p.out_step, ebs.EBS_NHWC,
                           res_packed=res_packed, res_bits=res_bits, res_scale=res_step)
        ebs.ebs_conv2d_mixed(src, n, p.h_in, p.w_in, p.packed_w, d, epi, None, y, out, stream=stream)
        return y, out, ho, wo

    # ------------------------------------------------------------------ one batch
    def forward(self, images_u8_nhwc: torch.Tensor, stream=None) -> torch.Tensor:
        """images: uint8 [N, H, W, 3] on the device.  Returns fp32 logits [N, classes]."""
        n = images_u8_nhwc.shape[0]
        f = self.first
        px = self._planes(("input", "q"), n, f.h_in, f.w_in, f.desc.c_in, 8)
        if f.s2d_offset >= 0:                                    # stride-2 first layer in space-to-depth form
            ebs.ebs_pack_acts_s2d(images_u8_nhwc, n, f.src_c, f.src_h, f.src_w, f.s2d_offset, 8, px, stream=stream)
        else:
            ebs.ebs_pack_acts(images_u8_nhwc, ebs.EBS_U8_CODES, ebs.EBS_NHWC, n, f.desc.c_in, f.h_in, f.w_in, 8, 1.0, px,
                              stream=stream)
        _, x, ho1, wo1 = self._conv(f, px, n, stream=stream)
        x_bits, x_step = f.out_bits, f.out_step
        if self.pool is not None:                                # on the packed codes; bits and step are unchanged
            k, s, pd = self.pool
            hp, wp = (ho1 + 2 * pd - k) // s + 1, (wo1 + 2 * pd - k) // s + 1
            xp = self._planes(("maxpool", "q"), n, hp, wp, f.desc.c_out, x_bits)
            ebs.ebs_maxpool_packed(x, n, ho1, wo1, f.desc.c_out, x_bits, k, s, pd, xp, stream=stream)
            x = xp
        y_last, ho, wo = None, 0, 0
        for bi, (c1, c2, ds) in enumerate(self.blocks):
            last = bi == len(self.blocks) - 1
            _, t, _, _ = self._conv(c1, x, n, stream=stream)
            if ds is not None:
                y_ds, _, _, _ = self._conv(ds, x, n, relu=False, want_y=True, stream=stream)
                y_last, x_new, ho, wo = self._conv(c2, t, n, residual=y_ds, want_y=last, stream=stream)
            else:
                y_last, x_new, ho, wo = self._conv(c2, t, n, res_packed=x, res_bits=x_bits, res_step=x_step,
                                                   want_y=last, stream=stream)
            x, x_bits, x_step = x_new, c2.out_bits, c2.out_step
        c_last = self.blocks[-1][1].desc.c_out
        pooled = self._get(("pool", "y"), n * c_last, torch.float32)
        ebs.ebs_global_avgpool(y_last, n, ho * wo, c_last, pooled, stream=stream)
        fc = self.fc
        pq = self._planes(("pool", "q"), n, 1, 1, c_last, fc.desc.a_bits)
        ebs.ebs_pack_acts(pooled, ebs.EBS_F32, ebs.EBS_NHWC, n, c_last, 1, 1, fc.desc.a_bits, fc.desc.a_scale, pq,
                          stream=stream)
        logits, _, _, _ = self._conv(fc, pq, n, relu=False, want_y=True, stream=stream)
        return logits.view(n, fc.desc.c_out)

    @property
    def launches_per_forward(self) -> int:
        return 2 + len(self.plans) + 1 + (1 if self.pool is not None else 0)


def calibrated_plans(layers, weight_codes, images_u8_nhwc: torch.Tensor, device=None, pool=None,
                     stem_s2d: bool = True) -> List[ConvPlan]:
    """Builds the per-layer plans of a basic-block network from integer weight codes.

    ``layers``: records with name, role, c_in, c_out, k, stride, pad, h_in, w_in, w_bits, a_bits,
    w_scale, in network order.  ``weight_codes[name]``: int8 tensor [Co, Ci, k, k] on the device.
    The per-channel scale and shift (a folded BatchNorm) and each quantizer's step are set from the
    statistics of ``images_u8_nhwc`` so that codes spread over their range.  This is set-up work,
    done once with torch reductions over the library's own outputs; it is not on the timed path.
    """
    device = torch.device("cuda:0") if device is None else device
    n = images_u8_nhwc.shape[0]
    by_name = {L.name: L for L in layers}
    tags = [L.name[:-2] for L in layers if L.name.endswith("c1")]
    plans: Dict[str, ConvPlan] = {}

    def run(L, src, a_scale, nb, residual=None, res=None, relu=True):
        d = ebs.conv_desc(L.c_in, L.c_out, L.k, L.k, L.stride, L.stride, L.pad, L.pad, L.w_bits, L.a_bits,
                          L.w_scale, a_scale)
        pw = torch.empty(ebs.ebs_packed_weight_bytes(d) // 4, dtype=torch.int32, device=device)
        ebs.ebs_pack_weights(weight_codes[L.name], ebs.EBS_I8_CODES, ebs.EBS_NCHW, d, pw)
        ho, wo = ebs.ebs_conv_out_shape(d, L.h_in, L.w_in)
        acc = torch.empty((n, ho, wo, L.c_out), dtype=torch.int32, device=device)
        ebs.ebs_conv2d_mixed(src, n, L.h_in, L.w_in, pw, d, None, acc, None, None)
        S = float(L.w_scale) * float(a_scale)
        af = acc.double()
        gain = 1.0 / max(float(af.std()) * S, 1e-12)
        cs = torch.full((L.c_out,), gain, dtype=torch.float32, device=device)
        cb = torch.full((L.c_out,), -float(af.mean()) * S * gain, dtype=torch.float32, device=device)
        y = torch.empty((n, ho, wo, L.c_out), dtype=torch.float32, device=device)
        kw = dict(res_packed=res[0], res_bits=res[1], res_scale=res[2]) if res else {}
        ebs.ebs_conv2d_mixed(src, n, L.h_in, L.w_in, pw, d, ebs.epilogue(cs, cb, residual, relu, **kw), None, y, None)
        step, out = 0.0, None
        if nb:
            flat = y.flatten()
            if flat.numel() > (1 << 22):
                flat = flat[:: flat.numel() // (1 << 22)]
            step = max(float(torch.quantile(flat, 0.995)), 1e-6) / ((1 << nb) - 1)
            out = torch.empty(ebs.ebs_packed_act_bytes(n, ho, wo, L.c_out, nb) // 4, dtype=torch.int32, device=device)
            ebs.ebs_conv2d_mixed(src, n, L.h_in, L.w_in, pw, d, ebs.epilogue(cs, cb, residual, relu, nb, step, **kw),
                                 None, None, out)
        plans[L.name] = ConvPlan(L.name, L.role, d, L.h_in, L.w_in, pw, cb, cs, nb, step)
        return y, out, step, (ho, wo)

    first, fc = layers[0], layers[-1]
    px = torch.empty(ebs.ebs_packed_act_bytes(n, first.h_in, first.w_in, first.c_in, 8) // 4, dtype=torch.int32,
                     device=device)
    ebs.ebs_pack_acts(images_u8_nhwc, ebs.EBS_U8_CODES, ebs.EBS_NHWC, n, first.c_in, first.h_in, first.w_in, 8, 1.0, px)
    x_bits = by_name[tags[0] + "c1"].a_bits
    _, x, x_step, hw1 = run(first, px, 1.0 / 255.0, x_bits)
    if pool is not None:
        k, s, pd = pool
        hp, wp = (hw1[0] + 2 * pd - k) // s + 1, (hw1[1] + 2 * pd - k) // s + 1
        xp = torch.empty(ebs.ebs_packed_act_bytes(n, hp, wp, first.c_out, x_bits) // 4, dtype=torch.int32, device=device)
        ebs.ebs_maxpool_packed(x, n, hw1[0], hw1[1], first.c_out, x_bits, k, s, pd, xp)
        x = xp
    y_last, hw = None, (0, 0)
    for bi, tag in enumerate(tags):
        c1, c2, ds = by_name[tag + "c1"], by_name[tag + "c2"], by_name.get(tag + "ds")
        _, t, t_step, _ = run(c1, x, x_step, c2.a_bits)
        nb = by_name[tags[bi + 1] + "c1"].a_bits if bi + 1 < len(tags) else 0
        if ds is not None:
            y_ds, _, _, _ = run(ds, x, x_step, 0, relu=False)
            y_last, x_new, s_new, hw = run(c2, t, t_step, nb, residual=y_ds)
        else:
            y_last, x_new, s_new, hw = run(c2, t, t_step, nb, res=(x, x_bits, x_step))
        x, x_bits, x_step = x_new, nb, s_new
    c_last = by_name[tags[-1] + "c2"].c_out
    pooled = torch.empty((n, c_last), dtype=torch.float32, device=device)
    ebs.ebs_global_avgpool(y_last, n, hw[0] * hw[1], c_last, pooled)
    s_fc = max(float(pooled.max()), 1e-6) / 255.0
    pq = torch.empty(ebs.ebs_packed_act_bytes(n, 1, 1, c_last, fc.a_bits) // 4, dtype=torch.int32, device=device)
    ebs.ebs_pack_acts(pooled, ebs.EBS_F32, ebs.EBS_NHWC, n, c_last, 1, 1, fc.a_bits, s_fc, pq)
    run(fc, pq, s_fc, 0, relu=False)
    torch.cuda.synchronize(device)
    out = [plans[L.name] for L in layers]
    if stem_s2d:
        out[0] = space_to_depth_stem(out[0], weight_codes[first.name])
    return out


class FusedBasicBlockNet:
    """The same network as BasicBlockNet through ebs_resnet_cifar_forward: one launch per batch, one thread
    block per image, activations resident in shared memory.  Built from the same ConvPlan list."""

    def __init__(self, plans: List[ConvPlan], device=None, trace: bool = False):
        self.device = torch.device("cuda:0") if device is None else device
        self.plans = plans
        first, fc = plans[0], plans[-1]
        by_name = {p.name: p for p in plans}
        blocks = [(p, by_name[p.name[:-2] + "c2"], by_name.get(p.name[:-2] + "ds")) for p in plans[1:-1]
                  if p.name.endswith("c1")]
        self._keep = []
        self.trace_offsets: Dict[str, int] = {}
        trace_bytes = 0

        def record(p: ConvPlan, src, dst, *, res=0, res_buf=0, res_step=0.0, hold=0, zero_dst=0, relu=1, last=False):
            nonlocal trace_bytes
            d = p.desc
            ho, wo = ebs.ebs_conv_out_shape(d, p.h_in, p.w_in)
            off = -1
            if trace and not hold and not last:
                off = trace_bytes
                self.trace_offsets[p.name] = off
                trace_bytes += ho * wo * d.c_out
            S = ebs.ebs_combined_scale(d.w_scale, d.a_scale)          # the library's own fp32 roundings
            inv = ebs.ebs_reciprocal_step(p.out_step) if p.out_bits else 0.0
            self._keep.append((p.packed_w, p.ch_scale, p.ch_bias))
            return ebs.ebs_fused_layer(
                p.packed_w.data_ptr() + ebs.ebs_packed_weight_plane_bytes(d),
                None if p.ch_scale is None else p.ch_scale.data_ptr(), None if p.ch_bias is None else p.ch_bias.data_ptr(),
                d.c_in, d.c_out, d.kh, d.stride_h, p.h_in, p.w_in, src, -1 if last else dst, res, relu, p.out_bits, hold,
                zero_dst, off, float(S), inv, float(res_step), res_buf)

        X, T, XS = 1, 2, 0
        layers = [record(first, 0, X)]
        x_step = first.out_step
        for bi, (c1, c2, ds) in enumerate(blocks):
            last = bi == len(blocks) - 1
            if ds is not None:
                layers.append(record(c1, X, T, zero_dst=1))
                layers.append(record(ds, X, XS, hold=1, relu=0))
                layers.append(record(c2, T, X, res=2, zero_dst=1, last=last))
            else:
                layers.append(record(c1, X, T))
                layers.append(record(c2, T, X, res=1, res_buf=X, res_step=x_step, last=last))
            x_step = c2.out_step
        self.n_layers = len(layers)
        self.layers_dev = torch.empty(self.n_layers * ctypes_sizeof(ebs.ebs_fused_layer), dtype=torch.uint8, device=self.device)
        ebs.ebs_fused_plan_upload(layers, self.layers_dev)
        fd = fc.desc
        S_fc = ebs.ebs_combined_scale(fd.w_scale, fd.a_scale)
        a_inv = ebs.ebs_reciprocal_step(fd.a_scale)
        self.head = ebs.ebs_fused_head(fc.packed_w.data_ptr() + ebs.ebs_packed_weight_plane_bytes(fd),
                                       None if fc.ch_scale is None else fc.ch_scale.data_ptr(),
                                       None if fc.ch_bias is None else fc.ch_bias.data_ptr(), fd.c_in, fd.c_out,
                                       float(a_inv), float(S_fc))
        self.classes = fd.c_out
        self.img_h, self.img_w = first.h_in, first.w_in
        self.trace_bytes = trace_bytes
        self._logits = None
        self._trace = None

    def forward(self, images_u8_nhwc: torch.Tensor, stream=None) -> torch.Tensor:
        n = images_u8_nhwc.shape[0]
        if self._logits is None or self._logits.shape[0] != n:
            self._logits = torch.empty((n, self.classes), dtype=torch.float32, device=self.device)
            self._trace = (torch.zeros((n, self.trace_bytes), dtype=torch.uint8, device=self.device)
                           if self.trace_bytes else None)
        ebs.ebs_resnet_cifar_forward(images_u8_nhwc, n, self.img_h, self.img_w, self.layers_dev, self.n_layers,
                                     self.head, self._logits, self._trace, self.trace_bytes, stream=stream)
        return self._logits

    def traced_codes(self, name: str, plan: ConvPlan) -> torch.Tensor:
        """Output codes of layer `name` of the last forward pass, uint8 [N, Ho, Wo, C] (trace=True only)."""
        ho, wo = ebs.ebs_conv_out_shape(plan.desc, plan.h_in, plan.w_in)
        off = self.trace_offsets[name]
        return self._trace[:, off: off + ho * wo * plan.desc.c_out].reshape(-1, ho, wo, plan.desc.c_out)


def ctypes_sizeof(t) -> int:
    import ctypes
    return ctypes.sizeof(t)
