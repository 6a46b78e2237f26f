"""GPU parity of the whole-network wiring: the shortcut taken from packed codes inside the epilogue,
global average pooling, and a complete ResNet-20 forward pass chained through the C ABI, each against
the CPU oracle on the same seeded inputs."""
import os

import numpy as np
import pytest
import torch

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def ebs():
    if not torch.cuda.is_available():
        pytest.skip("needs a CUDA device")
    import paper_2003_07577_b200 as pkg
    from paper_2003_07577_b200 import binding
    if not os.path.exists(binding.LIB_PATH):
        pkg.build()
    binding.lib()
    return binding


@pytest.fixture(scope="module")
def U(ebs):
    from tests import _util
    return _util


@pytest.fixture(scope="module")
def gen():
    from workloads import gen as g
    return g


def _to(a, U):
    return torch.from_numpy(np.ascontiguousarray(a)).to(U.dev())


@pytest.mark.parametrize("res_bits,co,next_bits", [(1, 16, 2), (2, 32, 3), (3, 64, 1), (4, 21, 4), (8, 70, 8), (5, 130, 2)])
def test_shortcut_from_packed_codes(ebs, U, oracle, res_bits, co, next_bits):
    """y += fl32(res_scale * code) with the codes read from packed planes, every kernel family."""
    rng = np.random.default_rng(res_bits * 1000 + co)
    wb, ab, c = 2, 3, 40
    qa = U.rand_codes(rng, (2, c, 9, 7), ab, False)
    qw = U.rand_codes(rng, (co, c, 3, 3), wb, True)
    q_res = U.rand_codes(rng, (2, co, 9, 7), res_bits, False)
    w_scale, a_scale, res_scale = 0.021, 0.04, 0.37 / ((1 << res_bits) - 1)
    d = U.desc_for(c, co, 3, 1, 1, wb, ab, w_scale, a_scale)
    acc = oracle.conv2d_codes(qa, qw, (1, 1), (1, 1))
    S = oracle.combined_scale(w_scale, a_scale)
    cb = rng.uniform(-0.2, 0.2, co).astype(np.float32)
    res = oracle.dequant_codes(q_res, res_scale)
    step = np.float32(0.9 / ((1 << next_bits) - 1))
    y_ref, q_ref = oracle.epilogue(acc, S, None, cb, res, relu=True, next_bits=next_bits,
                                   inv_next=np.float32(1.0) / step)
    p_res = U.pack_acts_codes(q_res, res_bits)
    epi = ebs.epilogue(None, _to(cb, U), None, True, next_bits, float(step), ebs.EBS_NHWC, res_packed=p_res,
                       res_bits=res_bits, res_scale=res_scale)
    for variant in U.all_variants(d, 7, 9, n=2, epi=epi, want_y=True, want_packed=True, min_count=12):
        out = U.run_conv(qa, qw, d, epi, want_acc=False, want_y=True, next_bits=next_bits, variant=variant)
        assert np.array_equal(out["y"], y_ref), f"variant {variant}"
        assert np.array_equal(oracle.unpack_acts(out["packed"], co), q_ref), f"variant {variant}"
    assert 0 < q_ref.mean() < (1 << next_bits) - 1
    # packed-only output (no fp32 tensor written) takes the same shortcut
    out = U.run_conv(qa, qw, d, epi, want_acc=False, want_y=False, next_bits=next_bits)
    assert np.array_equal(oracle.unpack_acts(out["packed"], co), q_ref)


def test_shortcut_argument_checks(ebs, U):
    d = U.desc_for(16, 16, 3, 1, 1, 2, 2)
    px = torch.zeros(ebs.ebs_packed_act_bytes(1, 4, 4, 16, 2) // 4, dtype=torch.int32, device=U.dev())
    pw = torch.zeros(ebs.ebs_packed_weight_bytes(d) // 4, dtype=torch.int32, device=U.dev())
    y = torch.empty(1 * 4 * 4 * 16, dtype=torch.float32, device=U.dev())
    for bits in (0, 9):
        epi = ebs.epilogue(res_packed=px, res_bits=bits, res_scale=0.1)
        with pytest.raises(RuntimeError):
            ebs.ebs_conv2d_mixed(px, 1, 4, 4, pw, d, epi, None, y, None)


@pytest.mark.parametrize("n,hw,c", [(3, 64, 64), (1, 49, 2048), (5, 7, 21), (128, 64, 64)])
def test_global_avgpool(ebs, U, oracle, n, hw, c):
    rng = np.random.default_rng(n + hw + c)
    y = rng.standard_normal((n, c, hw, 1)).astype(np.float32) * 3.0
    out = torch.empty((n, c), dtype=torch.float32, device=U.dev())
    ebs.ebs_global_avgpool(_to(y.transpose(0, 2, 3, 1), U), n, hw, c, out)
    assert np.array_equal(out.cpu().numpy(), oracle.global_avgpool(y))


def _oracle_network(oracle, gen, specs, imgs, sample, pool=None):
    """The ResNet-20 forward pass in oracle calls on the sampled images.  Also fixes, per layer, the
    folded-BatchNorm shift and the step of the next quantizer (a calibration: any positive values
    would serve the comparison, these keep the codes spread over their range)."""
    x = imgs[sample]
    a0 = 1.0 / 255.0
    plan, trace = {}, {}
    by_name = {s.layer.name: s for s in specs}
    order = [s.layer.name for s in specs]

    def conv(spec, src, a_scale, residual=None, relu=True, nb=0):
        L = spec.layer
        acc = oracle.conv2d_codes(src, gen.weight_codes(spec), (L.stride, L.stride), (L.pad, L.pad))
        S = oracle.combined_scale(spec.w_scale, a_scale)
        gain = 1.0 / max(float(np.std(acc)) * float(S), 1e-12)          # folded BatchNorm: unit variance, zero mean
        cs = np.full(L.c_out, gain, np.float32)
        bias = np.full(L.c_out, -float(np.mean(acc)) * float(S) * gain, np.float32)
        y0, _ = oracle.epilogue(acc, S, cs, bias, residual, relu=relu)
        step = 0.0
        q = None
        if nb:
            step = float(np.float32(max(np.percentile(y0, 99.5), 1e-6) / ((1 << nb) - 1)))
            _, q = oracle.epilogue(acc, S, cs, bias, residual, relu=relu, next_bits=nb,
                                   inv_next=np.float32(1.0) / np.float32(step))
        plan[L.name] = dict(a_scale=a_scale, bias=bias, scale=cs, out_bits=nb, out_step=step)
        trace[L.name] = q
        return y0, q, step

    blocks = [nm[:-2] for nm in order if nm.endswith("c1")]
    first = by_name["conv1"]
    nb = by_name[blocks[0] + "c1"].a_bits
    _, qx, sx = conv(first, x, a0, nb=nb)
    if pool is not None:
        qx = oracle.maxpool_codes(qx, *pool)
        trace["maxpool"] = qx
    y_last = None
    for bi, tag in enumerate(blocks):
        c1, c2, ds = by_name[tag + "c1"], by_name[tag + "c2"], by_name.get(tag + "ds")
        _, qt, st = conv(c1, qx, sx, nb=c2.a_bits)
        if ds is not None:
            res, _, _ = conv(ds, qx, sx, relu=False)
        else:
            res = oracle.dequant_codes(qx, sx)
        nb = by_name[blocks[bi + 1] + "c1"].a_bits if bi + 1 < len(blocks) else 0
        y_last, qx, sx = conv(c2, qt, st, residual=res, nb=nb)
    pooled = oracle.global_avgpool(y_last)
    fc = by_name["fc"]
    s_fc = float(np.float32(max(float(pooled.max()), 1e-6) / 255.0))
    qp = oracle.quantize_acts(pooled.reshape(len(sample), -1, 1, 1), s_fc, 8)
    logits, _, _ = conv(fc, qp, s_fc, relu=False)
    return plan, trace, logits.reshape(len(sample), -1), qp


def _gpu_network(ebs, U, gen, specs, plan, pool=None, stem_s2d=False):
    from paper_2003_07577_b200.network import BasicBlockNet, ConvPlan, space_to_depth_stem
    plans = []
    for spec in specs:
        L, pl = spec.layer, plan[spec.layer.name]
        d = ebs.conv_desc(L.c_in, L.c_out, L.k, L.k, L.stride, L.stride, L.pad, L.pad, spec.w_bits, spec.a_bits,
                          spec.w_scale, pl["a_scale"])
        plans.append(ConvPlan(L.name, L.role, d, L.h_in, L.w_in, U.pack_weight_codes(gen.weight_codes(spec), d),
                              ch_bias=_to(pl["bias"], U), ch_scale=_to(pl["scale"], U), out_bits=pl["out_bits"], out_step=pl["out_step"]))
    if stem_s2d:
        converted = space_to_depth_stem(plans[0], _to(gen.weight_codes(specs[0]).astype(np.int8), U))
        assert converted.s2d_offset >= 0, "the first layer did not qualify for the space-to-depth form"
        plans[0] = converted
    return BasicBlockNet(plans, U.dev(), pool=pool)


def test_resnet20_forward_matches_the_oracle(ebs, U, oracle, gen):
    """Whole network at batch 32: every layer's packed output and the logits of the sampled images
    equal the oracle's, bit for bit."""
    n = 32
    sample = [0, 13, 31]
    specs = gen.resnet20_network(0, n)
    imgs = gen.images_u8(0, n)
    plan, trace, logits_ref, qp_ref = _oracle_network(oracle, gen, specs, imgs, sample)
    net = _gpu_network(ebs, U, gen, specs, plan)
    x = _to(imgs.astype(np.uint8).transpose(0, 2, 3, 1), U)
    for _ in range(2):                                    # second pass reuses every buffer
        logits = net.forward(x)
        torch.cuda.synchronize()
    for spec in specs:
        L, q_ref = spec.layer, trace[spec.layer.name]
        if q_ref is None:
            continue
        bits = plan[L.name]["out_bits"]
        got = oracle.unpack_acts(U.packed_images(net._buf[(L.name, "q")], n, L.h_out, L.w_out, L.c_out, bits, sample),
                                 L.c_out)
        assert np.array_equal(got, q_ref), f"{L.name} W{spec.w_bits}A{spec.a_bits}"
        assert 0 < q_ref.mean() < (1 << bits) - 1
    got_p = oracle.unpack_acts(U.packed_images(net._buf[("pool", "q")], n, 1, 1, 64, 8, sample), 64)
    assert np.array_equal(got_p, qp_ref)
    assert np.array_equal(logits[sample].cpu().numpy(), logits_ref)
    assert np.unique(logits_ref.argmax(axis=1)).size >= 1 and np.isfinite(logits_ref).all()
    assert ebs.ebs_device_wait_timeouts() == 0


@pytest.mark.parametrize("blocks,n", [(3, 40), (5, 12)])
def test_fused_network_kernel_matches_the_oracle(ebs, U, oracle, gen, blocks, n):
    """The one-launch whole-network kernel (ResNet-20 and ResNet-32): every layer's codes (trace) and the logits
    of the sampled images equal the oracle's chain bit for bit, and the logits equal the layer-by-layer run's
    for all images."""
    from paper_2003_07577_b200.network import FusedBasicBlockNet
    sample = [0, n // 2, n - 1]
    specs = gen.resnet20_network(0, n) if blocks == 3 else gen.resnet_cifar_network(blocks, 1, n)
    imgs = gen.images_u8(0, n)
    plan, trace, logits_ref, _ = _oracle_network(oracle, gen, specs, imgs, sample)
    net = _gpu_network(ebs, U, gen, specs, plan)
    fused = FusedBasicBlockNet(net.plans, U.dev(), trace=True)
    x = _to(imgs.astype(np.uint8).transpose(0, 2, 3, 1), U)
    for _ in range(2):
        logits = fused.forward(x)
        torch.cuda.synchronize()
    assert ebs.ebs_device_wait_timeouts() == 0
    by_name = {p.name: p for p in net.plans}
    for spec in specs:
        name, q_ref = spec.layer.name, trace[spec.layer.name]
        if q_ref is None or name not in fused.trace_offsets:
            continue
        got = fused.traced_codes(name, by_name[name])[sample].cpu().numpy().transpose(0, 3, 1, 2)
        assert np.array_equal(got, q_ref), f"{name} W{spec.w_bits}A{spec.a_bits}"
    assert np.array_equal(logits[sample].cpu().numpy(), logits_ref)
    layerwise = net.forward(x)
    torch.cuda.synchronize()
    assert np.array_equal(logits.cpu().numpy(), layerwise.cpu().numpy())


def test_fused_network_plan_is_validated(ebs, U):
    from paper_2003_07577_b200 import binding
    d = U.desc_for(3, 16, 3, 1, 1, 8, 8)
    pw = torch.zeros(ebs.ebs_packed_weight_bytes(d) // 4, dtype=torch.int32, device=U.dev())
    w8 = pw.data_ptr() + ebs.ebs_packed_weight_plane_bytes(d)
    ok = binding.ebs_fused_layer(w8, None, None, 3, 16, 3, 1, 16, 16, 0, -1, 0, 1, 0, 0, 0, -1, 0.01, 0.0, 0.0, 0)
    dev = torch.empty(4096, dtype=torch.uint8, device=U.dev())
    ebs.ebs_fused_plan_upload([ok], dev)
    for field, value in (("k", 5), ("c_out", 128), ("h_in", 64), ("src", 1), ("dst", 1)):
        bad = binding.ebs_fused_layer.from_buffer_copy(ok)
        setattr(bad, field, value)
        with pytest.raises(RuntimeError):
            ebs.ebs_fused_plan_upload([bad], dev)


def _space_to_depth(x, off):
    """numpy form of the block layout: [N, C, H, W] -> [N, 4 C, Hs, Ws], channel (2 dy + dx) C + c of block (i, j) =
    pixel (2 i - off + dy, 2 j - off + dx), zero outside."""
    n, c, h, w = x.shape
    hs, ws = (h + off) // 2 + off, (w + off) // 2 + off
    out = np.zeros((n, 4 * c, hs, ws), dtype=x.dtype)
    for dy in (0, 1):
        for dx in (0, 1):
            for i in range(hs):
                hh = 2 * i - off + dy
                if not 0 <= hh < h:
                    continue
                for j in range(ws):
                    ww = 2 * j - off + dx
                    if 0 <= ww < w:
                        out[:, (2 * dy + dx) * c:(2 * dy + dx + 1) * c, i, j] = x[:, :, hh, ww]
    return out


@pytest.mark.parametrize("n,c,h,w,off,bits", [(2, 3, 16, 12, 1, 8), (1, 3, 8, 8, 0, 8), (3, 8, 10, 14, 1, 4), (2, 1, 6, 6, 0, 1),
                                              (1, 5, 12, 10, 1, 6)])
def test_space_to_depth_packing(ebs, U, oracle, n, c, h, w, off, bits):
    """ebs_pack_acts_s2d against the block layout written out in numpy, packed by the oracle."""
    rng = np.random.default_rng(n * 100 + c)
    x = rng.integers(0, 1 << bits, size=(n, c, h, w), dtype=np.int32)
    ref = _space_to_depth(x, off)
    hs, ws = ref.shape[2], ref.shape[3]
    xd = _to(x.astype(np.uint8).transpose(0, 2, 3, 1), U)
    out = torch.zeros(ebs.ebs_packed_act_bytes(n, hs, ws, 4 * c, bits) // 4, dtype=torch.int32, device=U.dev())
    ebs.ebs_pack_acts_s2d(xd, n, c, h, w, off, bits, out)
    torch.cuda.synchronize()
    got = oracle.unpack_acts(U.packed_images(out, n, hs, ws, 4 * c, bits, list(range(n))), 4 * c)
    assert np.array_equal(got, ref)


def test_space_to_depth_argument_checks(ebs, U):
    x = torch.zeros((1, 8, 8, 3), dtype=torch.uint8, device=U.dev())
    out = torch.zeros(4096, dtype=torch.int32, device=U.dev())
    for args in [(1, 9, 8, 8, 1, 8), (1, 3, 7, 8, 1, 8), (1, 3, 8, 8, 2, 8), (1, 3, 8, 8, 1, 9), (0, 3, 8, 8, 1, 8)]:
        with pytest.raises(ebs.EbsError):
            ebs.ebs_pack_acts_s2d(x, *args, out)


@pytest.mark.parametrize("bits,c,h,w,k,s,p", [(4, 64, 15, 14, 3, 2, 1), (1, 32, 8, 8, 2, 2, 0), (8, 70, 9, 11, 3, 1, 1),
                                              (3, 96, 7, 7, 3, 2, 0), (5, 33, 6, 5, 1, 1, 0), (7, 64, 12, 12, 3, 2, 1)])
def test_maxpool_on_packed_planes(ebs, U, oracle, bits, c, h, w, k, s, p):
    """Bit-plane-domain max pooling equals the oracle's maximum of codes, word for word (pad bits stay zero)."""
    rng = np.random.default_rng(bits * 100 + c + h)
    n = 3
    q = U.rand_codes(rng, (n, c, h, w), bits, False)
    ref = oracle.maxpool_codes(q, k, s, p)
    px = U.pack_acts_codes(q, bits)
    ho, wo = ref.shape[2], ref.shape[3]
    out = torch.full((ebs.ebs_packed_act_bytes(n, ho, wo, c, bits) // 4,), -1, dtype=torch.int32, device=U.dev())
    ebs.ebs_maxpool_packed(px, n, h, w, c, bits, k, s, p, out)
    torch.cuda.synchronize()
    assert np.array_equal(U.as_u32(out).reshape(n, ho, wo, (c + 31) // 32, bits), oracle.pack_acts(ref, bits))
    with pytest.raises(ebs.EbsError):
        ebs.ebs_maxpool_packed(px, n, h, w, c, bits, 3, 2, 3, out)          # padding as large as the window


def test_resnet18_imagenet_forward_matches_the_oracle(ebs, U, oracle, gen):
    """The ImageNet ResNet-18 (7x7 stride-2 first convolution at 8 bits, 3x3 stride-2 max pooling, eight basic blocks with
    projection shortcuts, average pooling, classifier) on 224x224 images at batch 4: every layer's packed output, the
    pooled codes and the logits of the sampled images equal the oracle chain bit for bit."""
    n, sample, pool = 4, [0, 3], (3, 2, 1)
    specs = gen.resnet18_network(0, n)
    assert specs[0].layer.role == "first" and specs[0].layer.k == 7 and specs[-1].layer.role == "fc"
    imgs = gen.images_u8(0, n, 224, 224)
    plan, trace, logits_ref, qp_ref = _oracle_network(oracle, gen, specs, imgs, sample, pool=pool)
    x = _to(imgs.astype(np.uint8).transpose(0, 2, 3, 1), U)
    # the first layer as given (7x7 stride 2 over the image) and in its space-to-depth form (4x4 stride 1 over 2x2 pixel
    # blocks): the same codes, so the same logits
    logits_plain = _gpu_network(ebs, U, gen, specs, plan, pool=pool).forward(x).clone()
    net = _gpu_network(ebs, U, gen, specs, plan, pool=pool, stem_s2d=True)
    logits = net.forward(x)
    torch.cuda.synchronize()
    assert torch.equal(logits, logits_plain)
    first = specs[0].layer
    got = oracle.unpack_acts(U.packed_images(net._buf[("maxpool", "q")], n, 56, 56, first.c_out, plan["conv1"]["out_bits"],
                                             sample), first.c_out)
    assert np.array_equal(got, trace["maxpool"]), "max pooling"
    for spec in specs:
        L, q_ref = spec.layer, trace[spec.layer.name]
        if q_ref is None:
            continue
        bits = plan[L.name]["out_bits"]
        got = oracle.unpack_acts(U.packed_images(net._buf[(L.name, "q")], n, L.h_out, L.w_out, L.c_out, bits, sample),
                                 L.c_out)
        assert np.array_equal(got, q_ref), f"{L.name} W{spec.w_bits}A{spec.a_bits}"
        assert 0 < q_ref.mean() < (1 << bits) - 1
    got_p = oracle.unpack_acts(U.packed_images(net._buf[("pool", "q")], n, 1, 1, 512, 8, sample), 512)
    assert np.array_equal(got_p, qp_ref)
    assert np.array_equal(logits[sample].cpu().numpy(), logits_ref)
    assert np.isfinite(logits_ref).all() and logits_ref.shape == (2, 1000)
    assert ebs.ebs_device_wait_timeouts() == 0
