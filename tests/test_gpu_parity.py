"""GPU parity: the CUDA path, called through the C ABI, against the CPU oracle on the same seeded inputs.

Bar: int32 accumulators, packed words and requantized codes bit-exact; fp32 outputs within 1e-5
relative (they are in fact computed with the same individually rounded operations).
"""
import itertools

import os

import numpy as np
import pytest
import torch

pytestmark = pytest.mark.gpu

RTOL = 1e-5


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


# ------------------------------------------------------------------ packing (rows a1, a2)

@pytest.mark.parametrize("c,ab,shape", [(3, 8, (2, 5, 7)), (16, 2, (3, 8, 8)), (32, 1, (1, 9, 4)), (48, 3, (2, 6, 5)),
                                        (64, 4, (2, 7, 7)), (70, 5, (1, 33, 3)), (130, 7, (1, 4, 9))])
@pytest.mark.parametrize("layout", [0, 1])
def test_pack_acts_codes(ebs, U, oracle, c, ab, shape, layout):
    rng = np.random.default_rng(c * 10 + ab)
    n, h, w = shape
    qa = U.rand_codes(rng, (n, c, h, w), ab, False)
    got = U.as_u32(U.pack_acts_codes(qa, ab, layout)).reshape(n, h, w, (c + 31) // 32, ab)
    assert np.array_equal(got, oracle.pack_acts(qa, ab))


@pytest.mark.parametrize("c,ab", [(16, 2), (40, 3), (64, 8), (3, 4)])
@pytest.mark.parametrize("layout", [0, 1])
def test_pack_acts_fp32_quantizes_like_the_oracle(ebs, U, oracle, c, ab, layout):
    rng = np.random.default_rng(c + ab)
    n, h, w = 2, 9, 7
    scale = np.float32(0.0371)
    x = rng.uniform(-0.5, 1.2 * scale * (1 << ab), size=(n, c, h, w)).astype(np.float32)
    # plant exact ties and out-of-range values
    x[0, 0, 0, :4] = np.array([0.5, 1.5, 2.5, -0.5], np.float32) * np.float32(0.25)
    qa = oracle.quantize_acts(x, scale, ab)
    src = np.ascontiguousarray(x.transpose(0, 2, 3, 1)) if layout == ebs.EBS_NHWC else x
    out = torch.empty(ebs.ebs_packed_act_bytes(n, h, w, c, ab) // 4, dtype=torch.int32, device=U.dev())
    ebs.ebs_pack_acts(torch.from_numpy(src).to(U.dev()), ebs.EBS_F32, layout, n, c, h, w, ab, float(scale), out)
    got = U.as_u32(out).reshape(n, h, w, (c + 31) // 32, ab)
    assert np.array_equal(oracle.unpack_acts(got, c), qa)
    assert np.array_equal(got, oracle.pack_acts(qa, ab))


@pytest.mark.parametrize("co,c,k,wb", [(5, 3, 7, 8), (16, 16, 3, 1), (33, 70, 3, 4), (64, 64, 1, 2), (8, 130, 3, 6)])
@pytest.mark.parametrize("layout", [0, 1])
def test_pack_weights(ebs, U, oracle, co, c, k, wb, layout):
    rng = np.random.default_rng(co + c + wb)
    qw = U.rand_codes(rng, (co, c, k, k), wb, True)
    d = U.desc_for(c, co, k, 1, k // 2, wb, 2)
    buf = U.pack_weight_codes(qw, d, layout)
    got = U.weight_planes(buf, d)
    assert np.array_equal(got, oracle.pack_weights(qw, wb))
    image = U.weight_byte_image(buf, d)                    # the byte copy of the same codes, zero padded
    assert np.array_equal(image[:co, :c], qw) and not image[co:].any() and not image[:, c:].any()
    # fp32 weights go through the quantizer first
    scale = np.float32(0.043)
    wf = ((qw + rng.uniform(-0.4, 0.4, qw.shape)) * scale).astype(np.float32)
    qref = oracle.quantize_weights(wf, scale, wb)
    d2 = U.desc_for(c, co, k, 1, k // 2, wb, 2, w_scale=float(scale))
    src = np.ascontiguousarray(wf.transpose(0, 2, 3, 1)) if layout == ebs.EBS_NHWC else wf
    out = torch.empty(ebs.ebs_packed_weight_bytes(d2) // 4, dtype=torch.int32, device=U.dev())
    ebs.ebs_pack_weights(torch.from_numpy(src).to(U.dev()), ebs.EBS_F32, layout, d2, out)
    assert np.array_equal(U.weight_planes(out, d2), oracle.pack_weights(qref, wb))
    assert np.array_equal(U.weight_byte_image(out, d2)[:co, :c], qref)


# ------------------------------------------------------------------ contraction + recombination (rows a3, a4)

@pytest.mark.parametrize("wb,ab", list(itertools.product(range(1, 9), range(1, 9))))
def test_conv_all_bitwidth_pairs(ebs, U, oracle, wb, ab):
    """Every (Wb, Ab): 3x3, ragged channel counts, several tiles and a ragged tail in both tile axes."""
    rng = np.random.default_rng(wb * 8 + ab)
    qa = U.rand_codes(rng, (3, 40, 13, 11), ab, False)
    qw = U.rand_codes(rng, (21, 40, 3, 3), wb, True)
    d = U.desc_for(40, 21, 3, 1, 1, wb, ab)
    ref = oracle.conv2d_codes(qa, qw, (1, 1), (1, 1))
    px, pw = U.pack_acts_codes(qa, ab), U.pack_weight_codes(qw, d)
    variants = U.all_variants(d, 11, 13, n=3, min_count=30)    # every family has instantiations per bit count
    for fam in ("popc", "mma", "umma", "umma_strip", "umma_resident", "umma_pipe"):
        assert any(ebs.ebs_conv_variant_family(v) == fam for v in variants if v >= 0), fam
    for variant in variants:
        got = U.run_conv(qa, qw, d, variant=variant, px=px, pw=pw)["acc"]
        assert np.array_equal(got, ref), f"variant {variant}"


@pytest.mark.parametrize("ab", range(1, 9))
@pytest.mark.parametrize("c,co,k", [(40, 22, 3), (16, 16, 3), (12, 10, 3), (16, 14, 2), (8, 12, 3), (64, 64, 1), (100, 34, 3)])
def test_warp_level_strip_kernel_all_activation_bitwidths(ebs, U, oracle, ab, c, co, k):
    """The warp-level strip variants (channel tile 16 / 32 / 64): every activation bitwidth, ragged channel tiles,
    one, two and four taps per MMA step (c_in 40 / 9-16 in the 16-byte-per-pixel form, odd and even tap counts / 8),
    with and without per-channel terms and packed output."""
    rng = np.random.default_rng(100 * ab + c + co)
    wb = 1 + (ab + c) % 8
    pad = k // 2
    qa = U.rand_codes(rng, (3, c, 13, 11), ab, False)
    qw = U.rand_codes(rng, (co, c, k, k), wb, True)
    d = U.desc_for(c, co, k, 1, pad, wb, ab, 0.03, 0.05)
    ref = oracle.conv2d_codes(qa, qw, (1, 1), (pad, pad))
    S = oracle.combined_scale(0.03, 0.05)
    cs = rng.uniform(0.5, 2.0, co).astype(np.float32)
    cb = rng.uniform(-0.3, 0.3, co).astype(np.float32)
    to = lambda a: torch.from_numpy(np.ascontiguousarray(a)).to(U.dev())
    px, pw = U.pack_acts_codes(qa, ab), U.pack_weight_codes(qw, d)
    for epi, (ecs, ecb) in ((ebs.epilogue(relu=True, next_a_bits=3, next_a_scale=0.6), (None, None)),
                            (ebs.epilogue(to(cs), to(cb), None, True, 3, 0.6), (cs, cb))):
        y_ref, q_ref = oracle.epilogue(ref, S, ecs, ecb, None, relu=True, next_bits=3,
                                       inv_next=np.float32(1.0) / np.float32(0.6))
        ran = 0
        for variant in U.variants_of("mma_strip"):
            if not U.applies(d, 13, 11, variant, n=3, epi=epi, want_y=True, want_packed=True):
                continue                                      # e.g. 16-channel tiles cannot write packed words of wider layers
            ran += 1
            out = U.run_conv(qa, qw, d, epi, want_acc=True, want_y=True, next_bits=3, variant=variant, px=px, pw=pw)
            assert np.array_equal(out["acc"], ref), f"variant {variant}"
            assert np.array_equal(out["y"], y_ref), f"variant {variant}"
            assert np.array_equal(oracle.unpack_acts(out["packed"], co), q_ref), f"variant {variant}"
        assert ran >= 1


GEOMS = [
    # c_in, c_out, k, stride, pad, h, w
    (3, 16, 3, 1, 1, 32, 32), (3, 8, 7, 2, 3, 30, 29), (16, 16, 3, 1, 1, 17, 9), (16, 32, 1, 2, 0, 16, 16),
    (32, 64, 3, 2, 1, 15, 15), (48, 10, 5, 1, 2, 9, 12), (64, 64, 3, 1, 0, 8, 8), (96, 33, 3, 2, 0, 11, 7),
    (128, 70, 1, 1, 0, 7, 7), (200, 17, 3, 1, 1, 6, 5), (64, 130, 3, 1, 1, 5, 5), (33, 5, 2, 1, 1, 6, 6),
]


@pytest.mark.parametrize("geom", GEOMS)
def test_conv_geometries_all_variants(ebs, U, oracle, geom):
    c, co, k, s, pad, h, w = geom
    rng = np.random.default_rng(sum(geom))
    wb, ab = 3, 2
    qa = U.rand_codes(rng, (2, c, h, w), ab, False)
    qw = U.rand_codes(rng, (co, c, k, k), wb, True)
    d = U.desc_for(c, co, k, s, pad, wb, ab)
    ref = oracle.conv2d_codes(qa, qw, (s, s), (pad, pad))
    px, pw = U.pack_acts_codes(qa, ab), U.pack_weight_codes(qw, d)
    for variant in U.all_variants(d, w, h, n=2, min_count=10):
        got = U.run_conv(qa, qw, d, variant=variant, px=px, pw=pw)["acc"]
        assert got.shape == ref.shape and np.array_equal(got, ref), f"variant {variant}"


def test_strip_kernel_refuses_strided_layers(ebs, U):
    d = U.desc_for(32, 32, 3, 2, 1, 2, 2)
    qa, qw = np.zeros((1, 32, 8, 8), np.int32), np.zeros((32, 32, 3, 3), np.int32)
    for fam in ("umma_strip", "umma_resident", "mma_strip"):
        for variant in U.variants_of(fam):
            with pytest.raises(RuntimeError):
                U.run_conv(qa, qw, d, variant=variant)


@pytest.mark.parametrize("c,co,k,s,pad,h,n,wb,ab", [(32, 64, 3, 1, 1, 30, 48, 2, 3), (64, 48, 1, 2, 0, 40, 64, 4, 2),
                                                    (96, 16, 3, 1, 0, 24, 60, 3, 8)])
def test_persistent_kernel_walks_several_tiles_per_cta(ebs, U, oracle, c, co, k, s, pad, h, n, wb, ab):
    """More pixel tiles than thread blocks: both accumulators, both stages and the tile loop wrap around."""
    rng = np.random.default_rng(c + co + k + n)
    qa = U.rand_codes(rng, (n, c, h, h), ab, False)
    qw = U.rand_codes(rng, (co, c, k, k), wb, True)
    d = U.desc_for(c, co, k, s, pad, wb, ab, 0.03, 0.07)
    ref = oracle.conv2d_codes(qa, qw, (s, s), (pad, pad))
    y_ref, q_ref = oracle.epilogue(ref, oracle.combined_scale(0.03, 0.07), relu=True, next_bits=4,
                                   inv_next=np.float32(1.0) / np.float32(0.9))
    px, pw = U.pack_acts_codes(qa, ab), U.pack_weight_codes(qw, d)
    epi = ebs.epilogue(relu=True, next_a_bits=4, next_a_scale=0.9)
    ran = 0
    for variant in U.variants_of("umma_resident") + U.variants_of("umma_pipe"):
        if not U.applies(d, h, h, variant, n=n, epi=epi, want_y=True, want_packed=True):
            continue                                          # e.g. 16-channel tiles cannot write packed words of wider layers
        out = U.run_conv(qa, qw, d, epi, want_acc=True, want_y=True, next_bits=4, variant=variant, px=px, pw=pw)
        assert np.array_equal(out["acc"], ref), f"variant {variant}"
        assert np.array_equal(out["y"], y_ref) and np.array_equal(oracle.unpack_acts(out["packed"], co), q_ref)
        ran += 1
    assert ran >= 4 and ebs.ebs_device_wait_timeouts() == 0


def test_no_device_wait_timed_out(ebs):
    """The bounded waits of the tcgen05 kernels never gave up in the tests above."""
    assert ebs.ebs_device_wait_timeouts() == 0


def test_conv_asymmetric_kernel_stride_pad(ebs, U, oracle):
    rng = np.random.default_rng(77)
    qa = U.rand_codes(rng, (2, 20, 11, 14), 4, False)
    qw = rng.integers(-4, 4, size=(9, 20, 3, 5), dtype=np.int32)
    d = ebs.conv_desc(20, 9, 3, 5, 2, 1, 0, 2, 3, 4, 0.05, 0.05)
    ref = oracle.conv2d_codes(qa, qw, (2, 1), (0, 2))
    assert np.array_equal(U.run_conv(qa, qw, d)["acc"], ref)


def test_conv_closed_forms(ebs, U):
    """Saturated inputs: acc = -(2^Ab-1) * C * taps inside the image; and the extreme magnitudes fit."""
    c, h, ab, wb = 96, 6, 8, 8
    qa = np.full((1, c, h, h), 255, dtype=np.int32)
    qw = np.full((4, c, 3, 3), -128, dtype=np.int32)
    d = U.desc_for(c, 4, 3, 1, 1, wb, ab)
    acc = U.run_conv(qa, qw, d)["acc"]
    unit = -128 * 255 * c
    assert acc[0, 0, 0, 0] == 4 * unit and acc[0, 3, 0, 2] == 6 * unit and acc[0, 1, 2, 3] == 9 * unit
    qw[:] = 127
    assert U.run_conv(qa, qw, d)["acc"][0, 2, 3, 3] == 9 * 127 * 255 * c


def test_gemm_as_1x1_conv(ebs, U, oracle):
    """The bit-plane GEMM of the bitwidth sweep, reduced: 256 x 192 x 1024 as a 1x1 convolution."""
    rng = np.random.default_rng(4)
    qa = U.rand_codes(rng, (1, 1024, 16, 16), 5, False)
    qw = U.rand_codes(rng, (192, 1024, 1, 1), 6, True)
    d = U.desc_for(1024, 192, 1, 1, 0, 6, 5)
    got = U.run_conv(qa, qw, d)["acc"]
    X = qa.transpose(0, 2, 3, 1).reshape(-1, 1024).astype(np.int64)
    ref = (X @ qw.reshape(192, 1024).astype(np.int64).T).reshape(1, 16, 16, 192).transpose(0, 3, 1, 2)
    assert np.array_equal(got, ref)
    assert np.array_equal(got, oracle.conv2d_codes(qa, qw))


# ------------------------------------------------------------------ epilogue (row a5) and dequant (row a6)

@pytest.mark.parametrize("next_bits,co", [(1, 16), (2, 32), (3, 64), (4, 21), (8, 70), (5, 130)])
def test_fused_epilogue_and_requantized_planes(ebs, U, oracle, next_bits, co):
    rng = np.random.default_rng(next_bits * 100 + co)
    wb, ab, c = 3, 3, 48
    qa = U.rand_codes(rng, (2, c, 9, 10), ab, False)
    qw = U.rand_codes(rng, (co, c, 3, 3), wb, True)
    w_scale, a_scale = 0.037, 0.052
    d = U.desc_for(c, co, 3, 1, 1, wb, ab, w_scale, a_scale)
    ref_acc = oracle.conv2d_codes(qa, qw, (1, 1), (1, 1))
    S = oracle.combined_scale(w_scale, a_scale)
    cs = rng.uniform(0.5, 2.0, co).astype(np.float32)
    cb = rng.uniform(-0.3, 0.3, co).astype(np.float32)
    res = rng.uniform(-0.2, 0.2, ref_acc.shape).astype(np.float32)
    y_ref0, _ = oracle.epilogue(ref_acc, S, cs, cb, res, relu=True)
    next_scale = np.float32(np.percentile(y_ref0, 99) / ((1 << next_bits) - 1) + 1e-6)
    inv_next = np.float32(1.0) / next_scale
    y_ref, q_ref = oracle.epilogue(ref_acc, S, cs, cb, res, relu=True, next_bits=next_bits, inv_next=inv_next)
    to = lambda a: torch.from_numpy(np.ascontiguousarray(a)).to(U.dev())
    res_nhwc = to(res.transpose(0, 2, 3, 1))
    for y_layout in (ebs.EBS_NHWC, ebs.EBS_NCHW):
        epi = ebs.epilogue(to(cs), to(cb), res_nhwc, True, next_bits, float(next_scale), y_layout)
        # the warp-level strip kernels write NHWC only; their 16-channel tile cannot pack wider layers
        # every variant the library accepts for this request (e.g. the warp-level strip kernels write NHWC only and
        # 16-channel tiles cannot pack wider layers: the library says so itself)
        for variant in U.all_variants(d, 10, 9, n=2, epi=epi, want_y=True, want_packed=True, min_count=12):
            out = U.run_conv(qa, qw, d, epi, want_acc=True, want_y=True, next_bits=next_bits, variant=variant)
            assert np.array_equal(out["acc"], ref_acc)
            assert np.allclose(out["y"], y_ref, rtol=RTOL, atol=0.0)
            assert np.array_equal(out["y"], y_ref)                       # same rounded operations: identical
            assert np.array_equal(oracle.unpack_acts(out["packed"], co), q_ref)
            assert np.array_equal(out["packed"], oracle.pack_acts(q_ref, next_bits))
    assert 0 < q_ref.mean() < (1 << next_bits) - 1                       # codes are not degenerate


def test_packed_only_output_feeds_next_layer(ebs, U, oracle):
    """Two chained layers with only packed planes between them equal the oracle's chain."""
    rng = np.random.default_rng(12)
    qa = U.rand_codes(rng, (2, 32, 10, 10), 2, False)
    qw1 = U.rand_codes(rng, (64, 32, 3, 3), 2, True)
    qw2 = U.rand_codes(rng, (40, 64, 1, 1), 4, True)
    d1 = U.desc_for(32, 64, 3, 2, 1, 2, 2, 0.05, 0.1)
    d2 = U.desc_for(64, 40, 1, 1, 0, 4, 3, 0.02, 0.15)
    acc1 = oracle.conv2d_codes(qa, qw1, (2, 2), (1, 1))
    bias = np.full(64, 1.5, np.float32)                   # recentres the pre-activation (a folded BatchNorm shift)
    _, q1 = oracle.epilogue(acc1, oracle.combined_scale(0.05, 0.1), None, bias, None, relu=True, next_bits=3,
                            inv_next=np.float32(1.0) / np.float32(0.15))
    ref2 = oracle.conv2d_codes(q1, qw2)
    epi = ebs.epilogue(ch_bias=torch.from_numpy(bias).to(U.dev()), relu=True, next_a_bits=3, next_a_scale=0.15)
    out1 = U.run_conv(qa, qw1, d1, epi, want_acc=False, next_bits=3)
    assert np.array_equal(oracle.unpack_acts(out1["packed"], 64), q1)
    px2 = torch.from_numpy(out1["packed"].view(np.int32).reshape(-1)).to(U.dev())
    got2 = U.run_conv(q1, qw2, d2, px=px2)["acc"]
    assert np.array_equal(got2, ref2) and q1.max() == 7 and 0.5 < q1.mean() < 6


@pytest.mark.parametrize("co,pixels", [(64, 1000), (21, 333), (3, 50), (16, 4096)])
def test_dequant(ebs, U, oracle, co, pixels):
    rng = np.random.default_rng(co)
    acc = rng.integers(-(1 << 27), 1 << 27, size=(1, co, pixels, 1), dtype=np.int32)
    cs = rng.uniform(0.5, 2.0, co).astype(np.float32)
    cb = rng.uniform(-100, 100, co).astype(np.float32)
    scale = np.float32(0.00173)
    to = lambda a: torch.from_numpy(np.ascontiguousarray(a)).to(U.dev())
    a_dev = to(acc.transpose(0, 2, 3, 1))
    for (s_, b_, relu) in [(None, None, False), (cs, cb, True), (cs, None, False), (None, cb, True)]:
        y = torch.empty((pixels, co), dtype=torch.float32, device=U.dev())
        ebs.ebs_dequant(a_dev, pixels, co, float(scale), None if s_ is None else to(s_), None if b_ is None else to(b_),
                        relu, y)
        torch.cuda.synchronize()
        ref, _ = oracle.epilogue(acc, scale, s_, b_, None, relu)
        got = y.cpu().numpy().reshape(1, pixels, 1, co).transpose(0, 3, 1, 2)
        assert np.allclose(got, ref, rtol=RTOL, atol=0.0) and np.array_equal(got, ref)


def test_host_entry_point(ebs, U, oracle):
    rng = np.random.default_rng(31)
    wb, ab, c, co = 2, 3, 24, 40
    qa = U.rand_codes(rng, (3, c, 12, 9), ab, False)
    qw = U.rand_codes(rng, (co, c, 3, 3), wb, True)
    d = U.desc_for(c, co, 3, 1, 1, wb, ab, 0.03, 0.07)
    pw = U.pack_weight_codes(qw, d)
    ref = oracle.conv2d_codes(qa, qw, (1, 1), (1, 1))
    y_ref, q_ref = oracle.epilogue(ref, oracle.combined_scale(0.03, 0.07), relu=True, next_bits=4,
                                   inv_next=np.float32(1.0) / np.float32(0.05))
    epi = ebs.epilogue(relu=True, next_a_bits=4, next_a_scale=0.05)
    x_host = torch.from_numpy(np.ascontiguousarray(qa.astype(np.uint8).transpose(0, 2, 3, 1))).pin_memory()
    ws = torch.empty(ebs.ebs_host_workspace_bytes(d, 3, 12, 9, ebs.EBS_U8_CODES, 4), dtype=torch.uint8, device=U.dev())
    acc_h = torch.empty((3, 12, 9, co), dtype=torch.int32).pin_memory()
    y_h = torch.empty((3, 12, 9, co), dtype=torch.float32).pin_memory()
    pn_h = torch.empty(ebs.ebs_packed_act_bytes(3, 12, 9, co, 4) // 4, dtype=torch.int32).pin_memory()
    ebs.ebs_conv2d_mixed_host(x_host, ebs.EBS_U8_CODES, ebs.EBS_NHWC, 3, 12, 9, pw, d, epi, ws, acc_h, y_h, pn_h)
    torch.cuda.synchronize()
    assert np.array_equal(acc_h.numpy().transpose(0, 3, 1, 2), ref)
    assert np.array_equal(y_h.numpy().transpose(0, 3, 1, 2), y_ref)
    got_q = oracle.unpack_acts(pn_h.numpy().view(np.uint32).reshape(3, 12, 9, 2, 4), co)
    assert np.array_equal(got_q, q_ref)
    # fp32 host input is quantized on the device
    xf = ((qa + rng.uniform(-0.3, 0.3, qa.shape)) * np.float32(0.07)).astype(np.float32)
    assert np.array_equal(oracle.quantize_acts(xf, 0.07, ab), qa)
    xf_host = torch.from_numpy(xf).pin_memory()
    ws2 = torch.empty(ebs.ebs_host_workspace_bytes(d, 3, 12, 9, ebs.EBS_F32, 0), dtype=torch.uint8, device=U.dev())
    acc_h.zero_()
    ebs.ebs_conv2d_mixed_host(xf_host, ebs.EBS_F32, ebs.EBS_NCHW, 3, 12, 9, pw, d, None, ws2, acc_h, None, None)
    torch.cuda.synchronize()
    assert np.array_equal(acc_h.numpy().transpose(0, 3, 1, 2), ref)


# ------------------------------------------------------------------ edge cases

EDGE = [
    # c_in, c_out, k, stride, pad, h, w, n, wb, ab        what it stresses
    (1, 1, 1, 1, 0, 1, 1, 1, 1, 1),                      # a single bit pair
    (5, 3, 3, 1, 1, 1, 1, 2, 2, 3),                      # 1x1 image: only the centre tap is inside
    (7, 9, 3, 1, 0, 3, 3, 1, 3, 2),                      # kernel covers the whole input: one output pixel
    (33, 2, 1, 3, 0, 7, 8, 1, 4, 4),                     # stride larger than the kernel
    (40, 70, 3, 1, 2, 4, 4, 1, 2, 2),                    # padding larger than needed: border outputs see few taps
    (64, 64, 3, 1, 1, 12, 11, 1, 8, 8),                  # widest codes
    (16, 16, 3, 2, 1, 33, 31, 3, 1, 8),                  # folded taps, odd sizes, stride 2
    (8, 24, 5, 1, 2, 9, 9, 2, 3, 3),                     # four taps per word
    (3, 16, 7, 2, 3, 21, 20, 2, 8, 8),                   # eight taps per word (first-layer shape)
    (257, 5, 1, 1, 0, 3, 130, 1, 5, 6),                  # one image row longer than a pixel tile, ragged channels
]


@pytest.mark.parametrize("case", EDGE)
def test_conv_edge_cases_all_variants(ebs, U, oracle, case):
    c, co, k, s, pad, h, w, n, wb, ab = case
    rng = np.random.default_rng(sum(case))
    qa = U.rand_codes(rng, (n, c, h, w), ab, False)
    qw = U.rand_codes(rng, (co, c, k, k), wb, True)
    d = U.desc_for(c, co, k, s, pad, wb, ab)
    ref = oracle.conv2d_codes(qa, qw, (s, s), (pad, pad))
    px, pw = U.pack_acts_codes(qa, ab), U.pack_weight_codes(qw, d)
    for variant in U.all_variants(d, w, h, n=n, min_count=10):
        got = U.run_conv(qa, qw, d, variant=variant, px=px, pw=pw)["acc"]
        assert got.shape == ref.shape and np.array_equal(got, ref), f"variant {variant}"
    assert ebs.ebs_device_wait_timeouts() == 0


def test_conv_at_the_int32_limit(ebs, U, oracle):
    """The largest reduction 8x8 bits allow (|acc| just below 2^31) with saturated codes, and one more channel refused."""
    c = 65793                                               # 65793 * 128 * 255 = 2^31 - 2^15 - ... < 2^31
    assert c * 128 * 255 < 2 ** 31 <= (c + 1) * 128 * 255
    qa = np.full((1, c, 1, 2), 255, dtype=np.int32)
    qw = np.full((2, c, 1, 1), -128, dtype=np.int32)
    qw[1] = 127
    d = U.desc_for(c, 2, 1, 1, 0, 8, 8)
    got = U.run_conv(qa, qw, d)["acc"]
    assert got[0, 0, 0, 0] == -128 * 255 * c and got[0, 1, 0, 1] == 127 * 255 * c
    assert np.array_equal(got, oracle.conv2d_codes(qa, qw))
    with pytest.raises(ebs.EbsError) as err:
        ebs.ebs_packed_weight_bytes(U.desc_for(c + 1, 2, 1, 1, 0, 8, 8)) or ebs.ebs_conv_out_shape(
            U.desc_for(c + 1, 2, 1, 1, 0, 8, 8), 1, 2)
    assert err.value.status == ebs.EBS_ERR_OVERFLOW


# ------------------------------------------------------------------ the paper's own weight levels (w_levels = 1)

@pytest.mark.parametrize("wb,ab,c,co,k,s,pad", [(1, 1, 16, 16, 3, 1, 1), (1, 2, 64, 64, 3, 1, 1), (2, 3, 40, 21, 3, 2, 1),
                                                (4, 4, 128, 70, 1, 1, 0), (8, 8, 33, 9, 3, 1, 0), (3, 5, 8, 130, 5, 1, 2)])
def test_conv_with_paper_weight_levels_all_variants(ebs, U, oracle, wb, ab, c, co, k, s, pad):
    rng = np.random.default_rng(wb * 100 + ab * 10 + k)
    qa = U.rand_codes(rng, (2, c, 10, 9), ab, False)
    qs = U.rand_codes(rng, (co, c, k, k), wb, True)
    L = (1 << wb) - 1
    d = ebs.conv_desc(c, co, k, k, s, s, pad, pad, wb, ab, 1.0 / L, 0.05, w_levels=1)
    ref = oracle.conv2d_levels(qa, qs, (s, s), (pad, pad))
    S = oracle.combined_scale(1.0 / L, 0.05)
    y_ref, q_ref = oracle.epilogue(ref, S, relu=True, next_bits=3, inv_next=np.float32(1.0) / np.float32(0.4))
    px, pw = U.pack_acts_codes(qa, ab), U.pack_weight_codes(qs, d)
    epi = ebs.epilogue(relu=True, next_a_bits=3, next_a_scale=0.4)
    for variant in U.all_variants(d, 9, 10, n=2, epi=epi, want_y=True, want_packed=True, min_count=8):
        out = U.run_conv(qa, qs, d, epi, want_acc=True, want_y=True, next_bits=3, variant=variant, px=px, pw=pw)
        assert np.array_equal(out["acc"], ref), f"variant {variant}"
        assert np.array_equal(out["y"], y_ref), f"variant {variant}"
        assert np.array_equal(oracle.unpack_acts(out["packed"], co), q_ref), f"variant {variant}"


def test_pack_weights_fp32_to_paper_levels(ebs, U, oracle):
    rng = np.random.default_rng(5)
    wb, c, co, k = 3, 20, 12, 3
    L = (1 << wb) - 1
    w = rng.uniform(-1.1, 1.1, size=(co, c, k, k)).astype(np.float32)
    qs = oracle.quantize_weight_levels(w, 1.0 / L, wb)
    assert qs.min() == -(1 << (wb - 1)) and qs.max() == (1 << (wb - 1)) - 1
    d = ebs.conv_desc(c, co, k, k, 1, 1, 1, 1, wb, 2, 1.0 / L, 0.05, w_levels=1)
    out = torch.empty(ebs.ebs_packed_weight_bytes(d) // 4, dtype=torch.int32, device=U.dev())
    ebs.ebs_pack_weights(torch.from_numpy(w).to(U.dev()), ebs.EBS_F32, ebs.EBS_NCHW, d, out)
    assert np.array_equal(U.weight_planes(out, d), oracle.pack_weights(qs, wb))


def test_tensor_core_probe_runs_and_is_in_range(ebs):
    """ebs_probe_pipe kind 4 (tcgen05.mma kind::i8 from shared memory): returns, its bounded wait does not run out, and
    the rate lies between the warp-level int8 MMA's and twice the nominal dense int8 figure."""
    umma = 2 * ebs.ebs_probe_pipe(4, 500) / 1e12
    imma = 2 * ebs.ebs_probe_pipe(3, 200) / 1e12
    assert imma < umma < 9000.0, (imma, umma)
    assert ebs.ebs_device_wait_timeouts() == 0
