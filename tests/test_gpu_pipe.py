"""The persistent pipeline tcgen05 kernels (family "umma_pipe") against the CPU oracle: every stride form of the
addressing (stride 1, strided k x k as phase images, strided 1x1), several accumulators per tile, resident and
streamed weights, many tiles per thread block, all activation bit counts, and the give-up path of its bounded waits."""
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


def _check(ebs, U, oracle, n, c, co, k, s, pad, h, w, wb, ab, nb, affine=False, min_variants=1, only=None):
    rng = np.random.default_rng(n + 3 * c + 5 * co + 7 * k + 11 * s + h + w + wb * 16 + ab)
    qa = U.rand_codes(rng, (n, c, h, w), ab, False)
    m = (1 << (wb - 1)) - 1
    assert m >= 1
    qw = rng.integers(-m, m + 1, size=(co, c, k, k), dtype=np.int32)   # symmetric codes: zero-mean accumulators, half survive the ReLU
    d = U.desc_for(c, co, k, s, pad, wb, ab, 0.03, 0.07)
    ref = oracle.conv2d_codes(qa, qw, (s, s), (pad, pad))
    S = oracle.combined_scale(0.03, 0.07)
    cs = rng.uniform(0.5, 2.0, co).astype(np.float32) if affine else None
    cb = rng.uniform(-0.3, 0.3, co).astype(np.float32) if affine else None
    y0, _ = oracle.epilogue(ref, S, cs, cb, None, relu=True)
    step = np.float32(max(float(np.percentile(y0, 99)), 1e-3) / ((1 << nb) - 1))
    y_ref, q_ref = oracle.epilogue(ref, S, cs, cb, None, relu=True, next_bits=nb, inv_next=np.float32(1.0) / step)
    to = lambda a: None if a is None else torch.from_numpy(a).to(U.dev())
    epi = ebs.epilogue(to(cs), to(cb), None, True, nb, float(step))
    px, pw = U.pack_acts_codes(qa, ab), U.pack_weight_codes(qw, d)
    ran = 0
    for variant in U.variants_of("umma_pipe"):
        if only is not None and variant != only:
            continue
        if not U.applies(d, h, w, variant, n=n, epi=epi, want_y=True, want_packed=True):
            continue
        out = U.run_conv(qa, qw, d, epi, want_acc=True, want_y=True, next_bits=nb, variant=variant, px=px, pw=pw)
        assert np.array_equal(out["acc"], ref), f"variant {variant}: accumulators"
        assert np.array_equal(out["y"], y_ref), f"variant {variant}: fp32 outputs"
        assert np.array_equal(out["packed"], oracle.pack_acts(q_ref, nb)), f"variant {variant}: packed words"
        # packed-only output (the mode a network runs in)
        out = U.run_conv(qa, qw, d, epi, want_acc=False, want_y=False, next_bits=nb, variant=variant, px=px, pw=pw)
        assert np.array_equal(out["packed"], oracle.pack_acts(q_ref, nb)), f"variant {variant}: packed only"
        ran += 1
    assert ran >= min_variants
    assert q_ref.max() == (1 << nb) - 1
    assert ebs.ebs_device_wait_timeouts() == 0


@pytest.mark.parametrize("ab", range(1, 9))
@pytest.mark.parametrize("nb", [1, 3, 4, 8])
def test_pipe_all_activation_and_output_bit_counts(ebs, U, oracle, ab, nb):
    """3x3 stride 1, 64 -> 128 channels, whole channel tiles (the straight-line epilogue), several tiles."""
    _check(ebs, U, oracle, 5, 64, 128, 3, 1, 1, 14, 13, 2 + (ab + nb) % 7, ab, nb, min_variants=2)


@pytest.mark.parametrize("case", [
    # n, c, co, k, stride, pad, h, w
    (6, 64, 64, 3, 2, 1, 15, 14),       # strided 3x3: four phase images, odd and even sizes
    (3, 96, 128, 3, 2, 1, 16, 16),
    (4, 64, 256, 1, 2, 0, 14, 14),      # strided 1x1: one phase
    (2, 128, 64, 1, 1, 0, 20, 19),      # 1x1 stride 1: up to four accumulators per tile
    (2, 40, 70, 3, 1, 1, 9, 12),        # ragged input and output channels: general epilogue
    (3, 64, 64, 5, 2, 2, 13, 13),       # 5x5 stride 2: taps with quotients -1, 0, 1
    (2, 32, 64, 2, 2, 0, 12, 12),       # even kernel, stride = kernel
    (1, 64, 64, 3, 1, 0, 8, 8),         # no padding
    (3, 64, 128, 7, 2, 3, 20, 18),      # 49 taps
    (9, 256, 128, 3, 1, 1, 7, 7),       # small images: a strip spans several images
])
@pytest.mark.parametrize("affine", [False, True])
def test_pipe_geometries(ebs, U, oracle, case, affine):
    n, c, co, k, s, pad, h, w = case
    _check(ebs, U, oracle, n, c, co, k, s, pad, h, w, 3, 4, 4, affine=affine)


@pytest.mark.parametrize("case", [
    # n, c, co, k, stride, pad, h, w, ab
    (3, 64, 256, 1, 1, 0, 20, 19, 6),     # resident weights, one pair-tile and a ragged second one
    (4, 512, 256, 3, 1, 1, 9, 9, 3),      # streamed weights through the ring, strip halo across images
    (2, 1024, 512, 1, 1, 0, 24, 24, 8),   # deep reduction, two channel tiles, two accumulators per CTA
    (5, 128, 256, 3, 2, 1, 17, 16, 5),    # strided 3x3: four phase images
    (70, 64, 256, 1, 1, 0, 28, 28, 2),    # more pair-tiles than CTA pairs: the rings and both accumulator sets wrap
])
def test_pipe_cta_pair(ebs, U, oracle, case):
    """The 256-channel tile on a pair of CTAs (one MMA of 256 pixels over two SMs, half a weight tile each): the last
    variant of the family, forced."""
    n, c, co, k, s, pad, h, w, ab = case
    pair = U.variants_of("umma_pipe")[-1]
    _check(ebs, U, oracle, n, c, co, k, s, pad, h, w, 4, ab, 4, min_variants=1, only=pair)


def test_pipe_cta_pair_declines_what_it_does_not_cover(ebs, U):
    pair = U.variants_of("umma_pipe")[-1]
    d = U.desc_for(64, 128, 3, 1, 1, 4, 4, 0.03, 0.07)                 # 128 output channels: no whole 256-channel tile
    assert not U.applies(d, 16, 16, pair, n=2)
    d = U.desc_for(64, 256, 3, 1, 1, 4, 4, 0.03, 0.07)
    assert U.applies(d, 16, 16, pair, n=2)
    cs = torch.ones(256, device=U.dev())
    epi = ebs.epilogue(cs, None, None, True, 4, 1.0)                   # per-channel terms: the other variants
    assert not U.applies(d, 16, 16, pair, n=2, epi=epi, want_packed=True)


def test_pipe_streams_weights_that_do_not_fit_in_shared_memory(ebs, U, oracle):
    """512 -> 256 channels, 3x3: 1.2 MB of weight bytes per 256-channel tile stream through the stage ring."""
    _check(ebs, U, oracle, 4, 512, 256, 3, 1, 1, 9, 9, 4, 3, 3, min_variants=3)
    _check(ebs, U, oracle, 2, 2048, 512, 1, 1, 0, 10, 10, 2, 5, 2, min_variants=3)


def test_pipe_many_tiles_per_thread_block(ebs, U, oracle):
    """More work items than SMs: the stage ring, both accumulator sets and the item loop wrap around several times."""
    _check(ebs, U, oracle, 40, 64, 64, 3, 1, 1, 34, 34, 2, 2, 2, min_variants=1)
    _check(ebs, U, oracle, 64, 64, 256, 1, 1, 0, 28, 28, 5, 6, 5, min_variants=3)


def test_pipe_requantization_where_two_roundings_and_a_fused_one_differ(ebs, U, oracle):
    """y * (1/step) + 0.5 must be a rounded multiply followed by a rounded addition.  With the step 4 * s_w * s_a * 64 of
    the ResNet-20 bench layers the product at acc = 128 is the float just below 0.5, the sum rounds up to 1.0 (a tie, to
    even) and the code is 1; a fused multiply-add keeps the sum below 1.0 and gives 0.  A 1x1 layer with unit weights
    sweeps the accumulator over 0 .. 765 so that such values are present for every output bit count."""
    spec = [s for s in __import__("workloads.gen", fromlist=["gen"]).config2(0) if s.layer.name == "s3b3c1"][0]
    n, c, co, h, w = 4, 64, 64, 16, 12
    qa = np.zeros((n, c, h, w), np.int32)
    target = np.arange(n * h * w).reshape(n, h, w)                     # accumulator value wanted at each pixel
    for ch in range(c):                                               # spread it over channels with codes 0 .. 255
        take = np.clip(target - qa.sum(axis=1), 0, 15)
        qa[:, ch] = take
    qw = np.ones((co, c, 1, 1), np.int32)
    d = U.desc_for(c, co, 1, 1, 0, 2, 4, spec.w_scale, spec.a_scale)
    ref = oracle.conv2d_codes(qa, qw)
    assert ref.max() >= 700 and (ref == 128).any()
    S = oracle.combined_scale(spec.w_scale, spec.a_scale)
    step = np.float32(4.0 * spec.w_scale * spec.a_scale * 64)
    px, pw = U.pack_acts_codes(qa, 4), U.pack_weight_codes(qw, d)
    fused_differs = 0
    for nb in (1, 2, 3, 5):
        inv = np.float32(1.0) / step
        _, q_ref = oracle.epilogue(ref, S, relu=True, next_bits=nb, inv_next=inv)
        y = (ref.astype(np.float32) * S).astype(np.float64)
        q_fused = np.clip(np.floor((y * np.float64(inv) + 0.5).astype(np.float32)), 0, (1 << nb) - 1)   # one rounding
        fused_differs += int((q_fused != q_ref).sum())
        epi = ebs.epilogue(relu=True, next_a_bits=nb, next_a_scale=float(step))
        for variant in [-1] + U.variants_of("umma_pipe"):
            if variant >= 0 and not U.applies(d, h, w, variant, n=n, epi=epi, want_packed=True):
                continue
            out = U.run_conv(qa, qw, d, epi, want_acc=True, next_bits=nb, variant=variant, px=px, pw=pw)
            assert np.array_equal(out["acc"], ref)
            assert np.array_equal(oracle.unpack_acts(out["packed"], co), q_ref), f"variant {variant}, {nb} bits"
    assert fused_differs > 0, "the case no longer separates a fused multiply-add from two rounded operations"


@pytest.mark.parametrize("case", [
    # n, c, co, k, stride, pad, h, w, code bits
    (3, 64, 64, 3, 1, 1, 14, 13, 8), (2, 128, 256, 1, 1, 0, 12, 12, 5), (4, 64, 128, 3, 2, 1, 15, 14, 3),
    (2, 512, 128, 1, 2, 0, 10, 10, 8), (2, 96, 70, 3, 1, 1, 9, 9, 4),
])
def test_context_path_on_unpacked_byte_codes(ebs, U, oracle, case):
    """ebs_conv2d_i8 (activations as u8 NHWC codes, no bit planes): same accumulators, y and packed planes as the oracle."""
    n, c, co, k, s, pad, h, w, ab = case
    rng = np.random.default_rng(sum(case))
    qa = U.rand_codes(rng, (n, c, h, w), ab, False)
    qw = rng.integers(-3, 4, size=(co, c, k, k), dtype=np.int32)
    d = U.desc_for(c, co, k, s, pad, 3, ab, 0.03, 0.07)
    ref = oracle.conv2d_codes(qa, qw, (s, s), (pad, pad))
    S = oracle.combined_scale(0.03, 0.07)
    y0, _ = oracle.epilogue(ref, S, relu=True)
    step = np.float32(max(float(np.percentile(y0, 99)), 1e-3) / 15)
    y_ref, q_ref = oracle.epilogue(ref, S, relu=True, next_bits=4, inv_next=np.float32(1.0) / step)
    x = torch.from_numpy(np.ascontiguousarray(qa.astype(np.uint8).transpose(0, 2, 3, 1))).to(U.dev())
    pw = U.pack_weight_codes(qw, d)
    ho, wo = ebs.ebs_conv_out_shape(d, h, w)
    acc = torch.empty((n, ho, wo, co), dtype=torch.int32, device=U.dev())
    y = torch.empty((n, ho, wo, co), dtype=torch.float32, device=U.dev())
    pn = torch.empty(ebs.ebs_packed_act_bytes(n, ho, wo, co, 4) // 4, dtype=torch.int32, device=U.dev())
    epi = ebs.epilogue(relu=True, next_a_bits=4, next_a_scale=float(step))
    ebs.ebs_conv2d_i8(x, n, h, w, pw, d, epi, acc, y, pn)
    torch.cuda.synchronize()
    assert np.array_equal(acc.cpu().numpy().transpose(0, 3, 1, 2), ref)
    assert np.array_equal(y.cpu().numpy().transpose(0, 3, 1, 2), y_ref)
    assert np.array_equal(U.as_u32(pn).reshape(n, ho, wo, (co + 31) // 32, 4), oracle.pack_acts(q_ref, 4))


def test_context_path_refuses_what_it_cannot_run(ebs, U):
    d = U.desc_for(48, 64, 3, 1, 1, 3, 4)                          # c_in not a multiple of 32
    x = torch.zeros((1, 8, 8, 48), dtype=torch.uint8, device=U.dev())
    pw = torch.zeros(ebs.ebs_packed_weight_bytes(d) // 4, dtype=torch.int32, device=U.dev())
    acc = torch.empty((1, 8, 8, 64), dtype=torch.int32, device=U.dev())
    with pytest.raises(ebs.EbsError) as err:
        ebs.ebs_conv2d_i8(x, 1, 8, 8, pw, d, None, acc)
    assert err.value.status == ebs.EBS_ERR_UNSUPPORTED


def test_pipe_declines_layers_wider_than_its_zero_page(ebs, U, oracle):
    """The expanders read padding from a page of 8192 zero words, which has to cover a pixel's words at 8 planes: a layer
    with more than 32768 input channels goes to another kernel family, and the library's own choice stays exact."""
    c, co = 32768 + 64, 64
    d = U.desc_for(c, co, 1, 1, 0, 2, 2, 0.03, 0.07)
    for variant in U.variants_of("umma_pipe"):
        assert not U.applies(d, 4, 4, variant, n=1)
    rng = np.random.default_rng(11)
    qa = U.rand_codes(rng, (1, c, 4, 4), 2, False)
    qw = rng.integers(-1, 2, size=(co, c, 1, 1), dtype=np.int32)
    out = U.run_conv(qa, qw, d, None, want_acc=True)
    assert np.array_equal(out["acc"], oracle.conv2d_codes(qa, qw, (1, 1), (0, 0)))
