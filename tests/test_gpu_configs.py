"""Parity of the five benchmark configurations against the CPU oracle, on the same seeded inputs.

Full sizes run on the GPU exactly as bench.py launches them (heuristic kernel choice); the oracle
checks every output where it finishes in seconds (configs 1 and 2) and otherwise every output of
sampled images / sampled GEMM rows, which it computes one by one.
"""
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


@pytest.fixture(scope="module")
def gen():
    from workloads import gen as g
    return g


def check_layer(ebs, U, oracle, spec, qa, qw, sample=None, next_bits=3):
    """One layer at full batch on the GPU; oracle on all images or on `sample` images."""
    L = spec.layer
    n = qa.shape[0]
    d = U.spec_desc(spec)
    px, pw = U.pack_acts_codes(qa, spec.a_bits, ebs.EBS_NHWC), U.pack_weight_codes(qw, d)
    idx = list(range(n)) if sample is None else sample
    ref = oracle.conv2d_codes(qa[idx], qw, (L.stride, L.stride), (L.pad, L.pad))
    S = oracle.combined_scale(spec.w_scale, spec.a_scale)
    bias = np.full(L.c_out, -float(np.mean(ref)) * float(S), np.float32)           # centre the pre-activation
    y0, _ = oracle.epilogue(ref, S, None, bias, None, relu=True)
    next_scale = np.float32(max(np.percentile(y0, 99.5), 1e-6) / ((1 << next_bits) - 1))
    y_ref, q_ref = oracle.epilogue(ref, S, None, bias, None, relu=True, next_bits=next_bits,
                                   inv_next=np.float32(1.0) / next_scale)
    epi = ebs.epilogue(ch_bias=torch.from_numpy(bias).to(U.dev()), relu=True, next_a_bits=next_bits,
                       next_a_scale=float(next_scale))
    acc, y, pn = U.conv_on_device(px, n, L.h_in, L.w_in, pw, d, epi, True, True, next_bits)
    torch.cuda.synchronize()
    assert np.array_equal(U.images_nchw(acc, idx), ref), f"{L.name}: int32 accumulators"
    if sample is not None:
        # every image of the batch, interior ones included: the chosen kernel against the integer-pipe family on the GPU
        # (the literal plane-pair evaluation, itself oracle-checked on the sampled images just above and in the small cases)
        acc2 = torch.empty_like(acc)
        pn2 = torch.empty_like(pn)
        ebs.ebs_conv2d_mixed(px, n, L.h_in, L.w_in, pw, d, epi, acc2, None, pn2, variant=-2)
        torch.cuda.synchronize()
        assert torch.equal(acc, acc2), f"{L.name}: accumulators of the whole batch differ between kernel families"
        assert torch.equal(pn, pn2), f"{L.name}: packed planes of the whole batch differ between kernel families"
    got_y = U.images_nchw(y, idx)
    assert np.allclose(got_y, y_ref, rtol=RTOL, atol=0.0), f"{L.name}: fp32 outputs"
    got_q = oracle.unpack_acts(U.packed_images(pn, n, L.h_out, L.w_out, L.c_out, next_bits, idx), L.c_out)
    assert np.array_equal(got_q, q_ref), f"{L.name}: requantized codes"
    assert q_ref.max() == (1 << next_bits) - 1 and q_ref.min() == 0


def test_config1_single_layer(ebs, U, oracle, gen):
    spec = gen.config1(0)[0]
    check_layer(ebs, U, oracle, spec, gen.act_codes(spec), gen.weight_codes(spec), next_bits=2)


def test_config2_resnet20_full_batch(ebs, U, oracle, gen):
    """All 22 layers (first conv and classifier as W8A8) at batch 128, every output checked."""
    specs = gen.config2(0)
    assert len(specs) == 22
    for spec in specs:
        check_layer(ebs, U, oracle, spec, gen.act_codes(spec), gen.weight_codes(spec), next_bits=max(1, spec.a_bits % 5))


def test_config2_in_the_bench_launch_configuration(ebs, U, oracle, gen):
    """The 20 quantized layers at batch 128 exactly as bench.py launches them: no per-channel term, ReLU, int32
    accumulators plus the next layer's planes (its bit count, step 4 * s_w * s_a * c_in), the library's own kernel
    choice -- the form of the kernels without per-channel and shortcut terms. Every output is checked."""
    specs = [s for s in gen.config2(0) if s.layer.quantized]
    assert len(specs) == 20
    for i, spec in enumerate(specs):
        L = spec.layer
        next_bits = specs[(i + 1) % len(specs)].a_bits
        next_scale = np.float32(4.0 * spec.w_scale * spec.a_scale * L.c_in)
        qa, qw = gen.act_codes(spec), gen.weight_codes(spec)
        d = U.spec_desc(spec)
        px, pw = U.pack_acts_codes(qa, spec.a_bits, ebs.EBS_NHWC), U.pack_weight_codes(qw, d)
        ref = oracle.conv2d_codes(qa, qw, (L.stride, L.stride), (L.pad, L.pad))
        S = oracle.combined_scale(spec.w_scale, spec.a_scale)
        _, q_ref = oracle.epilogue(ref, S, None, None, None, relu=True, next_bits=next_bits,
                                   inv_next=np.float32(1.0) / next_scale)
        epi = ebs.epilogue(relu=True, next_a_bits=next_bits, next_a_scale=float(next_scale))
        acc, _, pn = U.conv_on_device(px, spec.batch, L.h_in, L.w_in, pw, d, epi, True, False, next_bits)
        torch.cuda.synchronize()
        idx = list(range(spec.batch))
        assert np.array_equal(U.images_nchw(acc, idx), ref), f"{L.name}: int32 accumulators"
        got_q = oracle.unpack_acts(U.packed_images(pn, spec.batch, L.h_out, L.w_out, L.c_out, next_bits, idx), L.c_out)
        assert np.array_equal(got_q, q_ref), f"{L.name}: requantized codes"
        assert np.array_equal(pn.cpu().numpy().view(np.uint32).ravel(),
                              oracle.pack_acts(q_ref, next_bits).ravel()), f"{L.name}: packed words (pad bits zero)"


def test_config3_resnet18_batch64_sampled_images(ebs, U, oracle, gen):
    for spec in gen.config3(0):
        qa = gen.act_codes(spec)
        n = qa.shape[0]
        picks = sorted({0, n - 1, *(int(v) for v in np.random.default_rng(spec.index).integers(1, n - 1, size=2))})
        check_layer(ebs, U, oracle, spec, qa, gen.weight_codes(spec), sample=picks, next_bits=4)


def test_config4_bitplane_gemm_all_pairs(ebs, U, oracle, gen):
    """4096^3 bit-plane GEMM for all 64 (Wb, Ab): full size on the GPU, oracle on sampled rows."""
    rng = np.random.default_rng(0)
    base_a = rng.integers(0, 256, size=(1, 4096, 64, 64), dtype=np.int32)
    base_w = rng.integers(0, 256, size=(4096, 4096, 1, 1), dtype=np.int32)
    rows = [(0, 0), (0, 63), (17, 5), (31, 32), (63, 63), (40, 1)]
    for wb in range(1, 9):
        u = base_w & ((1 << wb) - 1)
        qw = np.where(u >= (1 << (wb - 1)), u - (1 << wb), u).astype(np.int32)   # uniform signed codes
        spec0 = gen.config4(wb, 1)
        d_w = U.spec_desc(spec0)
        pw = U.pack_weight_codes(qw, d_w)
        for ab in range(1, 9):
            spec = gen.config4(wb, ab)
            qa = base_a & ((1 << ab) - 1)
            d = U.spec_desc(spec)
            px = U.pack_acts_codes(qa, ab, ebs.EBS_NHWC)
            acc, _, _ = U.conv_on_device(px, 1, 64, 64, pw, d)
            torch.cuda.synchronize()
            got = acc.cpu().numpy()                                      # [1, 64, 64, 4096]
            sel = np.stack([qa[0, :, r, c] for r, c in rows]).reshape(len(rows), 4096, 1, 1)
            ref = oracle.conv2d_codes(sel, qw)                           # [rows, 4096, 1, 1]
            for i, (r, c) in enumerate(rows):
                assert np.array_equal(got[0, r, c], ref[i, :, 0, 0]), f"W{wb}A{ab} row ({r},{c})"
            if (wb, ab) in ((1, 1), (3, 5), (5, 2), (8, 8)):           # every output: against the integer-pipe family on the GPU
                acc2 = torch.empty_like(acc)
                ebs.ebs_conv2d_mixed(px, 1, 64, 64, pw, d, None, acc2, None, None, variant=-2)
                torch.cuda.synchronize()
                assert torch.equal(acc, acc2), f"W{wb}A{ab}: kernel families disagree"
            # a property that holds at any size: column sums of acc = (sum of activation rows) . weights
            if (wb, ab) in ((1, 1), (4, 4), (8, 8)):
                colsum = got[0].reshape(-1, 4096).astype(np.int64).sum(axis=0)
                asum = qa[0].reshape(4096, -1).astype(np.int64).sum(axis=1)
                assert np.array_equal(colsum, qw.reshape(4096, 4096).astype(np.int64) @ asum)


def test_config5_resnet50_chain_batch256_sampled_images(ebs, U, oracle, gen):
    """The bottleneck stack chained through fused requantization: layer l's packed output is layer
    l+1's input.  The oracle runs the same chain on two sampled images and fixes the per-layer
    requantization steps; the GPU runs the full batch and must reproduce the sampled images' codes."""
    specs = gen.config5(0)
    n = specs[0].batch
    sample = [0, 101, n - 1]                                 # first, an interior and the last image
    qa0 = gen.act_codes(specs[0])
    L0 = specs[0].layer
    # ---- oracle chain on the sampled images (also decides bias / next step per layer)
    plan, x_ref, block_in = [], qa0[sample], None
    by_name = {s.layer.name: i for i, s in enumerate(specs)}
    for i, spec in enumerate(specs):
        L = spec.layer
        qw = gen.weight_codes(spec)
        if L.name.endswith("c1"):
            block_in = x_ref
        src = block_in if L.role == "shortcut" else x_ref
        nxt = specs[i + 1] if i + 1 < len(specs) else spec
        if nxt.layer.role == "shortcut":                      # c3 feeds the next block's c1, not the shortcut
            nxt = specs[i + 2] if i + 2 < len(specs) else spec
        nb = nxt.a_bits
        acc = oracle.conv2d_codes(src, qw, (L.stride, L.stride), (L.pad, L.pad))
        S = oracle.combined_scale(spec.w_scale, spec.a_scale)
        bias = np.full(L.c_out, -float(np.mean(acc)) * float(S), np.float32)
        y0, _ = oracle.epilogue(acc, S, None, bias, None, relu=True)
        step = np.float32(max(np.percentile(y0, 99.5), 1e-6) / ((1 << nb) - 1))
        _, q = oracle.epilogue(acc, S, None, bias, None, relu=True, next_bits=nb, inv_next=np.float32(1.0) / step)
        plan.append((bias, float(step), nb, q))
        if L.role != "shortcut":
            x_ref = q
    # ---- GPU chain at full batch
    px = U.pack_acts_codes(qa0, specs[0].a_bits, ebs.EBS_NHWC)
    del qa0
    block_px = None
    for i, spec in enumerate(specs):
        L = spec.layer
        bias, step, nb, q_ref = plan[i]
        d = U.spec_desc(spec)
        pw = U.pack_weight_codes(gen.weight_codes(spec), d)
        if L.name.endswith("c1"):
            block_px = px
        src = block_px if L.role == "shortcut" else px
        epi = ebs.epilogue(ch_bias=torch.from_numpy(bias).to(U.dev()), relu=True, next_a_bits=nb, next_a_scale=step)
        _, _, pn = U.conv_on_device(src, n, L.h_in, L.w_in, pw, d, epi, want_acc=False, next_bits=nb)
        torch.cuda.synchronize()
        got = oracle.unpack_acts(U.packed_images(pn, n, L.h_out, L.w_out, L.c_out, nb, sample), L.c_out)
        assert np.array_equal(got, q_ref), f"layer {i} {L.name} W{spec.w_bits}A{spec.a_bits}"
        assert q_ref.max() > 0
        if L.role != "shortcut":
            px = pn
