"""The no-allocation host call against the ordinary host call (collected last on purpose).

Some users of the library run where device allocation is off limits (inside another framework's
memory pool, under a fixed memory budget, in a loop that must never block on the allocator); for
them ebs_conv2d_mixed_host_noalloc keeps its scratch in a fixed 32 MiB array inside the library.
Its results must equal those of ebs_conv2d_mixed_host, call after call, although every call reuses
the same scratch bytes and finds the previous call's data in them.
"""
import numpy as np
import pytest
import torch

pytestmark = pytest.mark.gpu


def _host_layer(ebs, dev, rng, n, c, co, h, w, wb, ab, next_bits, use_noalloc, check_free=False):
    """Runs one layer from pinned host buffers through either entry point; returns host results."""
    qa = rng.integers(0, 1 << ab, size=(n, h, w, c), dtype=np.int32).astype(np.uint8)          # NHWC codes
    qw = rng.integers(-(1 << (wb - 1)), 1 << (wb - 1), size=(co, c, 3, 3), dtype=np.int32).astype(np.int8)
    d = ebs.conv_desc(c, co, 3, 3, 1, 1, 1, 1, wb, ab, 0.031, 0.047)
    pw = torch.empty(ebs.ebs_packed_weight_bytes(d) // 4, dtype=torch.int32, device=dev)
    ebs.ebs_pack_weights(torch.from_numpy(qw).to(dev), ebs.EBS_I8_CODES, ebs.EBS_NCHW, d, pw)
    bias = torch.full((co,), 0.8, dtype=torch.float32, device=dev)
    epi = ebs.epilogue(ch_bias=bias, relu=True, next_a_bits=next_bits, next_a_scale=0.21)
    x_host = torch.from_numpy(qa).pin_memory()
    acc = torch.zeros((n, h, w, co), dtype=torch.int32).pin_memory()
    y = torch.zeros((n, h, w, co), dtype=torch.float32).pin_memory()
    pn = torch.zeros(ebs.ebs_packed_act_bytes(n, h, w, co, next_bits) // 4, dtype=torch.int32).pin_memory()
    if use_noalloc:
        torch.cuda.synchronize()
        free_before = torch.cuda.mem_get_info(dev)[0]
        ebs.ebs_conv2d_mixed_host_noalloc(x_host, ebs.EBS_U8_CODES, ebs.EBS_NHWC, n, h, w, pw, d, epi, acc, y, pn)
        torch.cuda.synchronize()
        if check_free:          # after the first call on the device (which may load the module): no device memory taken
            assert torch.cuda.mem_get_info(dev)[0] == free_before, "the no-allocation call changed free device memory"
    else:
        ws = torch.empty(ebs.ebs_host_workspace_bytes(d, n, h, w, ebs.EBS_U8_CODES, next_bits), dtype=torch.uint8,
                         device=dev)
        ebs.ebs_conv2d_mixed_host(x_host, ebs.EBS_U8_CODES, ebs.EBS_NHWC, n, h, w, pw, d, epi, ws, acc, y, pn)
    torch.cuda.synchronize()
    return acc.numpy().copy(), y.numpy().copy(), pn.numpy().copy()


def test_noalloc_host_call_matches_host_call_twice_in_a_row():
    if not torch.cuda.is_available():
        pytest.skip("needs a CUDA device")
    from paper_2003_07577_b200 import binding as ebs
    ebs.lib()
    dev = torch.device("cuda:0")
    torch.cuda.set_device(dev)
    assert ebs.ebs_noalloc_scratch_bytes() == 32 << 20
    # two different layers back to back: the second call finds the first call's bytes in the scratch
    cases = [dict(n=3, c=40, co=48, h=17, w=13, wb=3, ab=2, next_bits=4),
             dict(n=2, c=16, co=21, h=9, w=30, wb=2, ab=4, next_bits=2)]
    for i, case in enumerate(cases):
        ref = _host_layer(ebs, dev, np.random.default_rng(100 + i), use_noalloc=False, **case)
        got = _host_layer(ebs, dev, np.random.default_rng(100 + i), use_noalloc=True, check_free=i > 0, **case)
        assert np.array_equal(got[0], ref[0]), f"call {i}: int32 accumulators differ"
        assert np.allclose(got[1], ref[1], rtol=1e-5, atol=0.0), f"call {i}: fp32 outputs differ"
        assert np.array_equal(got[2], ref[2]), f"call {i}: packed planes differ"
        assert np.abs(ref[0]).max() > 0 and ref[2].any()


def test_noalloc_rejects_layers_beyond_its_scratch():
    if not torch.cuda.is_available():
        pytest.skip("needs a CUDA device")
    from paper_2003_07577_b200 import binding as ebs
    d = ebs.conv_desc(64, 64, 3, 3, 1, 1, 1, 1, 2, 2, 0.05, 0.05)
    assert ebs.ebs_host_workspace_bytes(d, 64, 56, 56, ebs.EBS_U8_CODES, 2) > ebs.ebs_noalloc_scratch_bytes()
    x = torch.zeros(16, dtype=torch.uint8)
    pw = torch.zeros(ebs.ebs_packed_weight_bytes(d) // 4, dtype=torch.int32, device="cuda:0")
    out = torch.zeros(16, dtype=torch.int32)
    with pytest.raises(ebs.EbsError) as err:
        ebs.ebs_conv2d_mixed_host_noalloc(x, ebs.EBS_U8_CODES, ebs.EBS_NHWC, 64, 56, 56, pw, d, None, out, None, None)
    assert err.value.status == ebs.EBS_ERR_SCRATCH_TOO_SMALL and "scratch" in str(err.value)


def test_noalloc_accepts_a_layer_that_fills_its_scratch_exactly():
    """A layer whose workspace need equals the built-in scratch to the byte is served, and matches the oracle-checked
    host call; one more image is refused, and a call refused for a bad argument leaves nothing enqueued."""
    if not torch.cuda.is_available():
        pytest.skip("needs a CUDA device")
    from paper_2003_07577_b200 import binding as ebs
    ebs.lib()
    dev = torch.device("cuda:0")
    torch.cuda.set_device(dev)
    limit = ebs.ebs_noalloc_scratch_bytes()
    # 1x1 layer, u8 codes in, int32 accumulators out: need = n*h*w*(c + c*ab/8 + 8*co) bytes in multiples of 256
    c, co, ab, h, w = 64, 52, 4, 64, 64                     # 64 + 32 + 8 * 52 = 512 bytes per pixel: 16 images = 32 MiB
    d = ebs.conv_desc(c, co, 1, 1, 1, 1, 0, 0, 3, ab, 0.05, 0.05)
    per_image = ebs.ebs_host_workspace_bytes(d, 1, h, w, ebs.EBS_U8_CODES, 0)
    assert limit % per_image == 0, "the case was chosen to fill the scratch exactly"
    n = limit // per_image
    assert ebs.ebs_host_workspace_bytes(d, n, h, w, ebs.EBS_U8_CODES, 0) == limit
    rng = np.random.default_rng(7)
    qa = rng.integers(0, 1 << ab, size=(n, h, w, c), dtype=np.int32).astype(np.uint8)
    qw = rng.integers(-4, 4, size=(co, c, 1, 1), dtype=np.int32).astype(np.int8)
    pw = torch.empty(ebs.ebs_packed_weight_bytes(d) // 4, dtype=torch.int32, device=dev)
    ebs.ebs_pack_weights(torch.from_numpy(qw).to(dev), ebs.EBS_I8_CODES, ebs.EBS_NCHW, d, pw)
    x_host = torch.from_numpy(qa).pin_memory()
    acc = torch.zeros((n, h, w, co), dtype=torch.int32).pin_memory()
    ebs.ebs_conv2d_mixed_host_noalloc(x_host, ebs.EBS_U8_CODES, ebs.EBS_NHWC, n, h, w, pw, d, None, acc, None, None)
    torch.cuda.synchronize()
    ref = qa.reshape(-1, c).astype(np.int64) @ qw.reshape(co, c).astype(np.int64).T       # a 1x1 layer is a matrix product
    assert np.array_equal(acc.numpy().reshape(-1, co), ref)
    with pytest.raises(ebs.EbsError) as err:
        ebs.ebs_conv2d_mixed_host_noalloc(x_host, ebs.EBS_U8_CODES, ebs.EBS_NHWC, n + 1, h, w, pw, d, None, acc, None, None)
    assert err.value.status == ebs.EBS_ERR_SCRATCH_TOO_SMALL
    # a bad epilogue (packed output asked for with a non-positive step) is refused before any copy is enqueued:
    # the accumulators of the good call above are still what the host buffer holds afterwards
    pn = torch.zeros(ebs.ebs_packed_act_bytes(1, h, w, co, 2) // 4, dtype=torch.int32).pin_memory()
    bad = ebs.epilogue(relu=True, next_a_bits=2, next_a_scale=-1.0)
    keep = acc.numpy().copy()
    with pytest.raises(ebs.EbsError) as err:
        ebs.ebs_conv2d_mixed_host_noalloc(x_host, ebs.EBS_U8_CODES, ebs.EBS_NHWC, 1, h, w, pw, d, bad, acc, None, pn)
    assert err.value.status == ebs.EBS_ERR_INVALID_ARG
    torch.cuda.synchronize()
    assert np.array_equal(acc.numpy(), keep)
