"""Pins for the CPU oracle: every check here is something other than the oracle itself.

Brute force in pure Python, the paper's printed coefficient matrix (Eq. 12), hand-derived
binary matrices, numpy int64 matmul, a float64 library convolution, closed forms and
bit-flip linearity.  A dropped term, wrong sign, wrong index or transposed operand in the
oracle fails at least one of them.
"""
import itertools
import os

import numpy as np
import pytest
import torch

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def rand_codes(rng, shape, bits, signed):
    if signed:
        return rng.integers(-(1 << (bits - 1)), (1 << (bits - 1)), size=shape, dtype=np.int32)
    return rng.integers(0, 1 << bits, size=shape, dtype=np.int32)


def brute_conv(qa, qw, stride, pad):
    """Seven nested Python loops over plain ints."""
    n_, c_, h_, w_ = qa.shape
    co_, _, kh, kw = qw.shape
    ho = (h_ + 2 * pad[0] - kh) // stride[0] + 1
    wo = (w_ + 2 * pad[1] - kw) // stride[1] + 1
    out = np.zeros((n_, co_, ho, wo), dtype=np.int64)
    A, Wt = qa.tolist(), qw.tolist()
    for n in range(n_):
        for co in range(co_):
            for y in range(ho):
                for x in range(wo):
                    tot = 0
                    for ci in range(c_):
                        for r in range(kh):
                            for s in range(kw):
                                yy, xx = y * stride[0] + r - pad[0], x * stride[1] + s - pad[1]
                                if 0 <= yy < h_ and 0 <= xx < w_:
                                    tot += A[n][ci][yy][xx] * Wt[co][ci][r][s]
                    out[n, co, y, x] = tot
    return out


@pytest.mark.parametrize("k,stride,pad", [(3, 1, 1), (3, 2, 1), (1, 1, 0), (1, 2, 0), (3, 1, 0), (5, 2, 2),
                                          (7, 2, 3), (2, 1, 1)])
def test_direct_conv_equals_brute_force(oracle, k, stride, pad):
    rng = np.random.default_rng(k * 100 + stride * 10 + pad)
    qa = rand_codes(rng, (2, 5, 7, 6), 3, False)
    qw = rand_codes(rng, (4, 5, k, k), 4, True)
    got = oracle.conv2d_codes(qa, qw, (stride, stride), (pad, pad))
    assert np.array_equal(got, brute_conv(qa, qw, (stride, stride), (pad, pad)))


def test_direct_conv_asymmetric_stride_pad(oracle):
    rng = np.random.default_rng(5)
    qa = rand_codes(rng, (1, 3, 9, 8), 2, False)
    qw = rand_codes(rng, (2, 3, 3, 3), 2, True)
    got = oracle.conv2d_codes(qa, qw, (2, 1), (0, 1))
    assert np.array_equal(got, brute_conv(qa, qw, (2, 1), (0, 1)))


@pytest.mark.parametrize("wb,ab", list(itertools.product([1, 2, 3, 5, 8], [1, 2, 4, 8])))
def test_bitplane_identity_signed(oracle, wb, ab):
    """Eq. 2 with the two's-complement top plane weighted -2^(Wb-1) equals the integer dot product."""
    rng = np.random.default_rng(wb * 16 + ab)
    qa = rand_codes(rng, (1, 6, 5, 5), ab, False)
    qw = rand_codes(rng, (3, 6, 3, 3), wb, True)
    ref = oracle.conv2d_codes(qa, qw, (1, 1), (1, 1))
    assert np.array_equal(oracle.conv2d_bitplanes(qa, qw, wb, ab, (1, 1), (1, 1), signed_w=True), ref)


def test_bitplane_identity_unsigned_is_the_papers_eq2(oracle):
    rng = np.random.default_rng(3)
    qa = rand_codes(rng, (1, 4, 4, 4), 3, False)
    qw = rand_codes(rng, (2, 4, 3, 3), 2, False)          # unsigned codes, all plane weights positive
    ref = brute_conv(qa, qw, (1, 1), (0, 0))
    assert np.array_equal(oracle.conv2d_bitplanes(qa, qw, 2, 3, signed_w=False), ref)
    # and reading signed codes as unsigned must NOT give the signed result (the sign matters)
    qws = rand_codes(rng, (2, 4, 3, 3), 2, True)
    assert not np.array_equal(oracle.conv2d_bitplanes(qa, qws, 2, 3, signed_w=False),
                              brute_conv(qa, qws, (1, 1), (0, 0)))


def test_lambda_w_matches_eq12_print(oracle):
    golden = np.loadtxt(os.path.join(GOLDEN, "eq12_lambda_w.txt"), dtype=np.int64)
    assert np.array_equal(oracle.lambda_w(2, 2, signed_w=False), golden)
    signed = golden.copy()
    signed[signed == 2] = -2
    assert np.array_equal(oracle.lambda_w(2, 2, signed_w=True), signed)


def test_bd_binary_matrix_order_by_hand(oracle):
    """Eq. 12's row order: (channel, plane) with the plane index minor; hand-expanded example."""
    qw = np.array([[1, 2, 3], [0, 3, 1]], dtype=np.int32).reshape(2, 3, 1, 1)      # 2x3 weight matrix
    qa = np.array([[5, 2], [7, 0], [1, 6]], dtype=np.int32).reshape(1, 3, 1, 2)    # 3x2 activation matrix
    O, P, B_w, B_x = oracle.bd_matrices(qa, qw, 2, 3, signed_w=False)
    assert B_w.tolist() == [[1, 0, 1], [0, 1, 1], [0, 1, 1], [0, 1, 0]]
    # columns (pixel, plane): pixel 0 = (5,7,1) -> bit0 (1,1,1) bit1 (0,1,0) bit2 (1,1,0); pixel 1 = (2,0,6)
    assert B_x.T.tolist() == [[1, 1, 1], [0, 1, 0], [1, 1, 0], [0, 0, 0], [1, 0, 1], [0, 0, 1]]
    assert P.shape == (4, 6)
    assert O.reshape(2, 2).tolist() == [[1 * 5 + 2 * 7 + 3 * 1, 1 * 2 + 0 + 3 * 6], [0 + 3 * 7 + 1, 0 + 0 + 6]]


@pytest.mark.parametrize("wb,ab,stride,pad", [(2, 2, 1, 1), (3, 1, 2, 1), (1, 3, 1, 0), (4, 2, 2, 0)])
def test_bd_matrix_route_equals_direct(oracle, wb, ab, stride, pad):
    rng = np.random.default_rng(wb * 7 + ab)
    qa = rand_codes(rng, (2, 3, 5, 4), ab, False)
    qw = rand_codes(rng, (3, 3, 3, 3), wb, True)
    O, P, _, _ = oracle.bd_matrices(qa, qw, wb, ab, (stride, stride), (pad, pad), signed_w=True)
    assert P.min() >= 0 and P.max() <= 3 * 9
    assert np.array_equal(O, oracle.conv2d_codes(qa, qw, (stride, stride), (pad, pad)))


def test_1x1_conv_is_integer_matmul(oracle):
    rng = np.random.default_rng(11)
    qa = rand_codes(rng, (2, 70, 6, 5), 4, False)
    qw = rand_codes(rng, (9, 70, 1, 1), 5, True)
    got = oracle.conv2d_codes(qa, qw)
    X = qa.transpose(0, 2, 3, 1).reshape(-1, 70).astype(np.int64)
    ref = (X @ qw.reshape(9, 70).astype(np.int64).T).reshape(2, 6, 5, 9).transpose(0, 3, 1, 2)
    assert np.array_equal(got, ref)


@pytest.mark.parametrize("k,stride,pad,c,co", [(3, 1, 1, 40, 12), (3, 2, 1, 33, 8), (7, 2, 3, 3, 16),
                                               (1, 2, 0, 64, 20)])
def test_against_float64_library_conv(oracle, k, stride, pad, c, co):
    """An independent library routine: exact in float64 because |acc| << 2^53."""
    rng = np.random.default_rng(c + co)
    qa = rand_codes(rng, (2, c, 13, 11), 8, False)
    qw = rand_codes(rng, (co, c, k, k), 8, True)
    ref = torch.nn.functional.conv2d(torch.from_numpy(qa).double(), torch.from_numpy(qw).double(),
                                     stride=stride, padding=pad).numpy()
    got = oracle.conv2d_codes(qa, qw, (stride, stride), (pad, pad))
    assert np.array_equal(got.astype(np.float64), ref)


@pytest.mark.parametrize("ab", [1, 2, 4, 8])
def test_closed_form_taps(oracle, ab):
    """All activations 2^Ab-1, all weights -1: acc = -(2^Ab-1) * C * (taps inside the image)."""
    c, h = 7, 6
    qa = np.full((1, c, h, h), (1 << ab) - 1, dtype=np.int32)
    qw = np.full((2, c, 3, 3), -1, dtype=np.int32)
    acc = oracle.conv2d_codes(qa, qw, (1, 1), (1, 1))
    unit = -((1 << ab) - 1) * c
    assert acc[0, 0, 0, 0] == 4 * unit and acc[0, 1, 0, h - 1] == 4 * unit       # corners
    assert acc[0, 0, 0, 2] == 6 * unit and acc[0, 0, 3, 0] == 6 * unit           # edges
    assert acc[0, 1, 2, 3] == 9 * unit                                           # interior
    assert np.array_equal(oracle.conv2d_bitplanes(qa, qw, 3, ab, (1, 1), (1, 1)), acc)


def test_closed_form_w1a1_is_minus_popcount(oracle):
    rng = np.random.default_rng(2)
    qa = rand_codes(rng, (1, 50, 1, 1), 1, False)
    qw = rand_codes(rng, (4, 50, 1, 1), 1, True)           # codes in {-1, 0}
    acc = oracle.conv2d_codes(qa, qw)
    for co in range(4):
        assert acc[0, co, 0, 0] == -int(np.count_nonzero(qa[0, :, 0, 0] & (qw[co, :, 0, 0] & 1)))


def test_bit_flip_linearity(oracle):
    """Flipping weight bit m at one position changes acc by c_m * 2^m * (activation there)."""
    rng = np.random.default_rng(9)
    wb, ab = 4, 3
    qa = rand_codes(rng, (1, 3, 4, 4), ab, False)
    qw = rand_codes(rng, (2, 3, 3, 3), wb, True)
    base = oracle.conv2d_codes(qa, qw, (1, 1), (0, 0)).astype(np.int64)
    for m in range(wb):
        u = (qw[1, 2, 0, 1] & ((1 << wb) - 1)) ^ (1 << m)                     # flip bit m of the 4-bit pattern
        q2 = qw.copy()
        q2[1, 2, 0, 1] = u - (1 << wb) if u >= (1 << (wb - 1)) else u
        delta = oracle.conv2d_codes(qa, q2, (1, 1), (0, 0)).astype(np.int64) - base
        bit_was_set = (qw[1, 2, 0, 1] >> m) & 1
        coef = -(1 << m) if m == wb - 1 else (1 << m)
        sign = -1 if bit_was_set else 1
        expect = np.zeros_like(base)
        expect[0, 1] = sign * coef * qa[0, 2, 0:2, 1:3]
        assert np.array_equal(delta, expect)


def test_overflow_is_reported(oracle):
    qa = np.full((1, 70000, 1, 1), 255, dtype=np.int32)
    qw = np.full((1, 70000, 1, 1), -128, dtype=np.int32)
    with pytest.raises(OverflowError):
        oracle.conv2d_codes(qa, qw)


# ---------------------------------------------------------------- quantizer (Eq. 1b, 1c)

def test_quantize_round_half_up(oracle):
    step = 0.25                                              # power of two: x/step is exact
    x = np.array([0.0, 0.124, 0.125, 0.126, 0.375, 0.625, 10.0, -0.3, -0.125, -0.375, -0.376], np.float32)
    q = oracle.quantize(x, 1.0 / step, -8, 7)
    #           0   0      .5->1  1     1.5->2 2.5->3  clamp  -1.2->-1  -.5->0  -1.5->-1  -1.504->-2
    assert q.tolist() == [0, 0, 1, 1, 2, 3, 7, -1, 0, -1, -2]
    assert oracle.quantize_acts(x, step, 2).tolist() == [0, 0, 1, 1, 2, 3, 3, 0, 0, 0, 0]


def test_quantize_matches_float64_away_from_ties(oracle):
    rng = np.random.default_rng(4)
    x = rng.uniform(-1, 5, size=4000).astype(np.float32)
    scale = np.float32(0.0371)
    v = x.astype(np.float64) / np.float64(scale)
    safe = np.abs(v - np.floor(v) - 0.5) > 1e-3
    ref = np.clip(np.floor(v + 0.5), 0, 15).astype(np.int32)
    got = oracle.quantize_acts(x, scale, 4)
    assert safe.sum() > 3900 and np.array_equal(got[safe], ref[safe])
    refw = np.clip(np.floor(v + 0.5), -4, 3).astype(np.int32)
    assert np.array_equal(oracle.quantize_weights(x, scale, 3)[safe], refw[safe])


def test_quantize_then_dequantize_is_eq1b(oracle):
    """alpha * quantize_b(clip(x,0,alpha)/alpha) with alpha = (2^b-1)*step, exact for power-of-two steps."""
    b, step = 3, 0.5
    alpha = ((1 << b) - 1) * step
    x = np.linspace(-1.0, 5.0, 97, dtype=np.float32)
    xt = np.clip(x.astype(np.float64), 0, alpha) / alpha
    ref = alpha * np.floor(((1 << b) - 1) * xt + 0.5) / ((1 << b) - 1)
    got = oracle.quantize_acts(x, step, b).astype(np.float64) * step
    assert np.array_equal(got, ref)


# ---------------------------------------------------------------- epilogue

def test_epilogue_exact_with_power_of_two_scales(oracle):
    rng = np.random.default_rng(6)
    acc = rng.integers(-5000, 5000, size=(2, 3, 4, 5), dtype=np.int32)
    S = np.float32(2.0 ** -7)
    y, q = oracle.epilogue(acc, S, relu=True, next_bits=3, inv_next=np.float32(0.25))
    ref_y = np.maximum(acc.astype(np.float64) * 2.0 ** -7, 0.0)
    assert np.array_equal(y.astype(np.float64), ref_y)
    assert np.array_equal(q, np.clip(np.floor(ref_y * 0.25 + 0.5), 0, 7).astype(np.int32))
    y2, _ = oracle.epilogue(acc, S, relu=False)
    assert np.array_equal(y2.astype(np.float64), acc.astype(np.float64) * 2.0 ** -7)


def test_epilogue_affine_order_and_tolerance(oracle):
    rng = np.random.default_rng(8)
    acc = rng.integers(-20000, 20000, size=(1, 4, 3, 3), dtype=np.int32)
    S = oracle.combined_scale(0.037, 0.052)
    assert S == np.float32(np.float32(0.037) * np.float32(0.052))
    cs = rng.uniform(0.5, 2, 4).astype(np.float32)
    cb = rng.uniform(-1, 1, 4).astype(np.float32)
    res = rng.uniform(-1, 1, acc.shape).astype(np.float32)
    y, _ = oracle.epilogue(acc, S, cs, cb, res, relu=False)
    ref = (acc.astype(np.float64) * np.float64(S)) * cs[None, :, None, None].astype(np.float64) \
        + cb[None, :, None, None] + res
    assert np.allclose(y, ref, rtol=1e-6, atol=1e-6)
    # each step rounded on its own, in this order
    step = (acc.astype(np.float32) * S)
    step = step * cs[None, :, None, None]
    step = step + cb[None, :, None, None]
    step = step + res
    assert np.array_equal(y, step)
    # a swapped scale/bias order would be far outside rounding error
    wrong = (acc.astype(np.float64) * np.float64(S) + cb[None, :, None, None]) * cs[None, :, None, None] + res
    assert not np.allclose(y, wrong, rtol=1e-3, atol=1e-3)


# ---------------------------------------------------------------- packing

def test_pack_words_by_hand(oracle):
    qa = np.zeros((1, 40, 1, 2), dtype=np.int32)
    qa[0, 0, 0, 0] = 1            # channel 0, plane 0
    qa[0, 33, 0, 0] = 2           # channel 33 -> word 1 bit 1, plane 1
    qa[0, 31, 0, 1] = 3           # channel 31 -> word 0 bit 31, planes 0 and 1
    p = oracle.pack_acts(qa, 2)
    assert p.shape == (1, 1, 2, 2, 2)
    assert p[0, 0, 0].tolist() == [[1, 0], [0, 2]]
    assert p[0, 0, 1].tolist() == [[1 << 31, 1 << 31], [0, 0]]
    qw = np.zeros((3, 40, 1, 2), dtype=np.int32)
    qw[2, 5, 0, 1] = -1           # two's complement 0b11 at 2 bits
    qw[1, 39, 0, 0] = -2          # 0b10
    pw = oracle.pack_weights(qw, 2)
    assert pw.shape == (1, 2, 2, 3, 2)
    assert pw[0, 1, 0, 2].tolist() == [1 << 5, 1 << 5]
    assert pw[0, 0, 1, 1].tolist() == [0, 1 << 7]
    assert int(pw.astype(np.uint64).sum()) == 2 * (1 << 5) + (1 << 7)


@pytest.mark.parametrize("c,ab", [(3, 8), (16, 2), (32, 1), (48, 3), (70, 4)])
def test_pack_roundtrip_and_zero_pad_bits(oracle, c, ab):
    rng = np.random.default_rng(c)
    qa = rand_codes(rng, (2, c, 3, 4), ab, False)
    p = oracle.pack_acts(qa, ab)
    assert np.array_equal(oracle.unpack_acts(p, c), qa)
    if c % 32:
        assert not np.any(p[:, :, :, -1, :] >> np.uint32(c % 32))


def test_packed_dot_equals_conv(oracle):
    """popcount(AND) over the packed words with plane weights reproduces the accumulator."""
    rng = np.random.default_rng(21)
    wb, ab, c = 3, 2, 45
    qa = rand_codes(rng, (1, c, 1, 1), ab, False)
    qw = rand_codes(rng, (2, c, 1, 1), wb, True)
    pa, pw = oracle.pack_acts(qa, ab), oracle.pack_weights(qw, wb)
    acc = oracle.conv2d_codes(qa, qw)
    for co in range(2):
        tot = 0
        for cw in range(2):
            for m in range(wb):
                for k in range(ab):
                    cnt = bin(int(pa[0, 0, 0, cw, k]) & int(pw[0, 0, cw, co, m])).count("1")
                    tot += (-1 if m == wb - 1 else 1) * (1 << (m + k)) * cnt
        assert tot == acc[0, co, 0, 0]


# ---------------------------------------------------------------- workload shapes

def test_layer_lists_reproduce_printed_mac_totals():
    from workloads import nets
    nets_by_name = {"resnet20_cifar": nets.resnet_cifar(3), "resnet32_cifar": nets.resnet_cifar(5),
                    "resnet56_cifar": nets.resnet_cifar(9), "resnet18_imagenet": nets.resnet18_imagenet()}
    with open(os.path.join(GOLDEN, "table_macs.txt")) as f:
        rows = [ln.split() for ln in f if ln.strip() and not ln.startswith("#")]
    assert len(rows) == 4
    for name, value, tol, *_ in rows:
        assert abs(nets.total_macs(nets_by_name[name]) - float(value)) <= float(tol), name
    r50 = [L for L in nets.resnet50_imagenet() if L.quantized]
    assert len(r50) == 52 and abs(nets.total_macs(r50) - 3.969e9) < 0.002e9


def test_generators_are_seeded_and_in_range():
    from workloads import gen
    a, b = gen.config2(0), gen.config2(0)
    assert [(s.w_bits, s.a_bits) for s in a] == [(s.w_bits, s.a_bits) for s in b]
    assert [(s.w_bits, s.a_bits) for s in a] != [(s.w_bits, s.a_bits) for s in gen.config2(1)]
    assert (a[0].w_bits, a[0].a_bits) == (8, 8) and (a[-1].w_bits, a[-1].a_bits) == (8, 8)
    assert sum(s.layer.quantized for s in a) == 20
    for s in gen.config3(0)[:3]:
        qw, qa = gen.weight_codes(s), gen.act_codes(s, batch=1, h_in=8)
        assert qw.min() >= -(1 << (s.w_bits - 1)) and qw.max() <= (1 << (s.w_bits - 1)) - 1
        assert qa.min() >= 0 and qa.max() <= (1 << s.a_bits) - 1
        assert np.array_equal(qw, gen.weight_codes(s))
    c1 = gen.config1()[0]
    assert (c1.w_bits, c1.a_bits, c1.batch) == (2, 2, 1) and 0.01 <= c1.w_scale <= 0.1


# ---------------------------------------------------------------- the paper's own weight levels (Eq. 1a)

def test_levels_conv_equals_brute_force_and_the_unsigned_bitplane_route(oracle):
    rng = np.random.default_rng(41)
    wb, ab = 3, 2
    L = (1 << wb) - 1
    qa = rand_codes(rng, (2, 5, 6, 5), ab, False)
    qs = rand_codes(rng, (3, 5, 3, 3), wb, True)                 # signed code = q_u - 2^(b-1)
    qu = qs + (1 << (wb - 1))                                    # the paper's unsigned level index
    levels = 2 * qu - L                                          # Eq. 1a numerator: 2*round(L x) - L
    assert levels.min() >= -L and levels.max() <= L and np.all(levels % 2 != 0) and np.array_equal(levels, 2 * qs + 1)
    got = oracle.conv2d_levels(qa, qs, (1, 1), (1, 1))
    assert np.array_equal(got, brute_conv(qa, levels, (1, 1), (1, 1)))
    # Eq. 2 with the paper's unsigned codes: sum (2 q_u - L) a = 2 * bitplane_sum(q_u, a) - L * window_sum(a)
    ones = np.ones_like(qs)
    window = brute_conv(qa, ones, (1, 1), (1, 1))
    unsigned_route = 2 * oracle.conv2d_bitplanes(qa, qu, wb, ab, (1, 1), (1, 1), signed_w=False).astype(np.int64) - L * window
    assert np.array_equal(got, unsigned_route)
    # and the form the GPU uses: 2 * (signed bit-plane sum) + window sum
    assert np.array_equal(got, 2 * oracle.conv2d_codes(qa, qs, (1, 1), (1, 1)).astype(np.int64) + window)


def test_weight_level_quantizer_is_eq1a(oracle):
    """q_u = round_half_up(L * (w_n/2 + 1/2)) for normalised weights w_n in [-1, 1], step 1/L."""
    for b in (1, 2, 3, 4, 8):
        L = (1 << b) - 1
        wn = np.linspace(-1.2, 1.2, 481).astype(np.float32)
        x = L * (wn.astype(np.float64) / 2 + 0.5)
        safe = np.abs(x - np.floor(x) - 0.5) > 1e-4
        ref_qu = np.clip(np.floor(x + 0.5), 0, L).astype(np.int32)
        got = oracle.quantize_weight_levels(wn, 1.0 / L, b) + (1 << (b - 1))
        assert np.array_equal(got[safe], ref_qu[safe]), b
        hat = (2 * got - L) / L                                  # the de-quantized weight of Eq. 1a
        assert hat.min() == -1.0 and hat.max() == 1.0
    # exact ties with a power-of-two step go up
    q = oracle.quantize_weight_levels(np.array([0.0, -2.0, 2.0, -0.5, 100.0, -100.0], np.float32), 1.0, 2)
    #   v=0: (0+3)/2=1.5 -> 2 ; v=-2: 0.5 -> 1 ; v=2: 2.5 -> 3 ; v=-.5: 1.25 -> 1 ; clamp 3 ; clamp 0     (q_u)
    assert (q + 2).tolist() == [2, 1, 3, 1, 3, 0]


def test_global_avgpool_pins(oracle):
    """Exact where the mathematics fixes it (integers with a power-of-two pixel count, constants);
    within fp32 summation error of the float64 mean elsewhere; order of axes checked by a ramp."""
    rng = np.random.default_rng(5)
    yi = rng.integers(-100, 100, size=(3, 5, 8, 8)).astype(np.float32)
    assert np.array_equal(oracle.global_avgpool(yi), yi.astype(np.float64).mean(axis=(2, 3)).astype(np.float32))
    y = rng.standard_normal((2, 7, 6, 5)).astype(np.float32)
    ref = y.astype(np.float64).mean(axis=(2, 3))
    got = oracle.global_avgpool(y)
    assert got.dtype == np.float32 and got.shape == (2, 7)
    assert np.allclose(got, ref, rtol=0, atol=30 * 2.0 ** -24 * np.abs(y).sum(axis=(2, 3)).max() / 30)
    ramp = np.zeros((2, 3, 4, 4), np.float32)
    ramp[1, 2] = 16.0
    assert np.array_equal(oracle.global_avgpool(ramp), np.array([[0, 0, 0], [0, 0, 16]], np.float32))


def test_dequant_codes_is_one_fp32_product(oracle):
    q = np.arange(0, 256)
    step = np.float32(0.0371)
    got = oracle.dequant_codes(q, step)
    assert got.dtype == np.float32
    assert np.array_equal(got, np.array([np.float32(float(step) * int(v)) for v in q], np.float32))


# ------------------------------------------------------------------ search stage (Eq. 1a-c, 6, 7, 11)

def test_quantize_unit_levels_half_up_and_idempotent(oracle):
    for b in (1, 2, 3, 5, 8):
        L = (1 << b) - 1
        grid = (np.arange(L + 1, dtype=np.float32) * (np.float32(1.0) / np.float32(L))).astype(np.float32)
        assert np.array_equal(oracle.quantize_unit(grid, b), grid)                   # levels are fixed points
        u = np.linspace(0, 1, 4001, dtype=np.float32)
        q = oracle.quantize_unit(u, b)
        assert np.all(np.diff(q) >= 0) and set(np.unique(q)) <= set(grid)             # monotone, on the grid
        assert np.all(np.abs(q.astype(np.float64) - u) <= 0.5 / L + 1e-6)              # nearest level
    assert oracle.quantize_unit(np.float32(0.5), 1) == 1.0                            # the tie goes up
    assert oracle.quantize_unit(np.float32(0.25), 2) == np.float32(1.0) / np.float32(3.0)   # 0.75 + 0.5 -> floor 1
    assert oracle.quantize_unit(np.float32(1.0), 3) == np.float32(7.0) * (np.float32(1.0) / np.float32(7.0))


def test_softmax_strengths_closed_forms(oracle):
    assert np.allclose(oracle.softmax_strengths([0, 0]), [0.5, 0.5])                  # the text's two-candidate example
    p = oracle.softmax_strengths([-1, 1])
    assert np.allclose(p, [1 / (1 + np.e ** 2), np.e ** 2 / (1 + np.e ** 2)], atol=1e-7) and p[1] > 0.88
    assert np.allclose(oracle.softmax_strengths(np.zeros(5)), 0.2) and oracle.softmax_strengths([3, 3, 3]).dtype == np.float32


def test_search_act_forward_special_cases(oracle):
    rng = np.random.default_rng(3)
    x = rng.uniform(-1, 8, 5000).astype(np.float32)
    alpha = 6.0
    one = oracle.search_act_forward(x, alpha, [3], [1.0])                             # one candidate: plain Eq. 1b
    ref = alpha * np.round(np.clip(x.astype(np.float64), 0, alpha) / alpha * 7 + 1e-12) / 7
    assert np.allclose(one, ref, atol=1e-5) and one.min() == 0 and one.max() == np.float32(alpha)
    assert set(np.unique(np.round(one / alpha * 7).astype(int))) == set(range(8))
    two = oracle.search_act_forward(x, alpha, [2, 3], [0.5, 0.5])                     # equal blend of two bitwidths
    a2, a3 = oracle.search_act_forward(x, alpha, [2], [1.0]), oracle.search_act_forward(x, alpha, [3], [1.0])
    assert np.allclose(two, 0.5 * a2.astype(np.float64) + 0.5 * a3, atol=1e-6)
    sharp = oracle.search_act_forward(x, alpha, [2, 3], [0.0, 1.0])                   # softmax -> max selects one branch
    assert np.array_equal(sharp, a3)


def test_search_weight_forward_special_cases(oracle):
    rng = np.random.default_rng(4)
    w = rng.standard_normal(4000) * 0.7
    for b in (1, 2, 4):
        L = (1 << b) - 1
        out, _ = oracle.search_weight_forward(w, [b], [1.0])
        lv = np.unique(np.round((out + 1) * L / 2).astype(int))
        assert np.allclose((out + 1) * L / 2, np.round((out + 1) * L / 2), atol=1e-9)   # on the level grid of [-1, 1]
        assert lv.min() == 0 and lv.max() == L and np.abs(out).max() == 1.0            # the largest weight maps to +-1
    out1, _ = oracle.search_weight_forward(w, [1], [1.0])
    assert np.array_equal(out1, np.where(w >= 0, 1.0, -1.0))                          # one bit: the sign
    out8, _ = oracle.search_weight_forward(w, [8], [1.0])
    assert np.abs(out8 - np.tanh(w) / np.abs(np.tanh(w)).max()).max() <= 1.0 / 255 + 1e-12   # fine grid: the normalized tanh
    blend, margin = oracle.search_weight_forward(w, [2, 3], [0.5, 0.5])
    o2, _ = oracle.search_weight_forward(w, [2], [1.0])
    o3, _ = oracle.search_weight_forward(w, [3], [1.0])
    assert np.allclose(blend, 0.5 * o2 + 0.5 * o3) and np.unique(np.round(blend, 9)).size > 4 and (margin >= 0).all()


def test_expected_flops_eq11(oracle):
    bits = [1, 2, 3, 4, 5]
    uniform = oracle.softmax_strengths(np.zeros(5))
    assert abs(oracle.expected_flops(1e6, bits, uniform, bits, uniform) - 9e6) < 1.0   # mean bitwidth 3 on both sides
    onehot = [0, 0, 1, 0, 0]
    assert oracle.expected_flops(40.81e6, bits, onehot, bits, [0, 1, 0, 0, 0]) == 40.81e6 * 3 * 2


def test_maxpool_codes_pins(oracle):
    """Max pooling of codes: brute force per output on a tiny tensor, the identity window, a hand-written case with
    padding, and the library routine torch.nn.functional.max_pool2d (which pads with -inf: the same thing for codes)."""
    import torch
    rng = np.random.default_rng(5)
    q = rng.integers(0, 16, size=(2, 3, 7, 6), dtype=np.int32)
    for k, s, p in ((3, 2, 1), (2, 2, 0), (3, 1, 1), (1, 1, 0), (3, 2, 0)):
        got = oracle.maxpool_codes(q, k, s, p)
        ho, wo = (7 + 2 * p - k) // s + 1, (6 + 2 * p - k) // s + 1
        assert got.shape == (2, 3, ho, wo)
        for n in range(2):
            for c in range(3):
                for i in range(ho):
                    for j in range(wo):
                        vals = [q[n, c, i * s + r - p, j * s + t - p] for r in range(k) for t in range(k)
                                if 0 <= i * s + r - p < 7 and 0 <= j * s + t - p < 6]
                        assert got[n, c, i, j] == max(vals)
        ref = torch.nn.functional.max_pool2d(torch.from_numpy(q.astype(np.float64)), k, s, p).numpy()
        assert np.array_equal(got, ref.astype(np.int32))
    assert np.array_equal(oracle.maxpool_codes(q, 1, 1, 0), q)
    one = np.array([[[[1, 5], [7, 2]]]], np.int32)
    assert np.array_equal(oracle.maxpool_codes(one, 3, 2, 1), np.array([[[[7]]]], np.int32))      # one window sees all
    assert np.array_equal(oracle.maxpool_codes(one, 2, 1, 1), np.array([[[[1, 5, 5], [7, 7, 5], [7, 7, 2]]]], np.int32))



@pytest.mark.parametrize("c,k,pad,h,w", [(3, 7, 3, 12, 10), (3, 5, 2, 8, 8), (2, 3, 1, 6, 8), (4, 3, 0, 8, 6), (1, 7, 2, 10, 10)])
def test_stride2_first_layer_equals_its_space_to_depth_form(oracle, c, k, pad, h, w):
    """A k x k stride-2 convolution equals the ceil(k/2)-square stride-1 convolution over 2 x 2 pixel blocks with the
    weights regrouped the same way (the form the network runner gives an ImageNet stem): both evaluated by the oracle's
    direct definition.  The block layout is written out here; the weight regrouping is the runner's own function."""
    import torch
    from paper_2003_07577_b200.network import space_to_depth_weights
    rng = np.random.default_rng(k * 10 + pad)
    x = rng.integers(0, 256, size=(2, c, h, w), dtype=np.int32)
    wt = rng.integers(-128, 128, size=(5, c, k, k), dtype=np.int32)
    ref = oracle.conv2d_codes(x, wt, (2, 2), (pad, pad))
    off, pb = pad & 1, (pad - (pad & 1)) // 2
    hs, ws = (h + off) // 2 + off, (w + off) // 2 + off
    xs = np.zeros((2, 4 * c, hs, ws), dtype=np.int32)
    for dy in (0, 1):
        for dx in (0, 1):
            for i in range(hs):
                for j in range(ws):
                    hh, ww = 2 * i - off + dy, 2 * j - off + dx
                    if 0 <= hh < h and 0 <= ww < w:
                        xs[:, (2 * dy + dx) * c:(2 * dy + dx + 1) * c, i, j] = x[:, :, hh, ww]
    w2 = space_to_depth_weights(torch.from_numpy(wt)).numpy()
    assert w2.shape == (5, 4 * c, (k + 1) // 2, (k + 1) // 2)
    got = oracle.conv2d_codes(xs, w2, (1, 1), (pb, pb))
    assert got.shape == ref.shape and np.array_equal(got, ref)
