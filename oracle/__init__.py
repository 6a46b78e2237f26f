"""CPU oracle for the binary-decomposition mixed-precision convolution.

TEST INFRASTRUCTURE ONLY: tests, the smoke check and the benchmark's CPU legs may
import this package; the product package never does, and this package never
imports the product.  It wraps ``ebs_oracle.c`` (plain C, built with gcc) through
ctypes and adds ``bd_matrices`` -- the paper's matrix form (Eq. 12-15) in numpy.

All tensors are numpy arrays in the paper's order: activations ``[N, C, H, W]``,
weights ``[C_out, C_in, kh, kw]``, one int32 per code.
"""
from __future__ import annotations

import ctypes
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "ebs_oracle.c")
_LIB = os.path.join(_HERE, "libebs_oracle.so")
_lib = None

OK, ERR_ARG, ERR_OVERFLOW = 0, -1, -3


def build(force: bool = False) -> str:
    """Compile the C oracle (gcc, -O2, OpenMP, no FMA contraction)."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        cmd = ["gcc", "-O2", "-std=c11", "-fopenmp", "-ffp-contract=off", "-fno-fast-math", "-shared",
               "-fPIC", "-o", _LIB, _SRC, "-lm"]
        subprocess.run(cmd, check=True)
    return _LIB


def _load():
    global _lib
    if _lib is None:
        build()
        lib = ctypes.CDLL(_LIB)
        i, f, p, z = ctypes.c_int, ctypes.c_float, ctypes.c_void_p, ctypes.c_size_t
        lib.oracle_num_threads.restype = i
        lib.oracle_out_dim.argtypes = [i, i, i, i]
        lib.oracle_out_dim.restype = i
        lib.oracle_quantize.argtypes = [p, z, f, i, i, p]
        lib.oracle_quantize.restype = None
        lib.oracle_conv2d_codes.argtypes = [p, p] + [i] * 11 + [p]
        lib.oracle_conv2d_codes.restype = i
        lib.oracle_conv2d_levels.argtypes = [p, p] + [i] * 11 + [p]
        lib.oracle_conv2d_levels.restype = i
        lib.oracle_quantize_weight_levels.argtypes = [p, z, f, i, p]
        lib.oracle_quantize_weight_levels.restype = None
        lib.oracle_conv2d_bitplanes.argtypes = [p, p] + [i] * 14 + [p]
        lib.oracle_conv2d_bitplanes.restype = i
        lib.oracle_epilogue.argtypes = [p, i, i, i, i, f, p, p, p, i, p, i, f, p]
        lib.oracle_epilogue.restype = None
        lib.oracle_pack_acts.argtypes = [p, i, i, i, i, i, p]
        lib.oracle_pack_acts.restype = None
        lib.oracle_pack_weights.argtypes = [p, i, i, i, i, i, p]
        lib.oracle_pack_weights.restype = None
        lib.oracle_unpack_acts.argtypes = [p, i, i, i, i, i, p]
        lib.oracle_unpack_acts.restype = None
        _lib = lib
    return _lib


def _ptr(a):
    return None if a is None else a.ctypes.data_as(ctypes.c_void_p)


def _i32(a):
    return np.ascontiguousarray(a, dtype=np.int32)


def _f32(a):
    return None if a is None else np.ascontiguousarray(a, dtype=np.float32)


def num_threads() -> int:
    return int(_load().oracle_num_threads())


def out_dim(size: int, pad: int, k: int, stride: int) -> int:
    return int(_load().oracle_out_dim(size, pad, k, stride))


def quantize(x, inv_step: float, lo: int, hi: int) -> np.ndarray:
    """Eq. 1c as integer codes: clamp(floor(fl32(x*inv_step) + 0.5), lo, hi)."""
    x = _f32(x)
    q = np.empty(x.shape, dtype=np.int32)
    _load().oracle_quantize(_ptr(x), x.size, np.float32(inv_step), lo, hi, _ptr(q))
    return q


def quantize_acts(x, a_scale: float, a_bits: int) -> np.ndarray:
    """Eq. 1b: codes in [0, 2^b - 1]; a_scale = alpha / (2^b - 1)."""
    inv = np.float32(1.0) / np.float32(a_scale)
    return quantize(x, inv, 0, (1 << a_bits) - 1)


def quantize_weights(w, w_scale: float, w_bits: int) -> np.ndarray:
    """Signed two's-complement codes in [-2^(b-1), 2^(b-1) - 1]."""
    inv = np.float32(1.0) / np.float32(w_scale)
    return quantize(w, inv, -(1 << (w_bits - 1)), (1 << (w_bits - 1)) - 1)


def conv2d_codes(qa, qw, stride=(1, 1), pad=(0, 0)) -> np.ndarray:
    """Direct integer convolution (the definition). Returns int32 [N, Co, Ho, Wo]."""
    qa, qw = _i32(qa), _i32(qw)
    n, c, h, w = qa.shape
    co, c2, kh, kw = qw.shape
    assert c == c2
    ho, wo = out_dim(h, pad[0], kh, stride[0]), out_dim(w, pad[1], kw, stride[1])
    acc = np.empty((n, co, ho, wo), dtype=np.int32)
    rc = _load().oracle_conv2d_codes(_ptr(qa), _ptr(qw), n, c, h, w, co, kh, kw, stride[0], stride[1],
                                     pad[0], pad[1], _ptr(acc))
    if rc == ERR_OVERFLOW:
        raise OverflowError("accumulator does not fit int32")
    if rc != OK:
        raise ValueError(f"oracle_conv2d_codes: bad arguments ({rc})")
    return acc


def conv2d_levels(qa, qw, stride=(1, 1), pad=(0, 0)) -> np.ndarray:
    """Convolution with the paper's weight levels 2*qw + 1 (Eq. 1a), qw the signed code q_u - 2^(b-1)."""
    qa, qw = _i32(qa), _i32(qw)
    n, c, h, w = qa.shape
    co, c2, kh, kw = qw.shape
    assert c == c2
    ho, wo = out_dim(h, pad[0], kh, stride[0]), out_dim(w, pad[1], kw, stride[1])
    acc = np.empty((n, co, ho, wo), dtype=np.int32)
    rc = _load().oracle_conv2d_levels(_ptr(qa), _ptr(qw), n, c, h, w, co, kh, kw, stride[0], stride[1],
                                      pad[0], pad[1], _ptr(acc))
    if rc == ERR_OVERFLOW:
        raise OverflowError("accumulator does not fit int32")
    if rc != OK:
        raise ValueError(f"oracle_conv2d_levels: bad arguments ({rc})")
    return acc


def quantize_weight_levels(w, w_scale: float, w_bits: int) -> np.ndarray:
    """Eq. 1a: nearest of the levels w_scale*(2 q_u - (2^b-1)); returns the signed code q_u - 2^(b-1)."""
    w = _f32(w)
    q = np.empty(w.shape, dtype=np.int32)
    inv = np.float32(1.0) / np.float32(w_scale)
    _load().oracle_quantize_weight_levels(_ptr(w), w.size, inv, w_bits, _ptr(q))
    return q


def conv2d_bitplanes(qa, qw, w_bits, a_bits, stride=(1, 1), pad=(0, 0), signed_w=True) -> np.ndarray:
    """Eq. 2 evaluated bit by bit (no packing), with the signed top weight plane."""
    qa, qw = _i32(qa), _i32(qw)
    n, c, h, w = qa.shape
    co, _, kh, kw = qw.shape
    ho, wo = out_dim(h, pad[0], kh, stride[0]), out_dim(w, pad[1], kw, stride[1])
    acc = np.empty((n, co, ho, wo), dtype=np.int32)
    rc = _load().oracle_conv2d_bitplanes(_ptr(qa), _ptr(qw), n, c, h, w, co, kh, kw, stride[0], stride[1],
                                         pad[0], pad[1], w_bits, a_bits, int(bool(signed_w)), _ptr(acc))
    if rc != OK:
        raise ValueError(f"oracle_conv2d_bitplanes: bad arguments ({rc})")
    return acc


def combined_scale(w_scale: float, a_scale: float) -> np.float32:
    """S = fl32(s_w * s_a), rounded once."""
    return np.float32(np.float32(w_scale) * np.float32(a_scale))


def epilogue(acc, S, ch_scale=None, ch_bias=None, residual=None, relu=False, next_bits=0, inv_next=0.0):
    """fp32 epilogue on [N, Co, Ho, Wo] accumulators. Returns (y, q) (q is None if next_bits == 0)."""
    acc = _i32(acc)
    n, co, ho, wo = acc.shape
    ch_scale, ch_bias, residual = _f32(ch_scale), _f32(ch_bias), _f32(residual)
    y = np.empty(acc.shape, dtype=np.float32)
    q = np.empty(acc.shape, dtype=np.int32) if next_bits else None
    _load().oracle_epilogue(_ptr(acc), n, co, ho, wo, np.float32(S), _ptr(ch_scale), _ptr(ch_bias),
                            _ptr(residual), int(bool(relu)), _ptr(y), max(int(next_bits), 1),
                            np.float32(inv_next), _ptr(q))
    return y, q


def dequant_codes(q, step) -> np.ndarray:
    """The value a code stands for: fl32(step * code) (Eq. 1b's second line, one fp32 product)."""
    return (np.float32(step) * np.asarray(q).astype(np.float32)).astype(np.float32)


def global_avgpool(y) -> np.ndarray:
    """Average over the pixels of [N, C, H, W] fp32 values, as the ResNets of Sec. 5 do before the
    classifier: pixels are added one by one in row-major order in fp32, then multiplied by fl32(1/HW)."""
    y = np.asarray(y, dtype=np.float32)
    n, c, h, w = y.shape
    acc = np.zeros((n, c), dtype=np.float32)
    for i in range(h):
        for j in range(w):
            acc = (acc + y[:, :, i, j]).astype(np.float32)
    return (acc * (np.float32(1.0) / np.float32(h * w))).astype(np.float32)


def maxpool_codes(q, k: int, stride: int, pad: int) -> np.ndarray:
    """Max pooling of unsigned activation codes [N, C, H, W] (the 3x3 stride-2 pooling between the first convolution and
    the first block of the ImageNet ResNets the paper evaluates, Sec. 5).  Codes of one tensor share one step, so the
    maximum of the real values is the maximum of the codes; window positions outside the image are ignored, which for
    codes (all >= 0, the image of a clipped activation) is the same as padding with the zero code.  Plain loops over the
    window; output size floor((size + 2 pad - k) / stride) + 1."""
    q = np.asarray(q)
    n, c, h, w = q.shape
    ho, wo = out_dim(h, pad, k, stride), out_dim(w, pad, k, stride)
    out = np.zeros((n, c, ho, wo), dtype=q.dtype)
    for i in range(ho):
        for j in range(wo):
            best = None
            for r in range(k):
                for s in range(k):
                    hi, wi = i * stride + r - pad, j * stride + s - pad
                    if 0 <= hi < h and 0 <= wi < w:
                        v = q[:, :, hi, wi]
                        best = v.copy() if best is None else np.maximum(best, v)
            if best is not None:
                out[:, :, i, j] = best
    return out


# ---------------------------------------------------------------- search stage (Sec. 4.1), plain numpy

def softmax_strengths(r) -> np.ndarray:
    """Coefficients of the deterministic search: softmax of the strengths (Eq. 5-6), evaluated in
    float64 and rounded to the fp32 values both sides are given."""
    r = np.asarray(r, dtype=np.float64)
    e = np.exp(r - r.max())
    return (e / e.sum()).astype(np.float32)


def quantize_unit(u, bits: int) -> np.ndarray:
    """quantize_b of Eq. 1c on fp32 values in [0, 1]: (1 / (2^b - 1)) * floor((2^b - 1) u + 0.5), the
    reciprocal rounded to fp32 once, every operation rounded to fp32 on its own (round half up)."""
    u = np.asarray(u, dtype=np.float32)
    L = np.float32((1 << bits) - 1)
    code = np.floor((u * L).astype(np.float32) + np.float32(0.5)).astype(np.float32)
    return ((np.float32(1.0) / L) * code).astype(np.float32)


def search_act_forward(x, alpha, bits, coeff) -> np.ndarray:
    """Eq. 1b per candidate bitwidth, blended as in Eq. 7:
    x_hat = alpha * sum_j coeff_j * quantize_{b_j}(clip(x, 0, alpha) * (1/alpha)), fp32, the reciprocal
    rounded once, candidates in order."""
    x = np.asarray(x, dtype=np.float32)
    a = np.float32(alpha)
    u = (np.minimum(np.maximum(x, np.float32(0.0)), a) * (np.float32(1.0) / a)).astype(np.float32)
    acc = np.zeros_like(u)
    for b, c in zip(bits, coeff):
        acc = (acc + (np.float32(c) * quantize_unit(u, int(b))).astype(np.float32)).astype(np.float32)
    return (a * acc).astype(np.float32)


def search_weight_forward(w, bits, coeff, per_candidate: bool = False):
    """Eq. 1a per candidate bitwidth, blended as in Eq. 6, in float64:
    u = tanh(w) / (2 max|tanh(w)|) + 1/2;  w_hat = sum_i coeff_i * (2 quantize_{b_i}(u) - 1).
    Also returns, per element, the smallest distance of (2^b - 1) u + 0.5 to an integer over the
    candidates: where it is tiny, a float32 evaluation may legitimately round to the other level.
    per_candidate = True returns the distances of every candidate instead ([len(bits), ...])."""
    w = np.asarray(w, dtype=np.float64)
    t = np.tanh(w)
    u = t / (2.0 * np.abs(t).max()) + 0.5
    out = np.zeros_like(u)
    margin = np.full(u.shape, 1.0)
    each = []
    for b, c in zip(bits, coeff):
        L = float((1 << int(b)) - 1)
        v = L * u + 0.5
        code = np.clip(np.floor(v), 0.0, L)
        each.append(np.abs(v - np.round(v)))
        margin = np.minimum(margin, each[-1])
        out += float(c) * (2.0 * code / L - 1.0)
    return out, (np.stack(each) if per_candidate else margin)


def expected_flops(macs, bits_w, coeff_w, bits_x, coeff_x) -> float:
    """Eq. 11: FLOP(sum_i f(r)_i b_i, sum_j f(s)_j b_j) with FLOP(M, K) = macs * M * K (Sec. 4.3)."""
    m = sum(float(c) * int(b) for b, c in zip(bits_w, coeff_w))
    k = sum(float(c) * int(b) for b, c in zip(bits_x, coeff_x))
    return float(macs) * m * k


def pack_acts(qa, a_bits: int) -> np.ndarray:
    """uint32 [N, H, W, ceil(C/32), Ab] bit-plane words, built bit by bit."""
    qa = _i32(qa)
    n, c, h, w = qa.shape
    out = np.empty((n, h, w, (c + 31) // 32, a_bits), dtype=np.uint32)
    _load().oracle_pack_acts(_ptr(qa), n, c, h, w, a_bits, _ptr(out))
    return out


def pack_weights(qw, w_bits: int) -> np.ndarray:
    """uint32 [kh, kw, ceil(C/32), Co, Wb] bit-plane words of two's-complement codes."""
    qw = _i32(qw)
    co, c, kh, kw = qw.shape
    out = np.empty((kh, kw, (c + 31) // 32, co, w_bits), dtype=np.uint32)
    _load().oracle_pack_weights(_ptr(qw), co, c, kh, kw, w_bits, _ptr(out))
    return out


def unpack_acts(packed, c: int) -> np.ndarray:
    """Inverse of pack_acts: int32 codes [N, C, H, W]."""
    packed = np.ascontiguousarray(packed, dtype=np.uint32)
    n, h, w, cw, ab = packed.shape
    assert cw == (c + 31) // 32
    qa = np.empty((n, c, h, w), dtype=np.int32)
    _load().oracle_unpack_acts(_ptr(packed), n, c, h, w, ab, _ptr(qa))
    return qa


def lambda_w(c_o: int, w_bits: int, signed_w: bool = True) -> np.ndarray:
    """Eq. 15: Lambda_w = diag(delta_w, ..., delta_w), shape (c_o, c_o*M), delta_w = [2^0 .. 2^(M-1)].

    With signed_w the last entry of delta_w is -2^(M-1) (two's-complement weights).
    """
    delta = np.array([1 << m for m in range(w_bits)], dtype=np.int64)
    if signed_w:
        delta[w_bits - 1] = -delta[w_bits - 1]
    L = np.zeros((c_o, c_o * w_bits), dtype=np.int64)
    for i in range(c_o):
        L[i, i * w_bits:(i + 1) * w_bits] = delta
    return L


def lambda_x_t(n: int, a_bits: int) -> np.ndarray:
    """Lambda_x^T of shape (n*K, n): block column j holds delta_x = [2^0 .. 2^(K-1)]."""
    delta = np.array([1 << k for k in range(a_bits)], dtype=np.int64)
    L = np.zeros((n * a_bits, n), dtype=np.int64)
    for j in range(n):
        L[j * a_bits:(j + 1) * a_bits, j] = delta
    return L


def bd_matrices(qa, qw, w_bits, a_bits, stride=(1, 1), pad=(0, 0), signed_w=True):
    """The paper's two-stage matrix form, for tiny shapes only.

    img2col (Sec. 4.3): W_hat is (c_o x s), X_hat is (s x n) with s = c_i*kh*kw and n
    the number of output pixels (of every image, side by side).  Eq. 12 / Eq. 15:
    W_hat = Lambda_w B_w with B_w in {0,1}^(c_o*M x s), rows ordered output channel
    major, plane minor; X_hat = B_x Lambda_x^T with B_x in {0,1}^(s x n*K), columns
    pixel major, plane minor.  Stage 1 (Eq. 13): P = B_w B_x, AND + bitcount only.
    Stage 2 (Eq. 14): a (M x K) kernel delta_w^T delta_x of powers of two applied
    with stride (M, K).  With signed_w the top entry of delta_w is -2^(M-1).

    Returns (O as int64 [N, Co, Ho, Wo], P, B_w, B_x).
    """
    qa = np.asarray(qa, dtype=np.int64)
    qw = np.asarray(qw, dtype=np.int64)
    n_img, c, h, w = qa.shape
    co, _, kh, kw = qw.shape
    ho, wo = out_dim(h, pad[0], kh, stride[0]), out_dim(w, pad[1], kw, stride[1])
    s = c * kh * kw
    n = n_img * ho * wo
    # img2col
    W_hat = qw.reshape(co, s)
    X_hat = np.zeros((s, n), dtype=np.int64)
    col = 0
    for b in range(n_img):
        for y in range(ho):
            for x in range(wo):
                row = 0
                for ci in range(c):
                    for r in range(kh):
                        for t in range(kw):
                            yy, xx = y * stride[0] + r - pad[0], x * stride[1] + t - pad[1]
                            if 0 <= yy < h and 0 <= xx < w:
                                X_hat[row, col] = qa[b, ci, yy, xx]
                            row += 1
                col += 1
    # binary expansion
    M, K = w_bits, a_bits
    B_w = np.zeros((co * M, s), dtype=np.uint8)
    for i in range(co):
        for m in range(M):
            B_w[i * M + m] = (W_hat[i] >> m) & 1          # two's complement bits for negatives
    B_x = np.zeros((s, n * K), dtype=np.uint8)
    for j in range(n):
        for k in range(K):
            B_x[:, j * K + k] = (X_hat[:, j] >> k) & 1
    # stage 1: AND + bitcount
    P = np.zeros((co * M, n * K), dtype=np.int64)
    for r in range(co * M):
        for q in range(n * K):
            P[r, q] = int(np.count_nonzero(B_w[r] & B_x[:, q]))
    # stage 2: power-of-two (M x K) kernel with stride (M, K)
    delta_w = np.array([1 << m for m in range(M)], dtype=np.int64)
    if signed_w:
        delta_w[M - 1] = -delta_w[M - 1]
    delta_x = np.array([1 << k for k in range(K)], dtype=np.int64)
    kernel = np.outer(delta_w, delta_x)
    O = np.zeros((co, n), dtype=np.int64)
    for i in range(co):
        for j in range(n):
            O[i, j] = int((P[i * M:(i + 1) * M, j * K:(j + 1) * K] * kernel).sum())
    # the same thing as the literal matrix product of Eq. 13
    O_literal = lambda_w(co, M, signed_w) @ P @ lambda_x_t(n, K)
    assert np.array_equal(O, O_literal), "strided power-of-two kernel disagrees with Lambda_w P Lambda_x^T"
    O = O.reshape(co, n_img, ho, wo).transpose(1, 0, 2, 3).copy()
    return O, P, B_w, B_x
