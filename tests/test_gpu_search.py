"""GPU parity of the search-stage forward kernels (Eq. 6-7) against the numpy oracle."""
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


DEV = "cuda:0"
CANDS = [([3], [1.0]), ([2, 3], [0.5, 0.5]), ([1, 2, 3, 4, 5], None), ([1, 2, 3, 4, 5, 6, 7, 8], None)]


@pytest.mark.parametrize("n", [1, 3, 4097, (1 << 20) + 3])
@pytest.mark.parametrize("cand", range(len(CANDS)))
def test_search_act_forward_is_bit_exact(ebs, oracle, n, cand):
    bits, coeff = CANDS[cand]
    rng = np.random.default_rng(n + cand)
    if coeff is None:
        coeff = oracle.softmax_strengths(rng.standard_normal(len(bits)))
    x = rng.uniform(-2.0, 9.0, n).astype(np.float32)
    x[: min(n, 8)] = np.array([0.0, 6.0, 3.0, -0.0, 5.9999995, 1e-9, 7.0, 0.4285714], np.float32)[: min(n, 8)]
    alpha = 6.0
    xd = torch.from_numpy(x).to(DEV)
    out = torch.empty_like(xd)
    ebs.ebs_search_act_forward(xd, alpha, bits, coeff, out)
    ref = oracle.search_act_forward(x, alpha, bits, coeff)
    assert np.array_equal(out.cpu().numpy(), ref)
    ebs.ebs_search_act_forward(xd, alpha, bits, coeff, xd)                 # in place
    assert np.array_equal(xd.cpu().numpy(), ref)


@pytest.mark.parametrize("n", [5, 4099, (1 << 20) + 1])
@pytest.mark.parametrize("cand", range(len(CANDS)))
def test_search_weight_forward_matches_float64_oracle(ebs, oracle, n, cand):
    """fp32 on the GPU (tanhf) against float64: equal within 1e-5 away from rounding ties; at an element
    whose pre-rounding value is within 1e-4 of a tie the two may pick adjacent levels of one candidate."""
    bits, coeff = CANDS[cand]
    rng = np.random.default_rng(7 * n + cand)
    if coeff is None:
        coeff = oracle.softmax_strengths(rng.standard_normal(len(bits)))
    w = (rng.standard_normal(n) * 0.8).astype(np.float32)
    wd = torch.from_numpy(w).to(DEV)
    out = torch.empty_like(wd)
    scratch = torch.zeros(4, dtype=torch.int32, device=DEV)
    ebs.ebs_search_weight_forward(wd, bits, coeff, out, scratch)
    ref, margins = oracle.search_weight_forward(w, bits, coeff, per_candidate=True)
    got = out.cpu().numpy().astype(np.float64)
    near = margins <= 1e-4                                        # [candidate, element]: that candidate sits at a tie
    safe = ~near.any(axis=0)
    assert safe.mean() > 0.95
    assert np.abs(got[safe] - ref[safe]).max() <= 1e-5
    # at a tie one candidate may land on the adjacent level: one level step of that candidate, nothing more
    steps = np.array([2.0 * abs(float(c)) / ((1 << b) - 1) for b, c in zip(bits, coeff)])
    allowed = (near * steps[:, None]).sum(axis=0) + 1e-5
    assert (np.abs(got - ref) <= allowed).all()
    assert np.float32(scratch.view(torch.float32)[0].item()) == np.abs(w).max()     # the reduction found max|w|
    assert got.max() <= 1.0 + 1e-6 and got.min() >= -1.0 - 1e-6


def test_expected_flops_and_argument_checks(ebs, oracle):
    bits = [1, 2, 3, 4, 5]
    cw, cx = oracle.softmax_strengths([0.3, -1, 2, 0, 0.5]), oracle.softmax_strengths([0, 0, 1, 1, -2])
    assert abs(ebs.ebs_expected_flops(40.81e6, bits, cw, bits, cx) / oracle.expected_flops(40.81e6, bits, cw, bits, cx) - 1) < 1e-12
    x = torch.zeros(16, dtype=torch.float32, device=DEV)
    for bad_bits, bad_coeff in (([], []), ([0], [1.0]), ([17], [1.0]), (list(range(1, 10)), [0.1] * 9)):
        with pytest.raises(RuntimeError):
            ebs.ebs_search_act_forward(x, 6.0, bad_bits, bad_coeff, x)
    with pytest.raises(RuntimeError):
        ebs.ebs_search_act_forward(x, 0.0, [2], [1.0], x)
