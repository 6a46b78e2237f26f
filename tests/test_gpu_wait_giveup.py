"""The give-up path of the bounded device-side waits (collected after the other kernel tests: it raises the
library's give-up counter, which those tests expect to be zero)."""
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


@pytest.mark.parametrize("form", ["single", "pair"])
def test_pipe_bounded_waits_give_up_and_recover(ebs, U, oracle, form):
    """The give-up path, made to run on purpose without faulting anything: with the wait limit at a few polls and the
    issuing thread told to issue no tensor-core work, every wait for the tensor core runs out with nothing in flight;
    each thread block raises its abort flag, leaves its loops, frees its tensor memory and returns.  The counter rises,
    ebs_check_device_status reports EBS_ERR_TIMEOUT once, and the next healthy launch is bit-exact."""
    rng = np.random.default_rng(5)
    qa = U.rand_codes(rng, (4, 64, 12, 12), 3, False)
    co = 64 if form == "single" else 256                      # the pair of CTAs works on whole 256-channel tiles
    qw = U.rand_codes(rng, (co, 64, 3, 3), 2, True)
    d = U.desc_for(64, co, 3, 1, 1, 2, 3)
    ref = oracle.conv2d_codes(qa, qw, (1, 1), (1, 1))
    variant = U.variants_of("umma_pipe")[0 if form == "single" else -1]
    assert U.applies(d, 12, 12, variant, n=4)
    assert ebs.ebs_check_device_status() == ebs.EBS_OK
    before = ebs.ebs_device_wait_timeouts()
    ebs.ebs_test_set_device_wait(64, True)
    try:
        U.run_conv(qa, qw, d, variant=variant)              # returns: every wait is bounded
    finally:
        ebs.ebs_test_set_device_wait(0, False)
    after = ebs.ebs_device_wait_timeouts()
    assert after > before, "no thread block reported that it gave up"
    assert ebs.ebs_check_device_status() == ebs.EBS_ERR_TIMEOUT
    assert ebs.ebs_check_device_status() == ebs.EBS_OK        # reported once
    got = U.run_conv(qa, qw, d, variant=variant)["acc"]       # the context is healthy: same launch, exact result
    assert np.array_equal(got, ref)
    assert ebs.ebs_device_wait_timeouts() == after
