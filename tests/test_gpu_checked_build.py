"""The range-checked build of the library (libebs_checked.so, -DEBS_CHECKED): the kernel parity tests pass on it with
an empty record, and its record works.  It stands in for a memory checker: every index the kernels compute from the
run-time geometry is tested before the access, a violation is recorded and the access skipped (nothing traps)."""
import os
import subprocess
import sys

import pytest
import torch

pytestmark = pytest.mark.gpu

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

RECORD_SCRIPT = r"""
import os, sys
import numpy as np
sys.path.insert(0, {root!r})
from paper_2003_07577_b200 import binding as ebs
from tests import _util as U
assert ebs.ebs_checked_build()
rng = np.random.default_rng(3)
cases = [("mma", 16, 16, 8), ("umma_pipe", 64, 64, 24), ("popc", 16, 16, 8)]
for family, c_in, c_out, hw in cases:
    qa = U.rand_codes(rng, (2, c_in, hw, hw), 3, False)
    qw = U.rand_codes(rng, (c_out, c_in, 3, 3), 2, True)
    d = U.desc_for(c_in, c_out, 3, 1, 1, 2, 3)
    vs = [v for v in U.variants_of(family) if U.applies(d, hw, hw, v, n=2)]
    assert vs, family
    assert ebs.ebs_checked_status(clear=True)[0] is False
    total = 2 * hw * hw * c_out
    ebs.ebs_test_checked_shrink(1)                       # the last accumulator now counts as out of range
    try:
        U.run_conv(qa, qw, d, variant=vs[0])
    finally:
        ebs.ebs_test_checked_shrink(0)
    recorded, site, index, limit = ebs.ebs_checked_status(clear=True)
    assert recorded and limit == total - 1 and index >= limit, (family, recorded, site, index, limit)
    assert site & 0xf in (2, 3), hex(site)               # an accumulator store of that kernel family
    U.run_conv(qa, qw, d, variant=vs[0])                 # true extents again: nothing recorded
    assert ebs.ebs_checked_status(clear=True)[0] is False
print("record ok")
"""


@pytest.fixture(scope="module")
def checked_library():
    if not torch.cuda.is_available():
        pytest.skip("needs a CUDA device")
    import importlib
    b = importlib.import_module("paper_2003_07577_b200.build")
    if not os.path.exists(b.LIB_CHECKED):
        b.build(checked=True)
    return b.LIB_CHECKED


def run_checked(args, timeout):
    env = dict(os.environ, EBS_LIBRARY="checked")
    return subprocess.run([sys.executable] + args, capture_output=True, text=True, env=env, cwd=ROOT, timeout=timeout)


def test_the_gpu_suite_passes_on_the_range_checked_library(checked_library):
    """Every GPU test of the repository (all kernel families and variants, odd sizes, strides, paddings, shortcut forms,
    the full-size configurations, the whole-network runs, the host calls) on the checked library: results identical to
    the oracle and, after every test, an empty record (tests/conftest.py checks it when EBS_LIBRARY=checked)."""
    res = run_checked(["-m", "pytest", "-x", "-q", "-m", "gpu", "tests", "--deselect", "tests/test_gpu_checked_build.py",
                       "-p", "no:cacheprovider"], timeout=1800)
    assert res.returncode == 0, res.stdout[-3000:] + res.stderr[-2000:]


def test_the_record_reports_a_refused_store(checked_library, tmp_path):
    """Result extents declared one element short (a test hook of the checked library): the kernels refuse the store of
    the last element, record site, index and limit, and finish; with the true extents nothing is recorded."""
    script = tmp_path / "record.py"
    script.write_text(RECORD_SCRIPT.format(root=ROOT))
    res = run_checked([str(script)], timeout=600)
    assert res.returncode == 0 and "record ok" in res.stdout, res.stdout[-3000:] + res.stderr[-3000:]


def test_the_normal_library_has_no_checks():
    from paper_2003_07577_b200 import binding as ebs
    if os.environ.get("EBS_LIBRARY") == "checked":
        pytest.skip("this process runs the checked library")
    assert not ebs.ebs_checked_build()
    with pytest.raises(ebs.EbsError):
        ebs.ebs_checked_status()
