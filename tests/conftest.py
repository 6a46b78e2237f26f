import os
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


def pytest_configure(config):
    config.addinivalue_line("markers", "gpu: needs a CUDA device (run on a B200)")
    config.addinivalue_line("markers", "expects_range_record: the test makes the range-checked library record on purpose")


@pytest.fixture(scope="session")
def oracle():
    import oracle as _oracle
    _oracle.build()
    return _oracle


@pytest.fixture(autouse=True)
def _range_checked_library_stays_clean(request):
    """When the suite runs on the range-checked library (EBS_LIBRARY=checked), every GPU test must leave its
    record empty: no kernel computed an index outside the buffer or shared-memory region it belongs to."""
    yield
    if os.environ.get("EBS_LIBRARY") != "checked" or request.node.get_closest_marker("gpu") is None:
        return
    if request.node.get_closest_marker("expects_range_record") is not None:
        return
    from paper_2003_07577_b200 import binding as ebs
    recorded, site, index, limit = ebs.ebs_checked_status(clear=True)
    assert not recorded, f"range check: site 0x{site:x} index {index} limit {limit}"
