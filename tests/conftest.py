import os
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


def pytest_configure(config):
    config.addinivalue_line("markers", "gpu: needs a CUDA device (run on a B200)")


@pytest.fixture(scope="session")
def oracle():
    from oracle import flare_oracle
    flare_oracle.build()
    return flare_oracle


def pytest_collection_modifyitems(config, items):
    import torch
    if torch.cuda.is_available():
        return
    skip = pytest.mark.skip(reason="no CUDA device")
    for item in items:
        if "gpu" in item.keywords:
            item.add_marker(skip)


def pytest_sessionfinish(session, exitstatus):
    """Write which bound every stored-tensor comparison met (see tests/_util.py) where FLARE_PARITY_REPORT names a file."""
    path = os.environ.get("FLARE_PARITY_REPORT")
    if not path:
        return
    from tests import _util
    with open(path, "w") as f:
        for what, bound, plain, excess in _util.BOUND_LOG:
            f.write(f"{what}\t{bound}\t{plain:.3e}\t{'' if excess is None else format(excess, '.3e')}\n")
