import sys
from pathlib import Path

import pytest

ROOT = Path(__file__).resolve().parent.parent
if str(ROOT) not in sys.path:
    sys.path.insert(0, str(ROOT))


def pytest_configure(config):
    config.addinivalue_line("markers", "gpu: needs a CUDA device (run with -m gpu)")


@pytest.fixture(scope="session")
def oracle():
    import oracle as o
    o.build()
    return o


@pytest.fixture(scope="session")
def libdodo():
    """Path of the built CUDA library (compiled with nvcc if stale; needs no GPU)."""
    from paper_2310_02409_b200 import build
    return build.build()


@pytest.fixture(scope="session")
def dodo(libdodo):
    """A library context on cuda:0.  The CUDA library is the only implementation: no fallback."""
    import torch
    assert torch.cuda.is_available(), "GPU tests need a CUDA device"
    from paper_2310_02409_b200 import api
    ctx = api.Dodo(0)
    yield ctx
    assert ctx.device_status() == 0, "a kernel reported a device-side problem"
    ctx.close()


@pytest.fixture(scope="session")
def errlog():
    """The session's log of observed parity errors (see parity_log.py)."""
    import parity_log
    return parity_log.LOG


def pytest_sessionfinish(session, exitstatus):
    import parity_log
    parity_log.LOG.dump(ROOT / "gpurun_out" / "parity_errors.json")
