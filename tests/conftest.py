import os
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


def pytest_configure(config):
    config.addinivalue_line("markers", "gpu: needs a CUDA device (B200)")


@pytest.fixture(scope="session")
def hat_lib():
    """Build (if stale) and load the CUDA library; a build failure fails the test."""
    from paper_2503_18989_b200 import build as hat_build
    from paper_2503_18989_b200 import binding
    # HAT_LIB=debug runs the suite against the build with device-side index checks
    hat_build.build(debug=os.environ.get("HAT_LIB") == "debug")
    return binding.lib()


@pytest.fixture(scope="session")
def cuda_device(hat_lib):
    import torch
    if not torch.cuda.is_available():
        pytest.fail("a test marked gpu ran without a CUDA device")
    return torch.device("cuda:0")
