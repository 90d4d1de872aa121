import os
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


def pytest_configure(config):
    config.addinivalue_line("markers", "gpu: needs a CUDA device (run with -m gpu on a B200)")


@pytest.fixture(scope="session")
def golden_dir():
    return os.path.join(ROOT, "tests", "golden")


@pytest.fixture(autouse=True)
def output_guard_bands(request):
    """After every GPU test: no kernel may have written outside a tensor the binding allocated for it (4 KiB
    bands of 0xA5 on both sides of every output; the accepted stand-in for a memory checker on this pool)."""
    yield
    if request.node.get_closest_marker("gpu") is None:
        return
    import sys
    binding = sys.modules.get("paper_2011_10680_b200.binding")
    if binding is not None:
        binding.check_guards()
