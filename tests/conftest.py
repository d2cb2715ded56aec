import os
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


def pytest_configure(config):
    config.addinivalue_line("markers", "gpu: needs a CUDA device (B200); run with -m gpu")


@pytest.fixture(scope="session", autouse=True)
def _build_native():
    """Compile the CPU-side helpers (oracle, input generator) and, if nvcc is present and the
    library is stale, the CUDA library, so that a fresh checkout can run the suite directly."""
    import oracle
    import synth_inputs
    oracle.build()
    synth_inputs.build()
    from paper_2405_05254_b200 import build as pkg_build
    if pkg_build._sources():
        pkg_build.build_cuda_library()
    yield
