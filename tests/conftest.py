import os
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


def pytest_configure(config):
    config.addinivalue_line("markers", "gpu: needs a CUDA device (run with -m gpu on a B200)")


@pytest.fixture(scope="session", autouse=True)
def _built_cpu_libs():
    """The generator and the oracle are small gcc builds, the library an nvcc build; make sure they exist."""
    import oracle
    import synth

    synth.build()
    oracle.build()
    # the CUDA library: a no-op when it is up to date, an nvcc build (no GPU needed) when it is missing or stale
    from paper_2407_13726_b200 import build as cuda_build

    cuda_build.build()
