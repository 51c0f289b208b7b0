import os
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


def pytest_configure(config):
    config.addinivalue_line("markers", "gpu: needs a CUDA device (run with -m gpu on a B200)")
    # The CUDA library is loaded when the test modules are imported, i.e. during collection: build it
    # before that (a no-op when it is up to date; an nvcc build, which needs no GPU, otherwise).
    from paper_2407_13726_b200 import build as cuda_build

    cuda_build.build()


@pytest.fixture(scope="session", autouse=True)
def _built_cpu_libs():
    """The generator and the oracle are small gcc builds; make sure they exist."""
    import oracle
    import synth

    synth.build()
    oracle.build()
