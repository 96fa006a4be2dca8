import os
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


def pytest_configure(config):
    config.addinivalue_line("markers", "gpu: needs a CUDA device (run on the B200 box)")


@pytest.fixture(scope="session", autouse=True)
def _build_host_helpers():
    """Compile the CPU-side helpers (oracle, input generator) once per session."""
    import oracle
    from paper_2609_13031_b200 import workloads
    oracle.build()
    workloads.build()
