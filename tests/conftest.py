import os
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


def pytest_configure(config):
    config.addinivalue_line("markers", "gpu: needs a CUDA device (B200); skipped by -m 'not gpu'")


@pytest.fixture(scope="session")
def c1_inputs():
    from paper_2609_29812_b200 import workloads
    return workloads.make_layer_inputs(workloads.config1(), seed=0)
