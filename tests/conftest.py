import os
import sys

import pytest

sys.path.insert(0, os.path.dirname(os.path.dirname(os.path.abspath(__file__))))


def pytest_configure(config):
    config.addinivalue_line("markers", "gpu: needs a CUDA device (sm_100a) and the built CUDA library")


@pytest.fixture(scope="session")
def oracle():
    from oracle import path_oracle

    path_oracle.build()
    return path_oracle
