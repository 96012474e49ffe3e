import os
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


def pytest_configure(config):
    config.addinivalue_line("markers", "gpu: needs a CUDA device (runs on the B200 box)")


@pytest.fixture(scope="session")
def repo_root():
    return ROOT


@pytest.fixture(scope="session")
def oracle_workers():
    """Worker processes that run the oracle on every host core (full-size parity checks)."""
    from oracle.parallel import OracleWorkers
    pool = OracleWorkers(min(os.cpu_count() or 1, 16), extra_sys_path=[os.path.join(ROOT, "tests")])
    yield pool
    pool.close()
