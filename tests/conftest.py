import sys
from pathlib import Path

import pytest

ROOT = Path(__file__).resolve().parent.parent
if str(ROOT) not in sys.path:
    sys.path.insert(0, str(ROOT))


def pytest_configure(config):
    config.addinivalue_line("markers", "gpu: needs a CUDA device (run on a B200 box)")


@pytest.fixture(scope="session")
def tiny_weights():
    from paper_2604_12247_b200 import inputs
    run = inputs.RUNS["tiny"]
    return inputs.make_weights(run.shape, run.seed)


@pytest.fixture(scope="session")
def tiny_damped_weights():
    from paper_2604_12247_b200 import inputs
    run = inputs.RUNS["tiny-damped"]
    return inputs.make_weights(run.shape, run.seed, damp_rho=run.damp_rho)
