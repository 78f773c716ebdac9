import os
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


def pytest_configure(config):
    config.addinivalue_line("markers", "gpu: needs a CUDA device (runs on the B200 box only)")
    config.addinivalue_line("markers", "slow: long-running oracle comparison")


@pytest.fixture(scope="session")
def tiny_weights():
    """Tiny fp32 draft / PRM / target weights (seed 0) as the oracle consumes them."""
    import rsd_inputs as ri
    d = ri.cpu_model_weights(ri.SHAPES["tiny_draft"], ri.SLOT_DRAFT, 0, False, ri.HEAD_LM)
    p = ri.cpu_model_weights(ri.SHAPES["tiny_draft"], ri.SLOT_PRM, 0, False, ri.HEAD_REWARD_SIGMOID)
    t = ri.cpu_model_weights(ri.SHAPES["tiny_target"], ri.SLOT_TARGET, 0, False, ri.HEAD_LM)
    return d, p, t
