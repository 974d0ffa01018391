import os
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


def pytest_configure(config):
    config.addinivalue_line("markers", "gpu: needs a CUDA device (runs the C-ABI CUDA path)")


@pytest.fixture(scope="session")
def tiny_cfg():
    """Configuration 0 (tiny fp32 instance): weights and inputs."""
    from paper_2605_18817_b200 import synth
    cfg = synth.CONFIGS[0]
    w, inp = synth.make_config(cfg)
    return cfg, w, inp
