import os
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


def pytest_configure(config):
    config.addinivalue_line("markers", "gpu: needs a CUDA device (B200, sm_100a)")


@pytest.fixture(scope="session")
def cfg0_inputs():
    import pc_inputs
    cfg = pc_inputs.get_config("cfg0")
    return cfg, pc_inputs.make_prefill_inputs(cfg)


@pytest.fixture(scope="session")
def cfg0_oracle(cfg0_inputs):
    """Full oracle pass over the tiny gate configuration (seconds)."""
    from oracle import parallelcomp_oracle as orc
    cfg, inp = cfg0_inputs
    return orc.hot_path(inp["q"], inp["k"], inp["v"], w=cfg.w, theta=cfg.rope_theta, m=cfg.m, k=cfg.k)
