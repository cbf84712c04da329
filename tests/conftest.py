import os
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


def pytest_configure(config):
    config.addinivalue_line("markers", "gpu: needs a CUDA device (run on a B200)")
    config.addinivalue_line("markers", "slow: long-running")


@pytest.fixture(scope="session")
def small_cfg():
    """A GQA decoder small enough for fp64 brute force, with non-unit norm gains."""
    import synth
    return synth.ModelConfig("small", n_blocks=4, d_model=64, n_heads=4, n_kv_heads=2, head_dim=16,
                             ffn=96, vocab=97, dtype="f32", seed=11, n_planted=2, init_std=0.2,
                             gain_std=0.1)


@pytest.fixture(scope="session")
def small_weights(small_cfg):
    import synth
    return synth.make_weights(small_cfg)
