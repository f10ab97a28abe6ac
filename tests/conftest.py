import os
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


def pytest_configure(config):
    config.addinivalue_line("markers", "gpu: needs a CUDA device (run on the B200 box)")


@pytest.fixture(scope="session")
def tiny_f32():
    """Small fp32 model with GQA and QK-norm, non-unit norm gains."""
    from s2d2_inputs import generate_weights, get_config
    wl = get_config("t_f32")
    return wl, generate_weights(wl.model, seed=3, gain_jitter=0.2)


@pytest.fixture(scope="session")
def tiny_moe():
    from s2d2_inputs import generate_weights, get_config
    wl = get_config("t_moe", model_n_layers=1, model_vocab=64)
    return wl, generate_weights(wl.model, seed=5, gain_jitter=0.2)
