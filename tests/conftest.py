import os
import sys

import numpy as np
import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


def pytest_configure(config):
    config.addinivalue_line("markers", "gpu: needs a CUDA device (run with -m gpu on a B200)")


def to_np(t):
    """torch tensor -> numpy; bf16 becomes its uint16 bit pattern (the oracle widens it)."""
    import torch
    t = t.detach().cpu()
    if t.dtype == torch.bfloat16:
        return t.contiguous().view(torch.int16).numpy().view(np.uint16)
    return t.numpy()


def weights_np(w):
    return {k: to_np(v) for k, v in w.items()}


@pytest.fixture(scope="session")
def rng():
    return np.random.default_rng(12345)
