import os
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


def pytest_configure(config):
    config.addinivalue_line("markers", "gpu: needs a CUDA device (run with -m gpu on a B200)")


@pytest.fixture(scope="session")
def tiny_case():
    """Config 1: fp32 (8,16,8,8), Batch Sampling k=2 of 8, seeded."""
    import bns_inputs as I
    N, C, H, W = 8, 16, 8, 8
    seed = 1810 + 1
    x = I.tiny_activations(N, C, H, W, seed)
    dy = I.upstream_gradient(x.shape, seed)
    gamma, beta = I.affine_parameters(C, seed)
    idx = I.batch_sample_indices(N, 2, seed, contiguous=False)
    return dict(N=N, C=C, H=H, W=W, x=x, dy=dy, gamma=gamma, beta=beta, eps=1e-5, idx=idx)
