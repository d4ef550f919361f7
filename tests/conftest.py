import os
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


def pytest_configure(config):
    config.addinivalue_line("markers", "gpu: needs a CUDA device (run with -m gpu on a B200)")


@pytest.fixture(scope="session", autouse=True)
def built_libraries():
    """Both shared libraries are compiled before any test runs (a no-op when they are up to date): the CUDA
    library needs only nvcc, not a GPU."""
    from paper_2608_18183_b200 import build
    from oracle import oracle as O
    build.build()
    O.build()


_cache = {}


def cached(key, fn):
    if key not in _cache:
        _cache[key] = fn()
    return _cache[key]


@pytest.fixture(scope="session")
def tiny():
    """(workload, weight image) of the tiny fp32 configuration."""
    from paper_2608_18183_b200 import synth
    w = synth.WORKLOADS["tiny"]
    return w, cached(("w", "tiny"), lambda: synth.make_weights(w.shape, w.weight_seed))


@pytest.fixture(scope="session")
def tiny_bf16():
    from paper_2608_18183_b200 import synth
    w = synth.WORKLOADS["tiny_bf16"]
    return w, cached(("w", "tiny_bf16"), lambda: synth.make_weights(w.shape, w.weight_seed))
