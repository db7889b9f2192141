"""Shared fixtures.  GPU tests are marked ``gpu``; everything else runs on a CPU-only box."""
import os
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


def pytest_configure(config):
    config.addinivalue_line("markers", "gpu: needs a CUDA device (run with -m gpu)")


@pytest.fixture(scope="session")
def libs():
    """Both shared libraries compiled in-tree (nvcc cross-compiles without a GPU)."""
    from paper_2608_16491_b200 import build
    build.build_all()
    import paper_2608_16491_b200 as frog
    return frog


@pytest.fixture(scope="session")
def cache_dir(tmp_path_factory):
    return str(tmp_path_factory.mktemp("frog_idx"))


@pytest.fixture(scope="session")
def tiny(libs, cache_dir):
    """Config 1 (n=10,000, d=32, 200 queries) with its index built by the host builder."""
    import datagen
    import oracle
    wl = datagen.make_workload("tiny")
    path = os.path.join(cache_dir, "tiny.idx")
    libs.build_index(wl.vectors, wl.attrs, path, seed=wl.seed)
    return wl, path, oracle.load_index(path)


def build_scaled(libs, cache_dir, name, n, nq, **kw):
    import datagen
    import oracle
    wl = datagen.make_workload(name, n=n, nq=nq)
    path = os.path.join(cache_dir, f"{name}_{n}.idx")
    if not os.path.exists(path):
        libs.build_index(wl.vectors, wl.attrs, path, seed=wl.seed, **kw)
    return wl, path, oracle.load_index(path)
