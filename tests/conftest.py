import os
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


def pytest_configure(config):
    config.addinivalue_line("markers", "gpu: needs a CUDA device (sm_100a) and the built library")


@pytest.fixture(scope="session")
def oracle():
    import oracle as _oracle
    _oracle.build()
    return _oracle


@pytest.fixture(scope="session", autouse=True)
def _library_present():
    """The shared library is a build product that is not in the source history: compile it when
    a fresh checkout has none or when a source is newer than it (nvcc cross-compiles for sm_100a
    without a GPU; a missing nvcc with a stale library fails here rather than testing old code)."""
    from paper_2101_06983_b200 import _build
    if _build.stale():
        _build.build()


@pytest.fixture(params=["auto", "sweeps"])
def plan_mode(request, monkeypatch):
    """Runs a test twice: with the library choosing its plan, and with GRADCACHE_PLAN=sweeps in
    the environment, which keeps small problems on the sweep kernels (or the FMA tiles), the
    kernels that large problems run."""
    if request.param == "sweeps":
        monkeypatch.setenv("GRADCACHE_PLAN", "sweeps")
    else:
        monkeypatch.delenv("GRADCACHE_PLAN", raising=False)
    return request.param


@pytest.fixture
def sweeps_only(monkeypatch):
    monkeypatch.setenv("GRADCACHE_PLAN", "sweeps")
