import os
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


def _build_library_if_stale():
    """The package refuses to import without its CUDA library, so the build script is loaded by
    path and run (a no-op when the library is newer than its sources) before any test imports it."""
    import importlib.util

    spec = importlib.util.spec_from_file_location(
        "_powerattn_build", os.path.join(ROOT, "paper_2503_03588_b200", "build.py"))
    mod = importlib.util.module_from_spec(spec)
    spec.loader.exec_module(mod)
    mod.build()


def pytest_configure(config):
    config.addinivalue_line("markers", "gpu: needs a CUDA device (run with -m gpu on a B200)")
    _build_library_if_stale()


@pytest.fixture(scope="session")
def oracle():
    from oracle import oracle as _oracle

    _oracle.build()
    return _oracle


@pytest.fixture
def pa_env(monkeypatch):
    """Sets PA_* environment switches for one test and makes the library re-read them (it reads
    the environment once); the previous state comes back, and is re-read, afterwards."""
    import paper_2503_03588_b200 as pa

    def set_env(**kv):
        for key, val in kv.items():
            monkeypatch.setenv(key, val)
        pa.pa_reload_environment()

    yield set_env
    monkeypatch.undo()
    pa.pa_reload_environment()
