import os
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


def pytest_configure(config):
    config.addinivalue_line("markers", "gpu: needs a CUDA device (run with -m gpu on a B200)")


def pytest_collection_modifyitems(config, items):
    """A plain `pytest tests/` on a machine without a CUDA device runs the CPU suite only: the
    GPU-marked tests are deselected unless a marker expression (-m gpu) asked for them."""
    if config.option.markexpr:
        return
    try:
        import torch
        have_gpu = torch.cuda.is_available()
    except Exception:
        have_gpu = False
    if have_gpu:
        return
    keep = [it for it in items if "gpu" not in it.keywords]
    dropped = [it for it in items if "gpu" in it.keywords]
    if dropped:
        config.hook.pytest_deselected(items=dropped)
        items[:] = keep


@pytest.fixture(scope="session")
def golden_dir():
    return os.path.join(ROOT, "tests", "golden")


@pytest.fixture(scope="session")
def mpq():
    """The Python binding over libmpq.so, built in-tree on demand (nvcc cross-compiles without a GPU)."""
    from paper_1905_13389_b200 import binding, build
    if not os.path.exists(binding.LIB_PATH):
        build.build()
    binding.lib()
    return binding


@pytest.fixture(scope="session")
def cuda(mpq):
    import torch
    if not torch.cuda.is_available():
        pytest.fail("GPU tests need a CUDA device; run them with -m gpu on a B200")
    torch.cuda.set_device(0)
    return torch.device("cuda:0")
