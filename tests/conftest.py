import os
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


def pytest_addoption(parser):
    parser.addoption("--checked-build", action="store_true", default=False,
                     help="run against the library built with -DENTRO_CHECKED (bounds checks on every address the "
                          "decode kernel computes by hand) and fail any test after which a violation was counted")


def pytest_configure(config):
    config.addinivalue_line("markers", "gpu: needs a CUDA device (run on the GPU box)")
    if config.getoption("--checked-build"):
        import paper_2505_02380_b200 as E
        from paper_2505_02380_b200 import build as build_mod
        E.LIB_PATH = os.environ["ENTRO_LIBRARY"] = build_mod.build(checked=True)   # lib() loads on first use


@pytest.fixture(autouse=True)
def _no_bounds_violation(request):
    """With --checked-build: no test may leave a counted violation behind."""
    yield
    if request.config.getoption("--checked-build") and "gpu" in request.keywords:
        import paper_2505_02380_b200 as E
        assert E.entro_checked_build()
        assert E.entro_check_violations() == 0


def pytest_collection_modifyitems(config, items):
    try:
        import torch
        has_gpu = torch.cuda.is_available()
    except Exception:
        has_gpu = False
    if has_gpu:
        return
    skip = pytest.mark.skip(reason="no CUDA device")
    for item in items:
        if "gpu" in item.keywords:
            item.add_marker(skip)
