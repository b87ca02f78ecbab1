import os
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


def pytest_configure(config):
    config.addinivalue_line("markers", "gpu: needs a CUDA device (sm_100a)")


def pytest_collection_modifyitems(config, items):
    try:
        import torch

        has_gpu = torch.cuda.is_available()
    except Exception:  # pragma: no cover
        has_gpu = False
    if has_gpu:
        return
    skip = pytest.mark.skip(reason="no CUDA device")
    for item in items:
        if "gpu" in item.keywords:
            item.add_marker(skip)


@pytest.fixture(scope="session", autouse=True)
def _built_library():
    """Compile libcpmtp.so once per session if it is missing or older than its sources (and the checked
    build too when CPMTP_LIBRARY=debug selects it)."""
    from paper_2410_17765_b200 import build

    build.build()
    if os.environ.get("CPMTP_LIBRARY") == "debug":
        build.build(debug=True)
    yield


@pytest.fixture(autouse=True)
def _index_checks_stay_clean(request):
    """With the checked build (CPMTP_LIBRARY=debug) every GPU test also asserts, when it ends, that none of the
    index checks compiled into the epilogues has failed so far."""
    yield
    if os.environ.get("CPMTP_LIBRARY") == "debug" and "gpu" in request.keywords:
        from paper_2410_17765_b200 import binding

        assert binding.debug_status() == 0, "an index check of the checked build failed"
