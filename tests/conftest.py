import os
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


def pytest_configure(config):
    config.addinivalue_line("markers", "gpu: needs a CUDA device (run with -m gpu on a B200)")
    # a fresh checkout has no built libraries (they are kept out of the history): build them once, in-tree
    from paper_2508_19263_b200 import build as zbuild
    if not os.path.exists(zbuild.LIB):
        zbuild.build_library()
    import oracle
    oracle.build()


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


_checked_tests = 0


@pytest.fixture(autouse=True)
def _no_refused_access_in_a_checked_build(request):
    """With the development build loaded (ZC_LIBRARY points at it) every GPU test ends with its counters at zero."""
    yield
    if "gpu" not in request.keywords or not os.environ.get("ZC_LIBRARY"):
        return
    from paper_2508_19263_b200 import binding as zc
    counts = zc.test_debug_counts()
    if counts is not None:
        global _checked_tests
        _checked_tests += 1
        assert counts == (0, 0), f"refused accesses (shared, global): {counts}"


def pytest_terminal_summary(terminalreporter):
    if _checked_tests:
        terminalreporter.write_line(f"debug build: checked the access counters after {_checked_tests} tests")
