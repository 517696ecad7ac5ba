import os
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


def pytest_addoption(parser):
    parser.addoption("--checked", action="store_true", default=False,
                     help="run against the checked build of the library (libcatekv_checked.so, built on demand): every "
                          "device-produced index is clamped to its segment and reported; each GPU test must leave "
                          "the checked status block at zero")


def pytest_configure(config):
    config.addinivalue_line("markers", "gpu: needs a CUDA device (runs the library's kernels)")
    config.addinivalue_line("markers", "trips_checks: (with --checked) the test makes an index check fire on purpose")
    config.addinivalue_line("markers", "timing: asserts on measured times (not part of the parity gate; run with -m timing)")
    if config.getoption("--checked"):
        # must happen before the binding is imported: it loads the library named by CATEKV_LIBRARY
        import paper_2608_30295_b200.build as b
        os.environ["CATEKV_LIBRARY"] = b.build(checked=True)


@pytest.fixture(scope="session")
def golden_dir():
    return os.path.join(ROOT, "tests", "golden")


@pytest.fixture(autouse=True)
def _checked_status_stays_clear(request):
    """With --checked: no GPU test may trip one of the library's index checks (the memory checker's stand-in)."""
    if not request.config.getoption("--checked") or request.node.get_closest_marker("gpu") is None:
        yield
        return
    import paper_2608_30295_b200 as pkg
    ck = pkg.binding
    assert ck.catekv_checked_build()
    ck.catekv_checked_status(clear=True)
    yield
    if request.node.get_closest_marker("trips_checks") is None:
        st = ck.catekv_checked_status(clear=True)
        assert st["flags"] == 0, f"an index check fired: {st}"
