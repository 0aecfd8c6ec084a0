import os
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


def pytest_configure(config):
    config.addinivalue_line("markers", "gpu: needs a CUDA device (run with -m gpu on a B200)")


@pytest.fixture(scope="session")
def toy_oracle():
    import fesc_synth as S
    from oracle.ckks import Oracle

    p = S.params("toy")
    return Oracle(p["log_n"], p["primes"], p["n_q"], p["n_p"], p["dnum"], p["seed"])


@pytest.fixture(autouse=True)
def _debug_build_reports_no_skipped_region(request):
    """Under the bounds-checking debug build (FESC_LIB names libfesc_b200_dbg.so) every GPU test must end with an empty
    bounds record: no kernel met a region outside the known extents."""
    yield
    if "FESC_LIB" not in os.environ or request.node.get_closest_marker("gpu") is None:
        return
    import paper_2608_17442_b200 as fesc

    if fesc.debug_bounds():
        hits, site, addr, nbytes = fesc.debug_bounds_report()
        assert hits == 0, f"{hits} skipped region(s); first: file {site >> 16} line {site & 0xffff}, address {addr:#x}, {nbytes} bytes"
