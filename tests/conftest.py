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
