"""The bounds-checking debug build (a stand-in for a memory checker): the library compiled with -DFESC_DEBUG_BOUNDS makes
every kernel compare the regions it is about to touch with the extents of the library's allocations and of the tensors
the binding passed, skips what lies outside and reports it through fesc_sync.  Two checks: the parity tests of the small
rings (and the N = 2^16 primitives) pass under that build with an empty record, and a call that is told to walk past the
registered extent of its buffer (inside a larger allocation, so nothing can fault) is caught, skipped and reported."""
import os
import subprocess
import sys

import numpy as np
import pytest

pytestmark = pytest.mark.gpu

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
IN_DEBUG_RUN = "FESC_LIB" in os.environ


def _debug_lib():
    from paper_2608_17442_b200 import build

    return build.build(debug_bounds=True)


@pytest.mark.skipif(IN_DEBUG_RUN, reason="this is the inner run")
def test_parity_suite_is_clean_under_the_debug_build():
    env = dict(os.environ, FESC_LIB=_debug_lib())
    files = ["tests/test_gpu_primitives.py", "tests/test_gpu_linear.py", "tests/test_gpu_conv.py", "tests/test_gpu_norm.py",
             "tests/test_gpu_scan.py", "tests/test_zz_no_alloc.py", "tests/test_gpu_debug_bounds.py"]
    skip = "not test_linear_full_ring_one_block and not workload_1 and not workload_3 and not ntt_sweep"
    r = subprocess.run([sys.executable, "-m", "pytest", "-x", "-q", "-m", "gpu", "-k", skip, "-rp", "-p", "no:cacheprovider"] + files,
                       cwd=ROOT, env=env, capture_output=True, text=True, timeout=1500)
    tail = (r.stdout + r.stderr)[-3000:]
    assert r.returncode == 0, tail
    assert "PASSED tests/test_gpu_debug_bounds.py::test_region_outside_the_registered_extent_is_skipped_and_reported" in r.stdout
    assert "PASSED tests/test_gpu_linear.py::test_linear_small_ring" in r.stdout and "failed" not in tail


@pytest.mark.skipif(not IN_DEBUG_RUN, reason="needs the debug build (runs inside the test above)")
def test_region_outside_the_registered_extent_is_skipped_and_reported():
    import torch
    import paper_2608_17442_b200 as fesc
    from tests.gpu_util import ctx_pair

    assert fesc.debug_bounds()
    ctx, orc, p = ctx_pair("small")
    N, limbs = orc.N, 4
    rng = np.random.default_rng(5)
    host = np.stack([rng.integers(0, int(q), N, dtype=np.uint64) for q in p["primes"][:limbs]])
    big = torch.from_numpy(np.stack([host, host]).view(np.int64)).cuda()      # two batches of `limbs` rows, one allocation
    ctx.sync()
    fesc.debug_bounds_clear()
    fesc.debug_bounds_report()
    view = big[0]                                   # the binding registers one batch ...
    ctx.ntt(view, 2, 0, limbs)                      # ... and the call asks for two
    with pytest.raises(fesc.FescError) as e:
        ctx.sync()
    assert e.value.code == fesc.EBOUNDS and "file 2" in str(e.value)          # file id 2: the transforms
    got = big.cpu().numpy().view(np.uint64)
    assert np.array_equal(got[0], orc.ntt(host, list(range(limbs))))   # inside the extent: transformed
    assert np.array_equal(got[1], host)             # outside: not touched
    ctx.sync()                                      # the failing sync started a new record; the context stays usable
    ctx.intt(big, 1, 0, limbs)                      # the whole tensor registered: clean
    ctx.sync()
    assert np.array_equal(big.cpu().numpy().view(np.uint64)[0], host)
    assert fesc.debug_bounds_report()[0] == 0
