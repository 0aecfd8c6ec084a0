"""Bit-exact scan-contract parity on the deployed ring (N = 2^16, 24 x 50-bit + 4 x 60-bit primes, 6 digits).

The deployed geometry (blocks of 256 tokens) is ~30 000 key switches per slice, far beyond what the CPU oracle can
follow, so the residue-level comparison at this ring uses a block of 4 tokens: n = 32768 slots, stride = d_s = 128,
P = 64, H = 8 (c_state = 256 channels = 4 heads per chunk, K_s = 2: one chunk pair, so the monomial pairing and the
conjugation run), B_blk = 4, L = 8 (two blocks, so the summary, the serialized carry and its injection run), l0 = 24.
Every kernel the scan sequences runs at its deployed size here: the two-kernel N = 2^16 transforms, the hand-over
of doubles between the key-switch kernels, the 16-ciphertext key-switch passes, the batched level adjusts and the
grouped class multiply-accumulate.

Default-mode case (hoisted rotations, leaves in groups of 4 tokens: what the benchmark runs): 364 rotations, 8
conjugations, 70 relinearisations = 442 key switches, 80 level adjusts, 194 plaintext products, 41 Galois keys;
the oracle follows it in about a minute on 16 host cores (keys included).  The plain-mode case (every rotation a
fesc_rotate with its own decomposition, token-by-token leaves) is 480 rotations + 8 + 70 = 558 key switches.
"""
import numpy as np
import pytest

from tests.gpu_util import run_scan_parity

pytestmark = pytest.mark.gpu

SHAPE = dict(L=8, H=8, P=64, d_s=128, B_blk=4, stride=128)


def test_scan_full_ring_default_mode_bit_exact():
    err = run_scan_parity("full", hoist=1, group=4, **SHAPE)
    assert err < 2.0**-18, np.log2(err)


def test_scan_full_ring_plain_mode_bit_exact():
    err = run_scan_parity("full", hoist=0, group=0, **SHAPE)
    assert err < 2.0**-18, np.log2(err)
