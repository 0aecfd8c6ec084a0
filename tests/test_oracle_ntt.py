"""Pins for the oracle's transform: the O(N^2) definition, schoolbook negacyclic
convolution (N <= 64), round trip, linearity, and the choice of psi."""
import numpy as np
import pytest

import fesc_synth as S
from oracle import ckks
from oracle.ckks import Oracle, _lib
from tests.bigint_ref import brev, negacyclic_schoolbook


def _mk(log_n, bits=30, n_q=2):
    primes = S.ntt_primes(bits, log_n, n_q, 7) + S.ntt_primes(bits + 6, log_n, 1, 7)
    return Oracle(log_n, primes, n_q, 1, n_q, 99)


@pytest.mark.parametrize("log_n", [2, 3, 4, 6])
def test_psi_is_minimal_primitive_root(log_n):
    o = _mk(log_n)
    N = o.N
    for q in o.q:
        psi = _lib.orc_min_psi(q, log_n)
        assert pow(psi, N, q) == q - 1
        # brute force over all residues for the smallest element of order 2N (tiny q only below)
    q = 97 if log_n <= 4 else None
    if q and (q - 1) % (2 * N) == 0:
        brute = min(x for x in range(2, q) if pow(x, N, q) == q - 1)
        assert _lib.orc_min_psi(q, log_n) == brute


@pytest.mark.parametrize("log_n", [2, 4, 6])
def test_ntt_matches_python_definition(log_n):
    o = _mk(log_n)
    N, q = o.N, o.q[0]
    a = S.uniform_residues_np(3, log_n, [q], N)
    psi = _lib.orc_min_psi(q, log_n)
    want = [sum(int(a[0, i]) * pow(psi, (2 * brev(t, log_n) + 1) * i, q) for i in range(N)) % q for t in range(N)]
    got = o.ntt(a, [0])[0]
    assert [int(x) for x in got] == want


@pytest.mark.parametrize("log_n", [8, 10])
def test_ntt_matches_direct_sum(log_n):
    o = _mk(log_n, bits=50)
    q = o.q[1]
    a = S.uniform_residues_np(4, log_n, [q], o.N)
    want = np.empty(o.N, dtype=np.uint64)
    _lib.orc_ntt_direct(a[0].copy(), want, q, log_n)
    assert np.array_equal(o.ntt(a, [1])[0], want)


@pytest.mark.parametrize("log_n", [3, 6, 12])
def test_round_trip_and_linearity(log_n):
    o = _mk(log_n, bits=36)
    idx = [0, 1, 2]
    a = S.uniform_residues_np(5, 0, [o.q[i] for i in idx], o.N)
    b = S.uniform_residues_np(5, 1, [o.q[i] for i in idx], o.N)
    assert np.array_equal(o.intt(o.ntt(a, idx), idx), a)
    assert np.array_equal(o.ntt(o.intt(a, idx), idx), a)
    assert np.array_equal(o.ntt(o.add(a, b, idx), idx), o.add(o.ntt(a, idx), o.ntt(b, idx), idx))


@pytest.mark.parametrize("log_n", [2, 5, 6])
def test_pointwise_product_is_negacyclic_convolution(log_n):
    o = _mk(log_n)
    q = o.q[0]
    a = S.uniform_residues_np(6, 0, [q], o.N)
    b = S.uniform_residues_np(6, 1, [q], o.N)
    c = o.intt(o.mul(o.ntt(a, [0]), o.ntt(b, [0]), [0]), [0])[0]
    assert [int(x) for x in c] == negacyclic_schoolbook(a[0], b[0], q)


def test_x_to_the_n_is_minus_one():
    o = _mk(4)
    q = o.q[0]
    x = np.zeros((1, o.N), dtype=np.uint64)
    x[0, 1] = 1
    xe = o.ntt(x, [0])
    acc = xe.copy()
    for _ in range(o.N - 1):
        acc = o.mul(acc, xe, [0])
    assert np.all(acc == q - 1)
