"""Pins for the BSGS projection (App. "Projection Kernel Breakdown"): decrypt(linear(Enc X)) = X W,
on the paper's toy shape (T=2, C=4, n1=n2=2, X 2x4, W 4x4) and on multi-block shapes."""
import numpy as np
import pytest

import fesc_synth as S
from oracle.ckks import Oracle, linear_diagonal, pack_linear_input


def _ctx(log_n):
    data = S.ntt_primes(40, log_n, 3, 5)
    special = S.ntt_primes(50, log_n, 1, 5)
    return Oracle(log_n, data + special, 3, 1, 3, 4242)


def _run(o, X, W, T, C, n1, n2, hoist=False, defer=False, raw=False):
    n = o.n
    assert C * T == n and n1 * n2 == C
    tokens, d_in = X.shape
    d_out = W.shape[1]
    gin, nout, tbs = -(-d_in // C), -(-d_out // C), -(-tokens // T)
    level, scale = 3, 2.0**30
    for q in range(1, n1):
        o.add_galois_key(q * T, 100 + q)
    for p in range(1, n2):
        o.add_galois_key(p * n1 * T, 200 + p)
    cts = np.empty((tbs, gin, 2, level, o.N), dtype=np.uint64)
    for tb in range(tbs):
        for g in range(gin):
            v = pack_linear_input(X[tb * T:(tb + 1) * T, g * C:(g + 1) * C], T, C, n)
            cts[tb, g] = o.encrypt(o.encode(v, scale, level), tb * gin + g)
    diags = np.empty((nout, n2, gin, n1, level, o.N), dtype=np.uint64)
    for b in range(nout):
        for p in range(n2):
            for g in range(gin):
                for q in range(n1):
                    diags[b, p, g, q] = o.encode(linear_diagonal(W, b, g, p, q, T, C, n1), float(o.q[level - 1]), level)
    out = o.linear(cts, diags, dict(n1=n1, n2=n2), {q: 100 + q for q in range(1, n1)}, {p: 200 + p for p in range(1, n2)},
                   hoist=hoist, defer=defer)
    if raw:
        return out
    Y = np.zeros((tbs * T, nout * C))
    for tb in range(tbs):
        for b in range(nout):
            slots = o.decrypt(out[tb, b], scale).real
            Y[tb * T:(tb + 1) * T, b * C:(b + 1) * C] = slots.reshape(C, T).T
    return Y[:tokens, :d_out]


def test_paper_toy_projection():
    o = _ctx(4)  # 8 slots = C*T = 4*2
    X, W = S.linear_inputs(11, 2, 4, 4)
    Y = _run(o, X, W * 50, 2, 4, 2, 2)
    assert np.abs(Y - X @ (W * 50)).max() < 1e-4


@pytest.mark.parametrize("shape", [(8, 8, 4, 2, 5, 19, 13), (4, 16, 4, 4, 9, 40, 20)])
def test_multi_block_projection(shape):
    T, C, n1, n2, tokens, d_in, d_out = shape
    o = _ctx(int(np.log2(T * C)) + 1)
    X, W = S.linear_inputs(12, tokens, d_in, d_out)
    Y = _run(o, X, W * 50, T, C, n1, n2)
    assert np.abs(Y - X @ (W * 50)).max() < 1e-4


def test_projection_with_hoisted_baby_rotations():
    o = _ctx(7)
    X, W = S.linear_inputs(14, 9, 19, 13)
    Y = _run(o, X, W * 50, 8, 8, 4, 2, hoist=True)
    assert np.abs(Y - X @ (W * 50)).max() < 1e-4


def test_projection_with_deferred_division_in_giant_steps():
    """One division by P per output: same values; with a single giant step the residues are those of the
    separate rotation (the sum has one term).  (With several the sums differ by a few units before the
    rescale, see the next test; the rescale then hides almost all of it.)"""
    o = _ctx(7)
    X, W = S.linear_inputs(15, 6, 20, 10)
    for hoist in (False, True):
        Y = _run(o, X, W * 50, 4, 16, 4, 4, hoist=hoist, defer=True)
        assert np.abs(Y - X @ (W * 50)).max() < 1e-4
    a = _run(o, X, W * 50, 4, 16, 8, 2, raw=True)
    b = _run(o, X, W * 50, 4, 16, 8, 2, defer=True, raw=True)
    assert np.array_equal(a, b)


def test_deferred_division_is_additive_up_to_rounding():
    """ModDown(sum raw_p) and sum ModDown(raw_p) differ by at most n2 - 1 in every coefficient (big-integer check
    of the claim that the deferred mode computes the same ciphertext up to rounding)."""
    from oracle.ckks import crt_lift_centered
    o = _ctx(5)
    level = 3
    data = list(range(level))
    for p in range(1, 4):
        o.add_galois_key(p, 300 + p)
    rng = np.random.default_rng(5)
    accs = [np.stack([np.stack([rng.integers(0, o.q[i], o.N, dtype=np.uint64) for i in data]) for _ in range(2)])
            for _ in range(4)]
    keys = {p: 300 + p for p in range(1, 4)}
    lazy = o.giant_sum_deferred(accs, keys)
    eager = accs[0]
    for p in range(1, 4):
        eager = o.ct_add(eager, o.rotate(accs[p], keys[p]))
    Q = 1
    for i in data:
        Q *= o.q[i]
    seen = 0
    for c in range(2):
        d = o.sub(lazy[c], eager[c], data)
        diff = crt_lift_centered(o.intt(d, data), [o.q[i] for i in data])
        assert max(abs(int(v)) for v in diff) <= 3
        seen += sum(1 for v in diff if int(v) != 0)
    assert seen > 0


def test_diagonal_formula_on_plain_slots():
    """The diagonal/rotation bookkeeping alone, on float vectors with np.roll standing for rho."""
    T, C, n1, n2 = 2, 8, 4, 2
    X, W = S.linear_inputs(13, T, 2 * C, 3 * C)
    for b in range(3):
        y = np.zeros(C * T)
        for p in range(n2):
            acc = np.zeros(C * T)
            for g in range(2):
                x = pack_linear_input(X[:, g * C:(g + 1) * C], T, C, C * T)
                for q in range(n1):
                    acc += np.roll(x, -q * T) * linear_diagonal(W, b, g, p, q, T, C, n1)
            y += np.roll(acc, -p * n1 * T)
        assert np.allclose(y.reshape(C, T).T, (X @ W)[:, b * C:(b + 1) * C])
