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


def test_token_major_packing_with_periodic_diagonals():
    """The transposed packing (slot r*C + c, one segment per token): a feature shift is the intra-segment shift Psi of
    App. "Projection Kernel Breakdown" (two rotations, masks folded into the diagonals), the projection is a baby-step /
    giant-step sum over 2 n1 - 1 and 2 n2 - 1 rotation amounts evaluated by the same `linear`, the result is X @ W, and
    every diagonal has period C in the slots, i.e. is constant on aligned runs of N / (2C) evaluation indices."""
    from oracle.ckks import (linear_diagonal_token_major, pack_linear_input_token_major, periodic_eval_runs,
                             token_major_amounts)
    p = S.params("small")
    orc = Oracle(p["log_n"], p["primes"], p["n_q"], p["n_p"], p["dnum"], p["seed"])
    n = orc.n
    T, C, n1, n2, level, scale = 32, 16, 4, 4, 4, 2.0**40
    tokens, d_in, d_out = 50, 24, 20                        # partial token block, partial input and output blocks
    X, W = S.linear_inputs(p["seed"] + 4, tokens, d_in, d_out)
    W = W * 10
    gin, nout, tbs = -(-d_in // C), -(-d_out // C), -(-tokens // T)
    baby, giant = token_major_amounts(C, n1, n2)
    assert baby == [0, 1, 1 - C, 2, 2 - C, 3, 3 - C] and giant == [0, 4, 4 - C, 8, 8 - C, 12, 12 - C]
    for i, a in enumerate(baby[1:], 1):
        orc.add_galois_key(a, 100 + i)
    for i, a in enumerate(giant[1:], 1):
        orc.add_galois_key(a, 200 + i)
    cts = np.empty((tbs, gin, 2, level, orc.N), dtype=np.uint64)
    for tb in range(tbs):
        for g in range(gin):
            v = pack_linear_input_token_major(X[tb * T:(tb + 1) * T, g * C:(g + 1) * C], T, C, n)
            cts[tb, g] = orc.encrypt(orc.encode(v, scale, level), 7000 + tb * gin + g)
    nb, ng, run = len(baby), len(giant), orc.N // (2 * C)
    diags = np.empty((nout, ng, gin, nb, level, orc.N), dtype=np.uint64)
    for b in range(nout):
        for gi in range(ng):
            for g in range(gin):
                for bi in range(nb):
                    v = linear_diagonal_token_major(W, b, g, gi, bi, T, C, n1)
                    assert np.array_equal(v.reshape(T, C), np.tile(v[:C], (T, 1)))        # period C in the slots
                    diags[b, gi, g, bi] = orc.encode(v, float(orc.q[level - 1]), level)
                    small = periodic_eval_runs(diags[b, gi, g, bi], run)                 # asserts constant runs
                    assert small.shape == (level, 2 * C)
                    assert np.array_equal(np.repeat(small, run, axis=1), diags[b, gi, g, bi])
    # the stay / wrap split covers every (input feature, output feature) pair exactly once
    cover = np.zeros((C, C), dtype=int)
    for gi in range(ng):
        for bi in range(nb):
            v = linear_diagonal_token_major(np.ones((C, C)), 0, 0, gi, bi, T, C, n1)[:C]
            pp, q = (gi + 1) // 2, (bi + 1) // 2
            for cpp in np.nonzero(v)[0]:
                c_out = cpp + C - pp * n1 if (gi and gi % 2 == 0) else cpp - pp * n1
                cover[(cpp + q) % C, c_out] += 1
    assert np.all(cover == 1)
    for hoist, defer in ((False, False), (True, True)):
        out = orc.linear(cts, diags, dict(n1=nb, n2=ng), {i: 100 + i for i in range(1, nb)},
                         {i: 200 + i for i in range(1, ng)}, hoist=hoist, defer=defer)
        Y = np.zeros((tbs * T, nout * C))
        for tb in range(tbs):
            for b in range(nout):
                Y[tb * T:(tb + 1) * T, b * C:(b + 1) * C] = orc.decrypt(out[tb, b], scale, 2).real.reshape(T, C)
        assert np.abs(Y[:tokens, :d_out] - X @ W).max() < 2.0**-18
    # a vector that is not periodic is refused by the compression
    with pytest.raises(AssertionError):
        periodic_eval_runs(orc.encode(np.arange(n) / n, scale, level), run)
    # deployed ring: period C = 256 at N = 2^16 leaves 512 of 65536 words per limb
    assert 65536 // (2 * 256) == 128
