"""Pins for the CKKS steps around the NeRMS protocol (Alg. "one Block": u = y~ (.) y~ and
y^ = gamma_RMS (.) (y~ (.) br(s_RMS))) on the projection packing: decrypted results equal the float64 definition."""
import numpy as np

import fesc_synth as S
from oracle.ckks import Oracle, pack_linear_input


def _ctx(log_n, n_q=4):
    data = S.ntt_primes(40, log_n, n_q, 5)
    special = S.ntt_primes(50, log_n, 1, 5)
    return Oracle(log_n, data + special, n_q, 1, n_q, 5151)


def run_norm(o, y, s, gamma, T, C, level, scale=2.0**40, key_base=700, nonce=300, add_key=None):
    """y [tokens, channels], s [tokens], gamma [channels] -> (cts, s_cts, gamma_pts, out, Y^ [tokens, channels])."""
    tokens, channels = y.shape
    n = o.n
    blocks, tbs = -(-channels // C), -(-tokens // T)
    steps = (n // T).bit_length() - 1
    for b in range(steps):
        (add_key or o.add_galois_key)(-(T << b), key_base + b)
    cts = np.empty((tbs, blocks, 2, level, o.N), dtype=np.uint64)
    s_cts = np.empty((tbs, 2, level, o.N), dtype=np.uint64)
    for tb in range(tbs):
        sv = np.zeros(n)
        part = s[tb * T:(tb + 1) * T]
        sv[:len(part)] = part
        s_cts[tb] = o.encrypt(o.encode(sv, float(o.q[level - 1]), level), nonce + 1000 + tb)
        for blk in range(blocks):
            v = pack_linear_input(y[tb * T:(tb + 1) * T, blk * C:(blk + 1) * C], T, C, n)
            cts[tb, blk] = o.encrypt(o.encode(v, scale, level), nonce + tb * blocks + blk)
    gamma_pts = np.empty((blocks, level - 1, o.N), dtype=np.uint64)
    for blk in range(blocks):
        gv = np.zeros(n)
        for c in range(C):
            if blk * C + c < channels:
                gv[c * T:(c + 1) * T] = gamma[blk * C + c]
        gamma_pts[blk] = o.encode(gv, float(o.q[level - 2]), level - 1)
    out = o.norm_scale(cts, s_cts, gamma_pts, T, key_base)
    Y = np.zeros((tbs * T, blocks * C))
    for tb in range(tbs):
        for blk in range(blocks):
            Y[tb * T:(tb + 1) * T, blk * C:(blk + 1) * C] = o.decrypt(out[tb, blk], scale).real.reshape(C, T).T
    return cts, s_cts, gamma_pts, out, Y[:tokens, :channels]


def test_norm_scale_matches_float_definition():
    o = _ctx(7)                                   # 64 slots = 8 channels x 8 tokens
    g = np.random.default_rng(11)
    y = g.standard_normal((20, 11))               # 3 token blocks (last partial), 2 channel blocks (last partial)
    s = 1.0 / np.sqrt((y * y).mean(axis=1) + 1e-5)
    gamma = g.uniform(0.5, 1.5, 11)
    *_, Y = run_norm(o, y, s, gamma, T=8, C=8, level=4)
    assert np.abs(Y - gamma[None, :] * y * s[:, None]).max() < 1e-5
    # the rows of the result have unit mean square before the weights (what the normalisation is for)
    assert np.allclose(((Y / gamma[None, :]) ** 2).mean(axis=1), 1.0, atol=1e-3)


def test_norm_scale_token_factor_reaches_every_channel_and_no_other_token():
    o = _ctx(6)                                   # 32 slots = 4 channels x 8 tokens
    y = np.ones((8, 4))
    s = np.zeros(8)
    s[3] = 2.0                                    # only token 3 is scaled; every other token must come out as zero
    gamma = np.array([1.0, -1.0, 0.5, 0.25])
    *_, Y = run_norm(o, y, s, gamma, T=8, C=4, level=3)
    want = np.zeros((8, 4))
    want[3] = 2.0 * gamma
    assert np.abs(Y - want).max() < 1e-5


def test_norm_square_is_the_slotwise_square():
    o = _ctx(6, n_q=3)
    g = np.random.default_rng(12)
    z = g.uniform(-1, 1, (3, o.n))
    cts = np.stack([o.encrypt(o.encode(z[i], 2.0**40, 3), 40 + i) for i in range(3)])
    u = o.norm_square(cts)
    assert u.shape == (3, 2, 2, o.N)
    scale = 2.0**80 / float(o.q[2])
    for i in range(3):
        assert np.abs(o.decrypt(u[i], scale).real - z[i] ** 2).max() < 1e-5
