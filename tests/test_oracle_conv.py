"""Pins for the causal depthwise convolution (Eq. conv1d_depthwise) on the projection packing: the decrypted
result equals the float64 convolution, across token-block boundaries and with a partial channel block."""
import numpy as np

import fesc_synth as S
from oracle.ckks import Oracle, conv_masks, pack_linear_input


def _ctx(log_n):
    data = S.ntt_primes(40, log_n, 3, 5)
    special = S.ntt_primes(50, log_n, 1, 5)
    return Oracle(log_n, data + special, 3, 1, 3, 4343)


def conv_reference(q, w, b):
    """eta_k[c] = b_c + sum_r w[c,r] q_{k-r}[c], q_t = 0 for t < 0 (plain loops)."""
    tokens, channels = q.shape
    out = np.zeros_like(q)
    for k in range(tokens):
        for c in range(channels):
            acc = b[c]
            for r in range(w.shape[1]):
                if k - r >= 0:
                    acc += w[c, r] * q[k - r, c]
            out[k, c] = acc
    return out


def run_conv(o, q, w, b, T, C, d_conv, level=3, scale=2.0**30, key_base=400):
    tokens, channels = q.shape
    n = o.n
    blocks, tbs = -(-channels // C), -(-tokens // T)
    for r in range(1, d_conv):
        o.add_galois_key(-r, key_base + r)
        o.add_galois_key(T - r, key_base + d_conv + r)
    cts = np.empty((tbs, blocks, 2, level, o.N), dtype=np.uint64)
    for tb in range(tbs):
        for blk in range(blocks):
            v = pack_linear_input(q[tb * T:(tb + 1) * T, blk * C:(blk + 1) * C], T, C, n)
            cts[tb, blk] = o.encrypt(o.encode(v, scale, level), 100 + tb * blocks + blk)
    ql = float(o.q[level - 1])
    masks = np.empty((blocks, 2 * d_conv - 1, level, o.N), dtype=np.uint64)
    bias = np.empty((blocks, level, o.N), dtype=np.uint64)
    for blk in range(blocks):
        M, bv = conv_masks(w, b, blk, T, C, n)
        for i in range(2 * d_conv - 1):
            masks[blk, i] = o.encode(M[i], ql, level)
        # scale * q_last overflows the 64-bit coefficient encoder: encode at `scale`, multiply by the integer q_last
        bias[blk] = o.mul_scalar(o.encode(bv, scale, level), [o.q[level - 1]] * level, list(range(level)))
    out = o.conv(cts, masks, bias, d_conv, T, key_base)
    Y = np.zeros((tbs * T, blocks * C))
    for tb in range(tbs):
        for blk in range(blocks):
            Y[tb * T:(tb + 1) * T, blk * C:(blk + 1) * C] = o.decrypt(out[tb, blk], scale).real.reshape(C, T).T
    return cts, masks, bias, out, Y[:tokens, :channels]


def test_conv_matches_float_reference_across_blocks():
    o = _ctx(7)                      # 64 slots = C*T = 8*8
    g = np.random.default_rng(3)
    q = g.standard_normal((20, 11))  # 3 token blocks (last partial), 2 channel blocks (last partial)
    w = g.standard_normal((11, 4)) * 0.5
    b = g.standard_normal(11)
    *_, Y = run_conv(o, q, w, b, T=8, C=8, d_conv=4)
    assert np.abs(Y - conv_reference(q, w, b)).max() < 1e-4


def test_conv_single_tap_is_a_scaled_copy_plus_bias():
    o = _ctx(6)
    g = np.random.default_rng(4)
    q = g.standard_normal((8, 4))
    w = g.standard_normal((4, 1))
    b = g.standard_normal(4)
    *_, Y = run_conv(o, q, w, b, T=8, C=4, d_conv=1)
    assert np.abs(Y - (q * w[:, 0] + b)).max() < 1e-4


def test_conv_reference_against_numpy_convolve():
    g = np.random.default_rng(5)
    q = g.standard_normal((13, 3))
    w = g.standard_normal((3, 4))
    b = g.standard_normal(3)
    want = np.stack([np.convolve(q[:, c], w[c])[:13] + b[c] for c in range(3)], axis=1)
    assert np.allclose(conv_reference(q, w, b), want)
