"""GPU parity for the causal depthwise convolution: residues equal the oracle's bit for bit, and the decrypted
result equals the float64 convolution (token-block boundaries, partial channel block, one-tap degenerate case)."""
import numpy as np
import pytest

import fesc_synth as S
from oracle.ckks import conv_masks, pack_linear_input
from tests.gpu_util import add_key, ctx_pair, to_dev, to_host
from tests.test_oracle_conv import conv_reference

pytestmark = pytest.mark.gpu


def _case(name, tokens, channels, T, C, d_conv, level, scale, key_base):
    import torch
    import paper_2608_17442_b200 as fesc

    pair = ctx_pair(name)
    ctx, orc, p = pair
    n = orc.n
    assert T * C == n
    g = np.random.default_rng(p["seed"] % 1000 + d_conv)
    q = g.standard_normal((tokens, channels))
    w = g.standard_normal((channels, d_conv)) * 0.5
    b = g.standard_normal(channels)
    blocks, tbs = -(-channels // C), -(-tokens // T)
    for r in range(1, d_conv):
        add_key(pair, -r, key_base + r)
        add_key(pair, T - r, key_base + d_conv + r)
    data = list(range(level))
    cts = np.empty((tbs, blocks, 2, level, orc.N), dtype=np.uint64)
    for tb in range(tbs):
        for blk in range(blocks):
            v = pack_linear_input(q[tb * T:(tb + 1) * T, blk * C:(blk + 1) * C], T, C, n)
            cts[tb, blk] = orc.encrypt(orc.encode(v, scale, level), 9000 + tb * blocks + blk)
    ql = float(orc.q[level - 1])
    masks = np.empty((blocks, 2 * d_conv - 1, level, orc.N), dtype=np.uint64)
    bias = np.empty((blocks, level, orc.N), dtype=np.uint64)
    for blk in range(blocks):
        M, bv = conv_masks(w, b, blk, T, C, n)
        for i in range(2 * d_conv - 1):
            masks[blk, i] = orc.encode(M[i], ql, level)
        bias[blk] = orc.mul_scalar(orc.encode(bv, scale, level), [orc.q[level - 1]] * level, data)
    want = orc.conv(cts, masks, bias, d_conv, T, key_base)
    out = torch.empty((tbs, blocks, 2, level - 1, orc.N), dtype=torch.int64, device="cuda")
    ctx.conv(to_dev(cts), to_dev(masks), to_dev(bias), fesc.ConvDesc(d_conv, T, blocks, tbs, level, key_base), out)
    ctx.sync()
    got = to_host(out)
    assert np.array_equal(got, want)
    Y = np.zeros((tbs * T, blocks * C))
    for tb in range(tbs):
        for blk in range(blocks):
            Y[tb * T:(tb + 1) * T, blk * C:(blk + 1) * C] = orc.decrypt(got[tb, blk], scale, level - 1).real.reshape(C, T).T
    return np.abs(Y[:tokens, :channels] - conv_reference(q, w, b)).max()


def test_conv_small_ring_blocks_and_partial_tails():
    # N = 1024: 512 slots = 16 channels x 32 tokens; 3 token blocks (last partial), 2 channel blocks (last partial)
    assert _case("small", 70, 21, 32, 16, 4, 5, 2.0**40, 6000) < 2.0**-18


def test_conv_single_tap_and_single_block():
    assert _case("small", 32, 16, 32, 16, 1, 3, 2.0**40, 6100) < 2.0**-18
    assert _case("small", 20, 5, 32, 16, 3, 24, 2.0**40, 6200) < 2.0**-18


def test_conv_full_ring_mamba_shape_slice():
    """N = 2^16, T = 128, C = 256, d_conv = 4, 24 limbs: two token blocks x one channel block."""
    assert _case("full", 200, 256, 128, 256, 4, 24, 2.0**40, 6300) < 2.0**-18


def test_conv_missing_key_is_reported():
    import torch
    import paper_2608_17442_b200 as fesc

    ctx, orc, _ = ctx_pair("small")
    z = torch.zeros((2, 1, 2, 3, orc.N), dtype=torch.int64, device="cuda")
    with pytest.raises(fesc.FescError) as e:
        ctx.conv(z, z, z, fesc.ConvDesc(4, 32, 1, 2, 3, 7900000), z)
    assert e.value.code == fesc.ENOKEY
