"""GPU parity for the CKKS steps around the NeRMS protocol: residues equal the oracle's bit for bit and the decrypted
result equals gamma (.) y (.) s per token (token-block and channel-block tails, the N = 2^16 deployed shape)."""
import numpy as np
import pytest

from tests.gpu_util import add_key, ctx_pair, random_ct, to_dev, to_host
from tests.test_oracle_norm import run_norm

pytestmark = pytest.mark.gpu


def _case(name, tokens, channels, T, C, level, key_base):
    import torch
    import paper_2608_17442_b200 as fesc

    pair = ctx_pair(name)
    ctx, orc, p = pair
    assert T * C == orc.n
    g = np.random.default_rng(p["seed"] % 1000 + tokens)
    y = g.standard_normal((tokens, channels))
    s = 1.0 / np.sqrt((y * y).mean(axis=1) + 1e-5)
    gamma = g.uniform(0.5, 1.5, channels)
    cts, s_cts, gamma_pts, want, Y = run_norm(orc, y, s, gamma, T, C, level, key_base=key_base, nonce=12000,
                                              add_key=lambda r, k: add_key(pair, r, k))
    tbs, blocks = cts.shape[0], cts.shape[1]
    out = torch.empty((tbs, blocks, 2, level - 2, orc.N), dtype=torch.int64, device="cuda")
    ctx.norm_scale(to_dev(cts), to_dev(s_cts), to_dev(gamma_pts), fesc.NormDesc(T, blocks, tbs, level, key_base), out)
    ctx.sync()
    assert np.array_equal(to_host(out), want)
    return np.abs(Y - gamma[None, :] * y * s[:, None]).max()


def test_norm_scale_small_ring_blocks_and_partial_tails():
    # N = 1024: 512 slots = 16 channels x 32 tokens; 3 token blocks (last partial), 2 channel blocks (last partial)
    assert _case("small", 70, 21, 32, 16, 5, 6500) < 2.0**-18
    assert _case("small", 32, 16, 32, 16, 3, 6600) < 2.0**-18          # lowest level, one block each


def test_norm_scale_full_ring_deployed_shape_slice():
    """N = 2^16, T = 128, C = 256, 24 limbs: two token blocks (last partial) x one channel block."""
    assert _case("full", 200, 256, 128, 256, 24, 6700) < 2.0**-18


@pytest.mark.parametrize("name,level,batch", [("small", 5, 3), ("small", 2, 1), ("wide", 4, 2), ("full", 24, 2)])
def test_norm_square_equals_oracle(name, level, batch):
    import torch

    ctx, orc, p = ctx_pair(name)
    ct = random_ct(orc, p["seed"], 77, level, batch)
    want = orc.norm_square(ct)
    out = torch.empty((batch, 2, level - 1, orc.N), dtype=torch.int64, device="cuda")
    ctx.norm_square(to_dev(ct), out, batch, level)
    ctx.sync()
    assert np.array_equal(to_host(out), want)


def test_norm_errors():
    import torch
    import paper_2608_17442_b200 as fesc

    ctx, orc, p = ctx_pair("small")
    z = torch.zeros((1, 1, 2, 5, orc.N), dtype=torch.int64, device="cuda")
    with pytest.raises(fesc.FescError) as e:
        ctx.norm_scale(z, z, z, fesc.NormDesc(32, 1, 1, 5, 7700000), z)       # no keys under this base
    assert e.value.code == fesc.ENOKEY
    with pytest.raises(fesc.FescError) as e:
        ctx.norm_scale(z, z, z, fesc.NormDesc(32, 1, 1, 2, 6500), z)          # two rescales need three limbs
    assert e.value.code == fesc.ELEVEL
    with pytest.raises(fesc.FescError) as e:
        ctx.norm_scale(z, z, z, fesc.NormDesc(24, 1, 1, 5, 6500), z)          # T not a power of two
    assert e.value.code == fesc.EINVAL
    ctx.norm_square(z, z, 0, 5)                                                # empty batch is a no-op
    ctx.sync()
