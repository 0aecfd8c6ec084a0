"""GPU parity for the scan-contract: every output residue equals the oracle's, and the decrypted result
equals the float64 recurrence, on the paper's toy shape and on 128-slot analogues of the deployed geometry
(carries over three blocks with a partial last block; two-digit token offsets with an odd chunk count)."""
import numpy as np
import pytest

import fesc_synth as S
from oracle.ckks import CONJ
from oracle.scan import (ScanConsts, ScanEvaluator, ScanShape, add_scan_keys, encrypt_inputs, float_recurrence,
                         key_id_for, unpack_output)
from tests.gpu_util import ctx_pair, run_scan_parity as _run, run_scan_parity_invariant as _run_inv, to_dev, to_host

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("hoist", [0, 1])
def test_scan_paper_toy_shape(hoist):
    assert _run("scan_toy", hoist, L=4, H=2, P=4, d_s=2, B_blk=4) < 2.0**-24


@pytest.mark.parametrize("hoist", [0, 1])
def test_scan_analogue_with_carries_and_partial_block(hoist):
    assert _run("scan_small", hoist, L=40, H=8, P=4, d_s=8, B_blk=16) < 2.0**-22


@pytest.mark.parametrize("hoist", [0, 1])
def test_scan_two_digit_offsets_and_odd_chunk_count(hoist):
    assert _run("scan_small", hoist, L=64, H=3, P=4, d_s=4, B_blk=32) < 2.0**-22


@pytest.mark.parametrize("network", ["ks", "sk"])
def test_scan_other_prefix_networks(network):
    """Kogge-Stone and Sklansky networks: bit-exact against the oracle's network of the same name (toy shape; carries
    over three blocks with a partial last block, plain and hoisted rotations)."""
    assert _run("scan_toy", 0, network, L=4, H=2, P=4, d_s=2, B_blk=4) < 2.0**-24
    assert _run("scan_small", 0, network, L=40, H=8, P=4, d_s=8, B_blk=16) < 2.0**-22
    assert _run("scan_small", 1, network, L=64, H=3, P=4, d_s=4, B_blk=32) < 2.0**-22


@pytest.mark.parametrize("hoist", [0, 1])
def test_scan_grouped_leaf_build(hoist):
    """Leaves built for groups of G tokens: bit-exact against the oracle's grouped mode (G = 2 on the toy shape, G = 4
    with carries over three blocks and a partial last block, G = 4 with two-digit group offsets, G = 2 under Sklansky)."""
    assert _run("scan_toy", hoist, group=2, L=4, H=2, P=4, d_s=2, B_blk=4) < 2.0**-24
    assert _run("scan_small", hoist, group=4, L=40, H=8, P=4, d_s=8, B_blk=16) < 2.0**-22
    assert _run("scan_small", hoist, group=4, L=64, H=3, P=4, d_s=4, B_blk=32) < 2.0**-22
    if hoist:
        assert _run("scan_small", hoist, "sk", 2, L=40, H=8, P=4, d_s=8, B_blk=16) < 2.0**-22


@pytest.mark.parametrize("hoist,group", [(0, 0), (1, 0), (0, 4), (1, 4)])
def test_scan_full_slot_variant_with_token_segments(hoist, group):
    """stride = d_s < B_blk: two token segments per block, every slot of the state ciphertexts in use."""
    assert _run("scan_small", hoist, group=group, L=40, H=8, P=4, d_s=8, B_blk=16, stride=8) < 2.0**-22


@pytest.mark.parametrize("hoist", [0, 1])
def test_scan_invariant_families_plaintext_decay(hoist):
    """desc.plain = 1 (S4D / S5 / LRU packets: plaintext abar, Bbar, Cbar, encrypted x): bit-exact against the oracle's
    invariant-family mode on the toy shape, with carries over three blocks and a partial last block, with grouped
    leaves, and with every slot in use; the library's key-switch count equals the oracle's rotations + conjugations
    (no relinearisation anywhere)."""
    assert _run_inv("scan_toy", hoist, L=4, H=2, P=4, d_s=2, B_blk=4) < 2.0**-24
    assert _run_inv("scan_small", hoist, L=40, H=8, P=4, d_s=8, B_blk=16) < 2.0**-22
    assert _run_inv("scan_small", hoist, group=4, L=40, H=8, P=4, d_s=8, B_blk=16) < 2.0**-22
    assert _run_inv("scan_small", hoist, group=4, L=40, H=8, P=4, d_s=8, B_blk=16, stride=8) < 2.0**-22
    assert _run_inv("scan_small", hoist, L=64, H=3, P=4, d_s=4, B_blk=32) < 2.0**-22


def test_scan_invariant_mode_refuses_other_networks_and_missing_tables():
    import torch
    import paper_2608_17442_b200 as fesc
    ctx, orc, p = ctx_pair("scan_toy")
    z = torch.zeros(8, dtype=torch.int64, device="cuda")
    for net, tables in ((fesc.NET_SKLANSKY, (z,) * 6), (fesc.NET_BRENT_KUNG, None)):
        desc = fesc.ScanDesc(4, 2, 4, 2, 4, 0, p["n_q"], 100000, 0, net, 0, 1)
        with pytest.raises(fesc.FescError) as e:
            ctx.scan_contract(z, None, None, None, desc, z, None, None, z, [0], None, z, None, tables)
        assert e.value.code == fesc.EINVAL


def test_scan_unknown_network_is_refused():
    import torch
    import paper_2608_17442_b200 as fesc
    ctx, orc, p = ctx_pair("scan_toy")
    z = torch.zeros(8, dtype=torch.int64, device="cuda")
    desc = fesc.ScanDesc(4, 2, 4, 2, 4, 0, p["n_q"], 100000, 0, 7)
    with pytest.raises(fesc.FescError) as e:
        ctx.scan_contract(z, z, z, z, desc, z, z, z, z, [0], [0], z)
    assert e.value.code == fesc.EINVAL
    for group, masks in ((3, (z,) * 6), (8, (z,) * 6), (2, None)):      # not a power of two; above d_s; no masks
        desc = fesc.ScanDesc(4, 2, 4, 2, 4, 0, p["n_q"], 100000, 0, 0, group)
        with pytest.raises(fesc.FescError) as e:
            ctx.scan_contract(z, z, z, z, desc, z, z, z, z, [0], [0], z, masks)
        assert e.value.code == fesc.EINVAL


def test_scan_missing_key_is_reported():
    import torch
    import paper_2608_17442_b200 as fesc

    ctx, orc, p = ctx_pair("scan_toy")
    z = torch.zeros((1, 2, 2, 10, orc.N), dtype=torch.int64, device="cuda")
    desc = fesc.ScanDesc(4, 2, 4, 2, 4, 0, 10, 7000000)     # no keys under this base
    with pytest.raises(fesc.FescError) as e:
        ctx.scan_contract(z, z, z[0], z[0], desc, z, z, z, z, [0] * 121, [0] * 121, z)
    assert e.value.code == fesc.ENOKEY


@pytest.mark.parametrize("hoist,group,stride,l0", [(1, 0, 256, 24), (1, 4, 256, 24), (1, 4, 128, 24), (1, 4, 128, 22)])
def test_scan_deployed_geometry_decrypts_to_recurrence(hoist, group, stride, l0):
    """N = 2^16, 24 limbs, stride 256, B_blk = 256, d_s = 128, P = 64 (the Mamba-2-base geometry) on a slice of
    the model: 4 heads (one chunk pair) and 512 tokens (two blocks, so the carry and its injection run).
    The oracle cannot follow ~36 000 key switches at this ring size, so the check here is the property that
    holds at any size: the decrypted output equals the float64 recurrence within 2^-18 (|m| <= 1.5).  Residue-level
    parity on this ring, with a block of 4 tokens, is in test_gpu_scan_full_ring.py."""
    import time
    import torch
    import paper_2608_17442_b200 as fesc

    ctx, orc, p = ctx_pair("full")
    sh = ScanShape(orc.n, L=512, H=4 if stride == 256 else 8, P=64, d_s=128, B_blk=256, stride=stride)
    assert (sh.stride, sh.c_state, sh.hpc, sh.K_s, sh.K_blk, sh.segs) == ((256, 128, 2, 2, 2, 1) if stride == 256 else
                                                                         (128, 256, 4, 2, 2, 2))
    x, a, B, C = S.scan_inputs(S.config_seed(5), sh.L, sh.H, sh.P, 1, sh.d_s)
    c = ScanConsts(orc, sh, l0, 40, "bk", group)     # l0 = 22: inputs two limbs down, output at the last level
    assert c.lv == (dict(l0=l0, l1=l0 - 3, lS=l0 - 11, linj=l0 - 18, lout=l0 - 21) if group else
                    dict(l0=24, l1=22, lS=14, linj=7, lout=4))
    for r in sh.rotation_amounts(bool(hoist), group) + [CONJ]:
        ctx.add_galois_key(r, key_id_for(sh, r))
    ctX, ctA, ctB, ctC = encrypt_inputs(orc, sh, c, x, a, B, C)
    adj_s = [c.adj_s.get((s, d), 0) for s in range(l0 + 1) for d in range(l0 + 1)]
    adj_p = [c.adj_p.get((s, d), 0) for s in range(l0 + 1) for d in range(l0 + 1)]
    out = torch.empty((sh.K_blk, sh.K_s, sh.segs, 2, c.lv["lout"], orc.N), dtype=torch.int64, device="cuda")
    desc = fesc.ScanDesc(sh.L, sh.H, sh.P, sh.d_s, sh.B, sh.stride, l0, 100000, hoist, 0, group)
    gm = [to_dev(m) for m in (c.mask_xg, c.mask_ag, c.mask_x2, c.mask_a2, c.mask_bg, c.mask_b2)] if group else None
    args = (to_dev(ctX), to_dev(ctA), to_dev(ctB), to_dev(ctC), desc, to_dev(c.mask_x), to_dev(c.mask_b),
            to_dev(c.mask_a), to_dev(c.mask_out), adj_s, adj_p, out, gm)
    ks0 = ctx.counters()[1]
    torch.cuda.synchronize()
    t0 = time.perf_counter()
    ctx.scan_contract(*args)
    ctx.sync()
    dt = time.perf_counter() - t0
    ks = ctx.counters()[1] - ks0
    m = unpack_output(orc, sh, c, to_host(out))
    ref = float_recurrence(x, a, B, C)
    err = np.abs(m - ref).max()
    print("scan slice: %d key switches in %.2f s (%.0f /s), scratch %.1f GiB, max err 2^%.2f, max|m| %.2f"
          % (ks, dt, ks / dt, ctx.counters()[3] / 2**30, np.log2(err), np.abs(ref).max()))
    assert err < 2.0**-18
