"""Pins for the scan-contract oracle: the float64 recurrence against its closed form, the paper's
composition / reduction counts, and decrypt(scan(Enc factors)) against the recurrence on the paper's
toy shape (L=4, H=2, P=4, d_s=2, K_s=2) and on a 128-slot analogue of the Mamba-2-base geometry."""
import math

import numpy as np
import pytest

import fesc_synth as S
from oracle.ckks import Oracle
from oracle.scan import (ScanConsts, ScanEvaluator, ScanShape, add_scan_keys, closed_form_counts, encrypt_inputs, encrypt_x,
                         float_recurrence, float_recurrence_invariant, levels, unpack_output)


def test_recurrence_matches_unrolled_closed_form():
    x, a, B, C = S.scan_inputs(3, 9, 2, 3, 1, 4)
    m = float_recurrence(x, a, B, C)
    for k in (0, 4, 8):
        want = np.zeros((2, 3))
        for kp in range(k + 1):
            decay = np.prod(a[kp + 1:k + 1], axis=0)          # per head
            want += decay[:, None] * x[kp] * float(B[kp, 0] @ C[k, 0])
        assert np.allclose(m[k], want, rtol=1e-12, atol=1e-12)
    # one hand-checked step: h_0 = 0 so m_0 = x_0 (B_0 . C_0)
    assert np.allclose(m[0], x[0] * float(B[0, 0] @ C[0, 0]))


def _bk_nodes(B):
    """(stage kind, left, right) of every composition of the network, 1-based positions."""
    logB = int(math.log2(B))
    nodes = []
    for s in range(1, logB + 1):
        nodes += [("up", k - (1 << (s - 1)), k) for k in range(1 << s, B + 1, 1 << s)]
    for s in range(logB - 1, 0, -1):
        nodes += [("down", k, k + (1 << (s - 1))) for k in range(1 << s, B, 1 << s) if k + (1 << (s - 1)) < B]
    return nodes


@pytest.mark.parametrize("B", [4, 8, 16, 256])
def test_brent_kung_network_counts_and_prefixes(B):
    nodes = _bk_nodes(B)
    logB = int(math.log2(B))
    assert sum(1 for n in nodes if n[0] == "up") == B - 1                    # App. "Prefix-Network Selection"
    assert sum(1 for n in nodes if n[0] == "down") == B - 1 - logB
    assert len(nodes) == 2 * B - logB - 2                                    # C_BK(n) = 2n - log2 n - 2
    # the network computes every inclusive prefix: track covered intervals
    cover = {k: (k, k) for k in range(1, B + 1)}
    for _, l, r in nodes:
        assert cover[l][1] + 1 == cover[r][0]
        cover[r] = (cover[l][0], cover[r][1])
    assert all(cover[k] == (1, k) for k in range(1, B + 1))


def _ks_nodes(B):
    """Kogge-Stone stages (1-based positions): stage s, every k > 2^(s-1) combines with k - 2^(s-1)."""
    return [[(k - (1 << (s - 1)), k) for k in range((1 << (s - 1)) + 1, B + 1)] for s in range(1, int(math.log2(B)) + 1)]


def _sk_nodes(B):
    """Sklansky stages (1-based positions): the upper half of every aligned block of 2^s takes the lower half's last."""
    stages = []
    for s in range(1, int(math.log2(B)) + 1):
        h = 1 << (s - 1)
        stages.append([(b * 2 * h + h, k) for b in range(B >> s) for k in range(b * 2 * h + h + 1, (b + 1) * 2 * h + 1)])
    return stages


@pytest.mark.parametrize("B", [4, 8, 16, 256])
def test_kogge_stone_and_sklansky_counts_and_prefixes(B):
    logB = int(math.log2(B))
    for stages, total in ((_ks_nodes(B), B * logB - (B - 1)), (_sk_nodes(B), B // 2 * logB)):
        assert len(stages) == logB and sum(len(st) for st in stages) == total     # App. "Prefix-Network Selection"
        cover = {k: (k, k) for k in range(1, B + 1)}
        for st in stages:
            prev = dict(cover)                                 # both operands come from the previous stage
            for l, r in st:
                assert prev[l][1] + 1 == prev[r][0]
                cover[r] = (prev[l][0], prev[r][1])
        assert all(cover[k] == (1, k) for k in range(1, B + 1))
    assert [len(st) for st in _ks_nodes(B)] == [B - (1 << (s - 1)) for s in range(1, logB + 1)]
    assert all(len(st) == B // 2 for st in _sk_nodes(B))


def _golden(name):
    import os
    path = os.path.join(os.path.dirname(__file__), "golden", name)
    return [[float(v) for v in line.split()] for line in open(path) if line.strip() and not line.startswith("#")]


def test_paper_ledger_values():
    # Table "real-phantom-scan": compositions of each prefix network over L' positions, times 2 K_s key switches
    for Lp, seq_k, seq_d, ks_k, ks_d, skl_k, skl_d, bk_k, bk_d in _golden("real_phantom_scan.txt"):
        Lp, lg = int(Lp), int(math.log2(Lp))
        counts = {"seq": Lp - 1, "ks": Lp * lg - (Lp - 1), "skl": Lp // 2 * lg, "bk": 2 * (Lp - 1) - lg}
        for key, printed in (("seq", seq_k), ("ks", ks_k), ("skl", skl_k), ("bk", bk_k)):
            assert abs(2 * 12 * counts[key] / 1e3 - printed) <= 0.0501, (Lp, key)
        assert (seq_d, ks_d, skl_d, bk_d) == (Lp - 1, lg, lg, 2 * lg - 1)
        assert counts["bk"] == len(_bk_nodes(Lp))                              # the network this build evaluates
    (d_s, K_s, printed), = _golden("cross_ssm_family.txt")
    assert (d_s, K_s) == (128, 12) and 2 * 12 * (2 * 127 - 7) == printed
    assert 2 * 12 * (2 * 127 - 7) == 5928                                     # Table "cross_ssm_family", Mamba-2
    # depth 2 ceil(log2 L') - 1
    assert [2 * int(math.log2(Lp)) - 1 for Lp in (128, 256, 512, 1024, 2048)] == [13, 15, 17, 19, 21]
    # K_s and reduction counts of the deployed shape (App. "Complex-Packed Reduction Accounting")
    assert math.ceil(1536 * 128 / 16384) == 12
    sh = ScanShape(32768, L=2048, H=24, P=64, d_s=128, B_blk=256)
    assert (sh.K_s, sh.K_blk, sh.c_state, sh.hpc, sh.stride) == (12, 8, 128, 2, 256)
    cf = closed_form_counts(sh)
    assert cf["reduce_rot"] == 86016 and cf["reduce_conj"] == 12288
    assert cf["compose"] == 96 * 502
    lv = levels(24, sh.logB, sh.K_blk)
    assert lv == dict(l0=24, l1=22, lS=14, linj=7, lout=4)
    assert 2 * 768 // 768 and 2 * 24 * 64 + 2 * 128 + 24 == 3352              # d_out of in_proj


def _run(name, hoist=False, network="bk", group=0, **shape_kw):
    p = S.params(name)
    orc = Oracle(p["log_n"], p["primes"], p["n_q"], p["n_p"], p["dnum"], p["seed"])
    sh = ScanShape(orc.n, **shape_kw)
    x, a, B, C = S.scan_inputs(p["seed"], sh.L, sh.H, sh.P, 1, sh.d_s)
    c = ScanConsts(orc, sh, p["n_q"], p["log_scale"], network, group)
    add_scan_keys(orc, sh, hoist=hoist, group=group)
    ev = ScanEvaluator(orc, sh, c, hoist=hoist)
    out = ev.run(*encrypt_inputs(orc, sh, c, x, a, B, C))
    return sh, ev, unpack_output(orc, sh, c, out), float_recurrence(x, a, B, C)


def test_paper_toy_shape():
    sh, ev, m, ref = _run("scan_toy", L=4, H=2, P=4, d_s=2, B_blk=4)
    assert sh.K_s == 2 and ev.count["compose"] == closed_form_counts(sh)["compose"] == 8
    assert ev.count["conj"] == closed_form_counts(sh)["reduce_conj"]
    assert np.abs(m - ref).max() < 2.0**-24


def test_analogue_with_carries_and_partial_block():
    sh, ev, m, ref = _run("scan_small", L=40, H=8, P=4, d_s=8, B_blk=16)
    cf = closed_form_counts(sh)
    assert (sh.K_s, sh.K_blk, sh.hpc) == (4, 3, 2)
    assert ev.count["compose"] == cf["compose"] == 312 and ev.count["conj"] == cf["reduce_conj"] == 96
    assert np.abs(m - ref).max() < 2.0**-22


def test_two_digit_offsets_and_odd_chunk_count():
    sh, ev, m, ref = _run("scan_small", L=64, H=3, P=4, d_s=4, B_blk=32)
    assert (sh.K_s, sh.K_blk, sh.dg, sh.hpc) == (3, 2, 16, 1)
    assert ev.count["conj"] == closed_form_counts(sh)["reduce_conj"] == 64
    assert np.abs(m - ref).max() < 2.0**-22


def test_hoisted_mode_same_values():
    """Radix-4 rotate-and-add chains (three rotations per two steps, one decomposition and one division by P) and
    hoisted low-digit extraction: every other count is unchanged and the decrypted contract output stays within the
    plain mode's bound."""
    sh, ev, m, ref = _run("scan_toy", hoist=True, L=4, H=2, P=4, d_s=2, B_blk=4)
    _, ev0, m0, _ = _run("scan_toy", L=4, H=2, P=4, d_s=2, B_blk=4)
    assert {k: v for k, v in ev.count.items() if k != "rot"} == {k: v for k, v in ev0.count.items() if k != "rot"}
    assert ev.count["rot"] > ev0.count["rot"]
    assert np.abs(m - ref).max() < 2.0**-24 and np.abs(m - m0).max() < 2.0**-24
    sh, ev, m, ref = _run("scan_small", hoist=True, L=64, H=3, P=4, d_s=4, B_blk=32)
    assert (sh.K_s, sh.K_blk, sh.dg) == (3, 2, 16)
    assert np.abs(m - ref).max() < 2.0**-22


@pytest.mark.parametrize("network", ["ks", "sk"])
def test_other_prefix_networks(network):
    """Kogge-Stone and Sklansky networks (App. "Prefix-Network Selection"): composition counts of the closed forms,
    the shallower level schedule, and the same contract output as the recurrence (toy shape; analogue with carries
    over three blocks and a partial last block)."""
    sh, ev, m, ref = _run("scan_toy", network=network, L=4, H=2, P=4, d_s=2, B_blk=4)
    assert ev.count["compose"] == closed_form_counts(sh, network)["compose"] == {"ks": 10, "sk": 8}[network]
    assert np.abs(m - ref).max() < 2.0**-24
    sh, ev, m, ref = _run("scan_small", network=network, L=40, H=8, P=4, d_s=8, B_blk=16)
    per_block = {"ks": 16 * 4 - 15, "sk": 8 * 4}[network]
    assert ev.count["compose"] == closed_form_counts(sh, network)["compose"] == 12 * per_block
    assert ev.c.lv["linj"] == ev.c.lv["lS"] - 1 and ev.c.lv["lout"] == ev.c.lv["linj"] - 3
    assert np.abs(m - ref).max() < 2.0**-22
    # deployed shape: depth log2 B instead of 2 log2 B - 1
    assert levels(24, 8, 8, network) == dict(l0=24, l1=22, lS=14, linj=8, lout=5)


def test_grouped_leaf_build():
    """Leaves built for groups of G tokens (one extraction, mask and fill per group, then every token as a masked sum
    of the group's 2(G-1) rotations): same contract output, same compositions, one level more, and exactly the
    rotations the closed form predicts fewer."""
    kw = dict(L=40, H=8, P=4, d_s=8, B_blk=16)
    sh, ev0, m0, ref = _run("scan_small", **kw)
    _, ev, m, _ = _run("scan_small", group=4, **kw)
    assert np.abs(m - ref).max() < 2.0**-22 and np.abs(m - m0).max() < 2.0**-22
    assert ev.c.lv == dict(l0=16, l1=13, lS=9, linj=6, lout=3) and ev0.c.lv["l1"] == 14
    assert ev.count["compose"] == ev0.count["compose"] and ev.count["ctmul"] == ev0.count["ctmul"]
    lg = lambda v: int(math.log2(v))
    B, G, P, R, d_s = sh.B, 4, sh.P, sh.R, sh.d_s
    plain = 2 * (B - 1) + B * (lg(d_s) + lg(R // P))
    grouped = 2 * (B // G - 1) + (B // G) * (lg(d_s // G) + lg(R // (G * P))) + 2 * (B // G) * 2 * (G - 1)
    # br(B) of every block (shared by the chunks) is built in groups too
    plain_b = (B - 1) + B * lg(sh.c_state)
    grouped_b = (B // G - 1) + (B // G) * lg(sh.n // (G * d_s)) + (B // G) * 2 * (G - 1)
    assert ev0.count["rot"] - ev.count["rot"] == sh.K_blk * (sh.K_s * (plain - grouped) + plain_b - grouped_b) == 996
    assert ev.count["ptmul"] - ev0.count["ptmul"] == sh.K_blk * (sh.K_s * (2 * (B // G) + 2 * B * G - 2 * B)
                                                                 + B // G + B * G - B)
    # the rotated copy kept for the class difference k = g - j is the rotation by k units
    for G in (2, 4, 8):
        shifts = sh.class_shifts(G, 3)
        assert len(set(shifts)) == 2 * (G - 1)
        for k in range(-(G - 1), G):
            if k:
                assert shifts[k - 1 if k > 0 else G - 2 - k] == 3 * k
    # deployed shape: 1 598 instead of 4 350 extraction and fill rotations per (block, chunk)
    big = ScanShape(32768, L=2048, H=24, P=64, d_s=128, B_blk=256)
    B, G, P, R, d_s = 256, 4, 64, big.R, 128
    assert 2 * (B - 1) + B * (lg(d_s) + lg(R // P)) == 4350
    assert 2 * (B // G - 1) + (B // G) * (lg(d_s // G) + lg(R // (G * P))) + 2 * (B // G) * 2 * (G - 1) == 1598
    assert levels(24, 8, 8, "bk", 4) == dict(l0=24, l1=21, lS=13, linj=6, lout=3)


def test_grouped_leaf_build_other_shapes_and_hoisted_rotations():
    sh, ev, m, ref = _run("scan_toy", group=2, L=4, H=2, P=4, d_s=2, B_blk=4)
    assert np.abs(m - ref).max() < 2.0**-24
    sh, ev, m, ref = _run("scan_small", hoist=True, group=4, L=64, H=3, P=4, d_s=4, B_blk=32)
    assert (sh.K_s, sh.K_blk) == (3, 2) and np.abs(m - ref).max() < 2.0**-22
    sh, ev, m, ref = _run("scan_small", network="sk", group=2, L=40, H=8, P=4, d_s=8, B_blk=16)
    assert np.abs(m - ref).max() < 2.0**-22


def test_full_slot_variant_with_token_segments():
    """stride = d_s < B_blk: every slot of a state ciphertext carries a state coordinate (s_state = n), a block's tokens
    come in B_blk/stride segments with one x / a / output ciphertext each, and half as many chunks do the same work."""
    kw = dict(L=40, H=8, P=4, d_s=8, B_blk=16)
    sh0, ev0, m0, ref = _run("scan_small", **kw)
    sh, ev, m, _ = _run("scan_small", stride=8, **kw)
    assert (sh0.K_s, sh0.segs, sh0.hpc) == (4, 1, 2) and (sh.K_s, sh.segs, sh.Bt, sh.hpc, sh.R) == (2, 2, 8, 4, 32)
    assert np.abs(m - ref).max() < 2.0**-22 and np.abs(m - m0).max() < 2.0**-22
    assert ev.count["compose"] == closed_form_counts(sh)["compose"] == ev0.count["compose"] // 2
    assert ev.count["ctmul"] == ev0.count["ctmul"] // 2 and ev.count["conj"] == ev0.count["conj"] // 2
    # with the grouped leaf build and hoisted rotations on top
    _, _, m, _ = _run("scan_small", hoist=True, group=4, stride=8, **kw)
    assert np.abs(m - ref).max() < 2.0**-22
    # deployed ring: K_s = 6 chunks of 4 heads, two segments of 128 tokens
    big = ScanShape(32768, L=2048, H=24, P=64, d_s=128, B_blk=256, stride=128)
    assert (big.K_s, big.segs, big.Bt, big.c_state, big.hpc, big.R) == (6, 2, 128, 256, 4, 8192)


# ---------------------------------------------------------------------------------------------------------------------
# invariant families (App. "Invariant Families"): plaintext decay, input factor and output factor
# ---------------------------------------------------------------------------------------------------------------------
def _invariant_factors(seed, d_s):
    g = S.rng(seed, 300)
    return g.uniform(0.9, 1.0, d_s), g.standard_normal(d_s) * 0.5, g.standard_normal(d_s) * 0.5


def test_invariant_recurrence_closed_form_and_reduction_to_the_selective_one():
    x, _, _, _ = S.scan_inputs(5, 11, 2, 3, 1, 4)
    abar, Bbar, Cbar = _invariant_factors(5, 4)
    m = float_recurrence_invariant(x, abar, Bbar, Cbar)
    # unrolled: m_k[e] = sum_i Cbar_i Bbar_i sum_{j<=k} abar_i^(k-j) x_j[e]
    for k in (0, 3, 10):
        want = sum((Cbar * Bbar * abar ** (k - j)).sum() * x[j] for j in range(k + 1))
        assert np.allclose(m[k], want, rtol=1e-12, atol=1e-12)
    # a decay that is the same for every state coordinate is the selective recurrence with constant factors
    alpha = 0.93
    a = np.full((11, 2), alpha)
    Bk, Ck = np.tile(Bbar, (11, 1, 1)), np.tile(Cbar, (11, 1, 1))
    assert np.allclose(float_recurrence_invariant(x, np.full(4, alpha), Bbar, Cbar), float_recurrence(x, a, Bk, Ck),
                       rtol=1e-12, atol=1e-12)


def _run_plain(name, hoist=False, group=0, **shape_kw):
    p = S.params(name)
    orc = Oracle(p["log_n"], p["primes"], p["n_q"], p["n_p"], p["dnum"], p["seed"])
    sh = ScanShape(orc.n, **shape_kw)
    x, _, _, _ = S.scan_inputs(p["seed"], sh.L, sh.H, sh.P, 1, sh.d_s)
    fac = _invariant_factors(p["seed"], sh.d_s)
    c = ScanConsts(orc, sh, p["n_q"], p["log_scale"], "bk", group, plain=fac)
    add_scan_keys(orc, sh, hoist=hoist, group=group)
    ev = ScanEvaluator(orc, sh, c, hoist=hoist)
    out = ev.run_plain(encrypt_x(orc, sh, c, x))
    return sh, ev, unpack_output(orc, sh, c, out), float_recurrence_invariant(x, *fac)


def test_invariant_scan_matches_the_recurrence_without_any_ciphertext_product():
    """Toy shape; three blocks with carries and a partial last block; grouped leaves with hoisted rotations; every slot
    in use with token segments.  No relinearisation anywhere (the table's "Affine relin." 0), the Brent-Kung
    composition count of the selective scan, and fewer rotations (no br(a), br(B), br(C))."""
    sh, ev, m, ref = _run_plain("scan_toy", L=4, H=2, P=4, d_s=2, B_blk=4)
    assert ev.count["ctmul"] == 0 and ev.count["compose"] == closed_form_counts(sh)["compose"] == 8
    assert np.abs(m - ref).max() < 2.0**-24
    kw = dict(L=40, H=8, P=4, d_s=8, B_blk=16)
    sh, ev, m, ref = _run_plain("scan_small", **kw)
    cf = closed_form_counts(sh)
    assert ev.count["ctmul"] == 0 and ev.count["compose"] == cf["compose"] == 312
    assert ev.count["conj"] == cf["reduce_conj"] == 96
    lg = lambda v: int(math.log2(v))
    # rotations: extraction and fill of br(x_t), state-axis reduction, output placement; nothing for a, B, C
    extract_fill = sh.K_blk * sh.K_s * ((sh.B - 1) + sh.B * lg(sh.d_s))
    assert ev.count["rot"] == extract_fill + cf["reduce_rot"] + sh.K_blk * sh.K_s * (sh.B - 1)
    assert np.abs(m - ref).max() < 2.0**-22
    _, ev_g, m_g, _ = _run_plain("scan_small", hoist=True, group=4, **kw)
    assert ev_g.count["ctmul"] == 0 and np.abs(m_g - ref).max() < 2.0**-22
    sh2, ev2, m2, _ = _run_plain("scan_small", hoist=True, group=4, stride=8, **kw)
    assert (sh2.K_s, sh2.segs) == (2, 2) and ev2.count["ctmul"] == 0 and np.abs(m2 - ref).max() < 2.0**-22


def test_invariant_rows_of_the_paper_table():
    """Table "cross_ssm_family", S4D / S5 / LRU rows: d_s, K_s at E = 1536 channels, and 0 affine relinearisations."""
    import os
    path = os.path.join(os.path.dirname(__file__), "golden", "cross_ssm_family.txt")
    rows = [[int(v) for v in line.split()[1:]] for line in open(path) if line.startswith("#inv")]
    assert rows == [[64, 6, 0], [128, 12, 0], [128, 12, 0]]
    # the paper's state chunks hold s_state = 16384 = n/2 slots: K_s = E d_s / s_state
    for d_s, K_s, relin in rows:
        assert 1536 * d_s // 16384 == K_s and relin == 0
    # this build's layouts at L = 128: S4D (d_s = 64) with one block of 128 tokens, S5 / LRU (d_s = 128) with stride 256
    assert ScanShape(32768, L=128, H=24, P=64, d_s=64, B_blk=128).K_s == 6
    assert ScanShape(32768, L=128, H=24, P=64, d_s=128, B_blk=128, stride=256).K_s == 12
