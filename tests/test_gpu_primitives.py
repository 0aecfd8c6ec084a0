"""GPU parity: key generation, NTT, ct-pt MAC, rotation, rescale and ct x ct must equal the
oracle's residues bit for bit on the same seeded inputs."""
import numpy as np
import pytest

import fesc_synth as S
from tests.gpu_util import add_key, ctx_pair, random_ct, to_dev, to_host

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("name", ["toy", "tiny", "small"])
def test_keygen_matches_oracle(name):
    pair = ctx_pair(name)
    ctx, orc, _ = pair
    assert np.array_equal(to_host(ctx.export_secret()), orc.s_eval)
    assert np.array_equal(to_host(ctx.export_key(0)), orc.keys[0][1])
    add_key(pair, 3, 7)
    add_key(pair, -(1 << 31), 8)
    assert np.array_equal(to_host(ctx.export_key(7)), orc.keys[7][1])
    assert np.array_equal(to_host(ctx.export_key(8)), orc.keys[8][1])


@pytest.mark.parametrize("name", ["toy", "tiny", "small"])
def test_ntt_small_rings(name):
    ctx, orc, p = ctx_pair(name)
    idx = list(range(p["n_q"] + p["n_p"]))
    batch = 3
    a = np.stack([S.uniform_residues_np(1, b, orc.q, orc.N) for b in range(batch)])
    d = to_dev(a)
    ctx.ntt(d, batch, 0, len(idx))
    want = np.stack([orc.ntt(a[b], idx) for b in range(batch)])
    assert np.array_equal(to_host(d), want)
    ctx.intt(d, batch, 0, len(idx))
    assert np.array_equal(to_host(d), a)
    # a sub-range of limbs starting at 1, inverse direction against the oracle
    sub = idx[1:4]
    b2 = np.ascontiguousarray(a[:, 1:4])
    d2 = to_dev(b2)
    ctx.intt(d2, batch, 1, 3)
    assert np.array_equal(to_host(d2), np.stack([orc.intt(b2[b], sub) for b in range(batch)]))


def test_ntt_full_ring_matches_oracle():
    ctx, orc, p = ctx_pair("full")
    idx = [0, 7, 23, 24, 27]   # 50-bit and 60-bit primes
    a = np.stack([S.uniform_residues_np(2, 0, [orc.q[i]], orc.N)[0] for i in idx])
    for i, pi in enumerate(idx):
        d = to_dev(a[i:i + 1])
        ctx.ntt(d, 1, pi, 1)
        assert np.array_equal(to_host(d)[0], orc.ntt(a[i:i + 1], [pi])[0]), pi
        ctx.intt(d, 1, pi, 1)
        assert np.array_equal(to_host(d)[0], a[i])
        d = to_dev(a[i:i + 1])
        ctx.intt(d, 1, pi, 1)
        assert np.array_equal(to_host(d)[0], orc.intt(a[i:i + 1], [pi])[0]), pi


def test_ntt_sweep_workload_round_trip():
    """Workload 2: 64 polynomials x 24 limbs of 50-bit primes at N = 2^16; forward then inverse is the
    identity bit for bit, and sampled limbs of the forward transform equal the oracle's."""
    import torch

    ctx, orc, p = ctx_pair("full")
    x = S.hashed_residues(S.config_seed(2), 0, orc.q[:24], 64 * orc.N, device="cuda")  # [24, 64*N]
    x = x.view(24, 64, orc.N).permute(1, 0, 2).contiguous()
    y = x.clone()
    ctx.ntt(y, 64, 0, 24)
    for (b, l) in ((0, 0), (17, 5), (63, 23)):
        assert np.array_equal(to_host(y[b, l]), orc.ntt(to_host(x[b, l])[None], [l])[0])
    ctx.intt(y, 64, 0, 24)
    assert torch.equal(x, y)


@pytest.mark.parametrize("name,level", [("toy", 6), ("toy", 3), ("tiny", 3), ("small", 24)])
def test_ct_pt_mac(name, level):
    ctx, orc, _ = ctx_pair(name)
    batch = 4
    ct = random_ct(orc, 3, 0, level, batch)
    acc = random_ct(orc, 3, 1, level, batch)
    pt = np.stack([S.uniform_residues_np(3, 9000 + b, orc.q[:level], orc.N) for b in range(batch)])
    d_acc = to_dev(acc)
    ctx.ct_pt_mac(to_dev(ct), to_dev(pt), d_acc, batch, level)
    want = np.stack([orc.ct_pt_mac(ct[b], pt[b], acc[b]) for b in range(batch)])
    assert np.array_equal(to_host(d_acc), want)
    # one plaintext shared by the batch
    d_acc = to_dev(acc)
    ctx.ct_pt_mac(to_dev(ct), to_dev(pt[0]), d_acc, batch, level, pt_stride=0)
    want = np.stack([orc.ct_pt_mac(ct[b], pt[0], acc[b]) for b in range(batch)])
    assert np.array_equal(to_host(d_acc), want)


def _check_rotate(name, level, batch, rot, key_id):
    import torch

    pair = ctx_pair(name)
    ctx, orc, _ = pair
    add_key(pair, rot, key_id)
    ct = random_ct(orc, 4, level * 100 + key_id, level, batch)
    out = torch.empty_like(to_dev(ct))
    ctx.rotate(to_dev(ct), out, batch, level, key_id)
    got = to_host(out)
    for b in range(batch):
        assert np.array_equal(got[b], orc.rotate(ct[b], key_id)), (name, level, b)


@pytest.mark.parametrize("level", [6, 5, 4, 3, 2, 1])
def test_rotate_toy_all_levels(level):
    _check_rotate("toy", level, 3, 1, 11)
    _check_rotate("toy", level, 2, -(1 << 31), 12)


def test_rotate_tiny():
    _check_rotate("tiny", 3, 4, 1, 21)
    _check_rotate("tiny", 3, 4, 5, 22)
    _check_rotate("tiny", 2, 1, 5, 22)


@pytest.mark.parametrize("level", [24, 23, 21, 9, 1])
def test_rotate_small_ring_full_limb_structure(level):
    _check_rotate("small", level, 5, 8, 31)


@pytest.mark.parametrize("name,level,batch", [("full", 24, 2), ("full", 22, 1), ("full_literal", 24, 1)])
def test_rotate_full_ring(name, level, batch):
    _check_rotate(name, level, batch, 8, 41)


@pytest.mark.parametrize("name,level", [("toy", 6), ("toy", 2), ("tiny", 3), ("small", 24), ("small", 10)])
def test_rescale(name, level):
    import torch

    ctx, orc, _ = ctx_pair(name)
    batch = 3
    ct = random_ct(orc, 5, level, level, batch)
    out = torch.empty((batch, 2, level - 1, orc.N), dtype=torch.int64, device="cuda")
    ctx.rescale(to_dev(ct), out, batch, level)
    got = to_host(out)
    for b in range(batch):
        assert np.array_equal(got[b], orc.rescale(ct[b]))


@pytest.mark.parametrize("name,level", [("toy", 6), ("toy", 3), ("small", 24), ("small", 6)])
def test_ct_ct_mul(name, level):
    import torch

    ctx, orc, _ = ctx_pair(name)
    batch = 3
    a = random_ct(orc, 6, level, level, batch)
    b_ = random_ct(orc, 6, level + 50, level, batch)
    out = torch.empty_like(to_dev(a))
    ctx.ct_ct_mul(to_dev(a), to_dev(b_), out, batch, level)
    got = to_host(out)
    for b in range(batch):
        assert np.array_equal(got[b], orc.ct_ct_mul(a[b], b_[b]))


def test_full_ring_rescale_and_ctmul():
    import torch

    ctx, orc, _ = ctx_pair("full")
    a = random_ct(orc, 7, 0, 24, 1)
    b_ = random_ct(orc, 7, 1, 24, 1)
    out = torch.empty_like(to_dev(a))
    ctx.ct_ct_mul(to_dev(a), to_dev(b_), out, 1, 24)
    want = orc.ct_ct_mul(a[0], b_[0])
    assert np.array_equal(to_host(out)[0], want)
    res = torch.empty((1, 2, 23, orc.N), dtype=torch.int64, device="cuda")
    ctx.rescale(out, res, 1, 24)
    assert np.array_equal(to_host(res)[0], orc.rescale(want))


def test_error_codes():
    import torch
    import paper_2608_17442_b200 as fesc

    ctx, orc, p = ctx_pair("toy")
    ct = to_dev(random_ct(orc, 8, 0, 6, 1))
    out = torch.empty_like(ct)
    with pytest.raises(fesc.FescError) as e:
        ctx.rotate(ct, out, 1, 6, 999)
    assert e.value.code == fesc.ENOKEY
    with pytest.raises(fesc.FescError) as e:
        ctx.rescale(ct, out, 1, 1)
    assert e.value.code == fesc.ELEVEL
    with pytest.raises(fesc.FescError) as e:
        fesc.Context(6, [97, 193, 257], 2, 1, 2, 1)   # not = 1 mod 2N
    assert e.value.code == fesc.EINVAL


def test_empty_batches_and_rejected_arguments():
    """Empty batches are no-ops that leave the outputs untouched; impossible shapes are refused before any launch."""
    import torch
    import paper_2608_17442_b200 as fesc

    pair = ctx_pair("toy")
    ctx, orc, p = pair
    add_key(pair, 1, 91)
    ct = to_dev(random_ct(orc, 9, 0, 6, 2))
    out = torch.full_like(ct, 7)
    ctx.ntt(ct, 0, 0, 6)
    ctx.intt(ct, 0, 0, 6)
    ctx.rotate(ct, out, 0, 6, 91)
    ctx.rotate_hoisted(ct, out, 0, 6, [91])
    ctx.rotate_sum_hoisted(ct, out, 0, 6, [91])
    ctx.ct_pt_mac(ct, ct[:, 0].contiguous(), out, 0, 6)
    ctx.rescale(ct, out, 0, 6)
    ctx.ct_ct_mul(ct, ct, out, 0, 6)
    ctx.sync()
    assert bool((out == 7).all())
    for bad in (lambda: ctx.ntt(ct, 1, 5, 9),                                   # limbs past the last prime
                lambda: ctx.rotate(ct, out, 1, 99, 91),                         # level above n_q
                lambda: ctx.rotate_sum_hoisted(ct, out, 1, 6, [91] * 9),        # more than 8 keys
                lambda: ctx.linear(ct, ct, fesc.BsgsDesc(0, 1, 1, 1, 1, 6, 1, 1), out),
                lambda: ctx.linear(ct, ct, fesc.BsgsDesc(2, 2, 1, 1, 1, 1, 1, 1), out),      # level 1 cannot rescale
                lambda: ctx.conv(ct, ct, ct, fesc.ConvDesc(9, 8, 1, 1, 6, 1), out),          # more than 8 taps
                lambda: ctx.conv(ct, ct, ct, fesc.ConvDesc(2, 5, 1, 1, 6, 1), out)):         # T does not divide the slots
        with pytest.raises(fesc.FescError) as e:
            bad()
        assert e.value.code in (fesc.EINVAL, fesc.ELEVEL)
    # one limb: transforms and multiply-accumulate still work
    one = to_dev(random_ct(orc, 10, 0, 1, 1))
    ref = to_host(one).copy()
    ctx.intt(one, 2, 0, 1)
    ctx.ntt(one, 2, 0, 1)
    assert np.array_equal(to_host(one), ref)


def test_bounded_wait_runs_out_and_is_reported():
    """A device-side wait that nothing completes gives up after its poll budget: the next sync reports
    FESC_ETIMEOUT once, and the context keeps working (no fault, no hang)."""
    import torch
    import paper_2608_17442_b200 as fesc

    ctx, orc, p = ctx_pair("toy")
    ctx.sync()
    ctx.selftest_wait_limit()
    with pytest.raises(fesc.FescError) as e:
        ctx.sync()
    assert e.value.code == fesc.ETIMEOUT
    ctx.sync()                                          # the status word was cleared
    data = to_dev(random_ct(orc, 14, 0, 6, 1))
    ref = to_host(data).copy()
    ctx.intt(data, 2, 0, 6)
    ctx.ntt(data, 2, 0, 6)
    ctx.sync()
    assert np.array_equal(to_host(data), ref)


@pytest.mark.parametrize("level", [1, 2, 3, 4, 5, 7, 8, 13, 21, 23])
def test_key_switch_paths_at_every_digit_shape(level):
    """Levels that leave a partial last digit, a single digit or a single limb, with batches of 1 to 6 ciphertexts
    (every per-thread batch tile of the inner product): plain, hoisted and rotate-and-add rotations, ct x ct and
    rescale against the oracle."""
    import torch

    pair = ctx_pair("small")
    ctx, orc, _ = pair
    for r, kid in ((2, 95), (-7, 96)):
        add_key(pair, r, kid)
    batch = 1 + level % 6
    ct = random_ct(orc, 15, level, level, batch)
    other = random_ct(orc, 16, level, level, batch)
    dev = to_dev(ct)
    out = torch.empty_like(dev)
    ctx.rotate(dev, out, batch, level, 95)
    rot = to_host(out)
    hout = torch.empty((2, batch, 2, level, orc.N), dtype=torch.int64, device="cuda")
    ctx.rotate_hoisted(dev, hout, batch, level, [95, 96])
    hrot = to_host(hout)
    ctx.rotate_sum_hoisted(dev, out, batch, level, [95, 96])
    srot = to_host(out)
    ctx.ct_ct_mul(dev, to_dev(other), out, batch, level)
    prod = to_host(out)
    for b in range(batch):
        assert np.array_equal(rot[b], orc.rotate(ct[b], 95)), (level, b)
        want = orc.rotate_hoisted(ct[b], [95, 96])
        assert np.array_equal(hrot[0, b], want[0]) and np.array_equal(hrot[1, b], want[1]), (level, b)
        assert np.array_equal(srot[b], orc.rotate_sum_hoisted(ct[b], [95, 96])), (level, b)
        assert np.array_equal(prod[b], orc.ct_ct_mul(ct[b], other[b])), (level, b)
    if level >= 2:
        res = torch.empty((batch, 2, level - 1, orc.N), dtype=torch.int64, device="cuda")
        ctx.rescale(dev, res, batch, level)
        got = to_host(res)
        for b in range(batch):
            assert np.array_equal(got[b], orc.rescale(ct[b])), (level, b)


@pytest.mark.parametrize("level,batch", [(4, 5), (7, 3), (14, 2)])
def test_full_ring_low_levels(level, batch):
    """N = 2^16 at the low levels the scan-contract works at (injection, reduction, output): rotations in all three
    modes, ct x ct and rescale against the oracle."""
    import torch

    pair = ctx_pair("full")
    ctx, orc, _ = pair
    for r, kid in ((1, 97), (-16, 98)):
        add_key(pair, r, kid)
    ct = random_ct(orc, 17, level, level, batch)
    other = random_ct(orc, 18, level, level, batch)
    dev = to_dev(ct)
    out = torch.empty_like(dev)
    ctx.rotate(dev, out, batch, level, 97)
    rot = to_host(out)
    ctx.rotate_sum_hoisted(dev, out, batch, level, [97, 98])
    srot = to_host(out)
    ctx.ct_ct_mul(dev, to_dev(other), out, batch, level)
    prod = to_host(out)
    res = torch.empty((batch, 2, level - 1, orc.N), dtype=torch.int64, device="cuda")
    ctx.rescale(dev, res, batch, level)
    resc = to_host(res)
    for b in range(batch):
        assert np.array_equal(rot[b], orc.rotate(ct[b], 97)), (level, b)
        assert np.array_equal(srot[b], orc.rotate_sum_hoisted(ct[b], [97, 98])), (level, b)
        assert np.array_equal(prod[b], orc.ct_ct_mul(ct[b], other[b])), (level, b)
        assert np.array_equal(resc[b], orc.rescale(ct[b])), (level, b)


def test_workload_1_end_to_end():
    """Tiny CKKS: 4 ciphertexts x random plaintext vector, rotate by +1 and +5, decrypt; residues
    bit-exact and slots within 2^-16 of the float64 result."""
    import torch

    pair = ctx_pair("tiny")
    ctx, orc, p = pair
    add_key(pair, 1, 101)
    add_key(pair, 5, 105)
    scale = 2.0**30
    z = S.uniform_slots(p["seed"], 0, 4, orc.n)
    w = S.uniform_slots(p["seed"], 1, 4, orc.n)
    cts = np.stack([orc.encrypt(orc.encode(z[i], scale, 3), i) for i in range(4)])
    pts = np.stack([orc.encode(w[i], scale, 3) for i in range(4)])
    prod = torch.zeros((4, 2, 3, orc.N), dtype=torch.int64, device="cuda")
    ctx.ct_pt_mac(to_dev(cts), to_dev(pts), prod, 4, 3)
    for key_id, r in ((101, 1), (105, 5)):
        out = torch.empty_like(prod)
        ctx.rotate(prod, out, 4, 3, key_id)
        got = to_host(out)
        for i in range(4):
            want = orc.rotate(orc.ct_pt_mac(cts[i], pts[i], np.zeros_like(cts[i])), key_id)
            assert np.array_equal(got[i], want)
            slots = orc.decrypt(got[i], scale * scale)
            assert np.abs(slots - np.roll(z[i] * w[i], -r)).max() < 2.0**-16


def test_workload_3_rotations_full_ring():
    """Key-switch / rotation workload: N = 2^16, 24 x 50-bit limbs + 4 x 60-bit special primes, 6 digits;
    32 ciphertexts of U[-1,1] slots at scale 2^40; 16 key slots (baby steps 1..8, giant steps 8*{1..8}).
    Every rotation of the batch is decrypted and compared with the float64 shift (2^-18); four sampled
    (ciphertext, key) pairs are compared with the oracle bit for bit."""
    import torch

    pair = ctx_pair("full")
    ctx, orc, p = pair
    amounts = list(range(1, 9)) + [8 * g for g in range(1, 9)]
    scale = 2.0**40
    z = S.uniform_slots(S.config_seed(3), 0, 32, orc.n)
    cts = np.stack([orc.encrypt(orc.encode(z[i], scale, 24), 3000 + i) for i in range(32)])
    d_in = to_dev(cts)
    out = torch.empty_like(d_in)
    sampled = {(0, 0), (7, 5), (19, 8), (31, 15)}
    worst = 0.0
    for k, r in enumerate(amounts):
        key_id = 300 + k
        ctx.add_galois_key(r, key_id)
        ctx.rotate(d_in, out, 32, 24, key_id)
        got = to_host(out)
        for i in range(32):
            worst = max(worst, np.abs(orc.decrypt(got[i], scale, 2).real - np.roll(z[i], -r)).max())
            if (i, k) in sampled:
                if key_id not in orc.keys:
                    orc.add_galois_key(r, key_id)
                assert np.array_equal(got[i], orc.rotate(cts[i], key_id)), (i, k)
    print("workload 3: max |decrypt - shift| = 2^%.2f over 512 rotations" % np.log2(worst))
    assert worst < 2.0**-18


@pytest.mark.parametrize("name,level,batch", [("toy", 6, 3), ("toy", 5, 2), ("small", 24, 5), ("small", 9, 2), ("full", 24, 2)])
def test_rotate_hoisted(name, level, batch):
    """Hoisted mode: one decomposition per ciphertext, several keys; residues equal the oracle's hoisted mode."""
    import torch

    pair = ctx_pair(name)
    ctx, orc, _ = pair
    rots = [(1, 51), (7, 52), (-(1 << 31), 53)]
    for r, kid in rots:
        add_key(pair, r, kid)
    ct = random_ct(orc, 11, level, level, batch)
    out = torch.empty((len(rots), batch, 2, level, orc.N), dtype=torch.int64, device="cuda")
    ctx.rotate_hoisted(to_dev(ct), out, batch, level, [k for _, k in rots])
    got = to_host(out)
    for b in range(batch):
        want = orc.rotate_hoisted(ct[b], [k for _, k in rots])
        for k in range(len(rots)):
            assert np.array_equal(got[k, b], want[k]), (name, level, b, k)


@pytest.mark.parametrize("name,level,batch,n_keys", [("toy", 6, 3, 3), ("toy", 5, 2, 1), ("small", 24, 9, 3),
                                                     ("small", 9, 2, 2), ("wide", 6, 3, 3), ("full", 24, 2, 3)])
def test_rotate_sum_hoisted(name, level, batch, n_keys):
    """ct + sum_k rot_k(ct) with one decomposition and one division by P: residues equal the oracle's definition."""
    import torch

    pair = ctx_pair(name)
    ctx, orc, _ = pair
    rots = [(-2, 71), (-4, 72), (-6, 73)][:n_keys]
    for r, kid in rots:
        add_key(pair, r, kid)
    ct = random_ct(orc, 12, level, level, batch)
    out = torch.empty((batch, 2, level, orc.N), dtype=torch.int64, device="cuda")
    ctx.rotate_sum_hoisted(to_dev(ct), out, batch, level, [k for _, k in rots])
    got = to_host(out)
    for b in range(batch):
        assert np.array_equal(got[b], orc.rotate_sum_hoisted(ct[b], [k for _, k in rots])), (name, level, b)


def test_inner_product_staged_by_bulk_copies(monkeypatch):
    """The persistent inner-product kernel whose operands arrive by bulk asynchronous copies with bounded mbarrier
    waits (FESC_INNER_TMA=1): plain, hoisted and rotate-and-add key switches stay bit-exact and no wait gives up."""
    import torch

    monkeypatch.setenv("FESC_INNER_TMA", "1")
    for name, level, batch in (("small", 24, 5), ("full", 24, 3)):
        pair = ctx_pair(name)
        ctx, orc, _ = pair
        rots = [(3, 81), (-5, 82)]
        for r, kid in rots:
            add_key(pair, r, kid)
        ct = random_ct(orc, 13, level, level, batch)
        dev = to_dev(ct)
        out = torch.empty_like(dev)
        ctx.rotate(dev, out, batch, level, 81)
        hout = torch.empty((2, batch, 2, level, orc.N), dtype=torch.int64, device="cuda")
        ctx.rotate_hoisted(dev, hout, batch, level, [81, 82])
        sout = torch.empty_like(dev)
        ctx.rotate_sum_hoisted(dev, sout, batch, level, [81, 82])
        ctx.sync()                                  # FESC_ETIMEOUT would be raised here
        got, hgot, sgot = to_host(out), to_host(hout), to_host(sout)
        for b in range(batch):
            assert np.array_equal(got[b], orc.rotate(ct[b], 81))
            want = orc.rotate_hoisted(ct[b], [81, 82])
            assert np.array_equal(hgot[0, b], want[0]) and np.array_equal(hgot[1, b], want[1])
            assert np.array_equal(sgot[b], orc.rotate_sum_hoisted(ct[b], [81, 82]))


def test_integer_paths_with_primes_above_50_bits():
    """Primes of 52 and 55 bits take the integer kernels (wide-lazy transform at N = 2^16, 128-bit lazy
    accumulation in ModUp / inner product / ModDown); same bit-exact bar."""
    import torch

    ctx, orc, p = ctx_pair("full52")
    a = np.stack([S.uniform_residues_np(21, i, [orc.q[i]], orc.N)[0] for i in range(3)])[None]
    d = to_dev(a)
    ctx.ntt(d, 1, 0, 3)
    assert np.array_equal(to_host(d)[0], orc.ntt(a[0], [0, 1, 2]))
    ctx.intt(d, 1, 0, 3)
    assert np.array_equal(to_host(d), a)
    d = to_dev(a)
    ctx.intt(d, 1, 0, 3)
    assert np.array_equal(to_host(d)[0], orc.intt(a[0], [0, 1, 2]))
    pair = ctx_pair("wide")
    ctx, orc, p = pair
    add_key(pair, 3, 61)
    add_key(pair, 9, 62)
    for level in (6, 5, 2):
        ct = random_ct(orc, 22, level, level, 3)
        out = torch.empty_like(to_dev(ct))
        ctx.rotate(to_dev(ct), out, 3, level, 61)
        got = to_host(out)
        for b in range(3):
            assert np.array_equal(got[b], orc.rotate(ct[b], 61))
        hout = torch.empty((2, 3, 2, level, orc.N), dtype=torch.int64, device="cuda")
        ctx.rotate_hoisted(to_dev(ct), hout, 3, level, [61, 62])
        for b in range(3):
            want = orc.rotate_hoisted(ct[b], [61, 62])
            assert np.array_equal(to_host(hout)[0, b], want[0]) and np.array_equal(to_host(hout)[1, b], want[1])
        ct2 = random_ct(orc, 23, level, level, 3)
        ctx.ct_ct_mul(to_dev(ct), to_dev(ct2), out, 3, level)
        got = to_host(out)
        for b in range(3):
            assert np.array_equal(got[b], orc.ct_ct_mul(ct[b], ct2[b]))
        if level >= 2:
            res = torch.empty((3, 2, level - 1, orc.N), dtype=torch.int64, device="cuda")
            ctx.rescale(to_dev(ct), res, 3, level)
            for b in range(3):
                assert np.array_equal(to_host(res)[b], orc.rescale(ct[b]))


def test_allocation_failure_is_reported_and_the_context_stays_usable():
    """Host-side failure injection: the next scratch allocation of the context reports FESC_ENOMEM (the driver is not
    called); the error comes back through the call, nothing is launched, and the next call works and is bit-exact."""
    import torch
    import paper_2608_17442_b200 as fesc

    pair = ctx_pair("small")
    ctx, orc, _ = pair
    add_key(pair, 3, 81)
    level, batch = 8, 2
    ct = random_ct(orc, 31, level, level, batch)
    dev = to_dev(ct)
    out = torch.full_like(dev, -1)
    ctx.trim()                                  # the next key switch has to reserve scratch again
    launches = ctx.counters()[4]
    ctx.test_fail_allocs(1)
    with pytest.raises(fesc.FescError) as e:
        ctx.rotate(dev, out, batch, level, 81)
    assert e.value.code == fesc.ENOMEM and "scratch allocation" in str(e.value)
    assert ctx.counters()[4] == launches and ctx.counters()[3] == 0
    assert bool((out == -1).all())
    ctx.rotate(dev, out, batch, level, 81)      # the injected failure is used up: this call reserves and runs
    ctx.sync()
    got = to_host(out)
    for b in range(batch):
        assert np.array_equal(got[b], orc.rotate(ct[b], 81))
    assert ctx.info().flags == 0 and ctx.info().digits == ctx.num_digits


def test_results_do_not_depend_on_the_run_or_the_stream():
    """The same rotation batch (plain, hoisted and rotate-and-add) run twice on the default stream and once on each
    of two other streams, one after the other: all outputs are byte-identical (no dependence on scheduling, on what
    the scratch arena held before, or on the stream)."""
    import torch

    pair = ctx_pair("full")
    ctx, orc, _ = pair
    add_key(pair, 3, 81)
    add_key(pair, -5, 82)
    level, batch = 24, 5
    dev = to_dev(random_ct(orc, 41, level, level, batch))

    def run():
        out = torch.empty_like(dev)
        hout = torch.empty((2, batch, 2, level, orc.N), dtype=torch.int64, device="cuda")
        sout = torch.empty_like(dev)
        ctx.rotate(dev, out, batch, level, 81)
        ctx.rotate_hoisted(dev, hout, batch, level, [81, 82])
        ctx.rotate_sum_hoisted(dev, sout, batch, level, [81, 82])
        ctx.sync()
        return out, hout, sout

    first = run()
    runs = [run()]
    for _ in range(2):
        st = torch.cuda.Stream()
        torch.cuda.synchronize()
        with torch.cuda.stream(st):
            runs.append(run())
        torch.cuda.synchronize()
    for r in runs:
        for a, b in zip(first, r):
            assert torch.equal(a, b)


def test_inner_product_worst_case_residues_with_many_digits():
    """Largest possible partial sums of the key inner product: 9 digits (the FP64 path folds back after every 7
    products, so a second interval starts), every residue of the switched polynomial equal to q - 1, plain,
    hoisted and summed over 8 keys in one pass; bit-exact."""
    import torch

    pair = ctx_pair("small_d9")
    ctx, orc, p = pair
    add_key(pair, 1, 91)
    add_key(pair, 2, 92)
    level, batch = 18, 2
    ct = random_ct(orc, 51, level, level, batch)
    qs = np.array(orc.q[:level], dtype=np.uint64)
    ct[:, 1] = (qs - 1)[None, :, None]                  # c1 = q - 1 everywhere (the automorphism leaves it so)
    out = torch.empty_like(to_dev(ct))
    ctx.rotate(to_dev(ct), out, batch, level, 91)
    hout = torch.empty((2, batch, 2, level, orc.N), dtype=torch.int64, device="cuda")
    ctx.rotate_hoisted(to_dev(ct), hout, batch, level, [91, 92])
    got, hgot = to_host(out), to_host(hout)
    for b in range(batch):
        assert np.array_equal(got[b], orc.rotate(ct[b], 91))
        want = orc.rotate_hoisted(ct[b], [91, 92])
        assert np.array_equal(hgot[0, b], want[0]) and np.array_equal(hgot[1, b], want[1])
    # sums over several sources in one pass: rotate-and-add over 8 keys = 72 products per accumulator (the FP64 sums fold
    # back after every 7th, the 128-bit sums on the special primes are reduced after every 8th)
    kids = []
    for i, r in enumerate([1, 2, 3, 4, -1, -2, -3, -4]):
        add_key(pair, r, 93 + i) if r not in (1, 2) else None
        kids.append({1: 91, 2: 92}.get(r, 93 + i))
    sout = torch.empty_like(to_dev(ct))
    ctx.rotate_sum_hoisted(to_dev(ct), sout, batch, level, kids)
    sgot = to_host(sout)
    for b in range(batch):
        assert np.array_equal(sgot[b], orc.rotate_sum_hoisted(ct[b], kids))


def test_rotations_refuse_an_output_at_the_inputs_address():
    """fesc_rotate and fesc_rotate_hoisted read the input while they write the output: the same buffer for both is
    refused (FESC_EINVAL) before anything is launched."""
    import torch
    import paper_2608_17442_b200 as fesc

    pair = ctx_pair("small")
    ctx, orc, _ = pair
    add_key(pair, 3, 81)
    ct = to_dev(random_ct(orc, 77, 4, 4, 2))
    launches = ctx.counters()[4]
    for call in (lambda: ctx.rotate(ct, ct, 2, 4, 81), lambda: ctx.rotate_hoisted(ct, ct, 2, 4, [81])):
        with pytest.raises(fesc.FescError) as e:
            call()
        assert e.value.code == fesc.EINVAL
    assert ctx.counters()[4] == launches
