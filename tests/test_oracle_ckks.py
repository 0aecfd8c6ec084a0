"""Pins for the oracle's CKKS layer against big-integer arithmetic and the slot semantics
the paper states (rho(v; r)_j = v_{(j+r) mod n}; conj; ptmul/ctmul = slot-wise product)."""
import math

import numpy as np
import pytest

import fesc_synth as S
from oracle import ckks
from oracle.ckks import CONJ, RELIN_KEY_ID, Oracle, _lib, crt_lift_centered
from tests.bigint_ref import centre, crt, negacyclic_mul_int, poly_from_rns, prod


def test_crt_lift_matches_bigint(toy_oracle):
    o = toy_oracle
    mods = o.q[:4]
    Q = prod(mods)
    rng = np.random.default_rng(1)
    vals = [int(rng.integers(0, 2**62)) * int(rng.integers(0, 2**50)) % Q for _ in range(o.N)]
    res = np.array([[v % q for v in vals] for q in mods], dtype=np.uint64)
    got = crt_lift_centered(res, mods)
    assert got == [centre(v, Q) for v in vals]
    assert [crt([v % q for q in mods], mods) for v in vals] == vals


def test_samplers():
    n = 1 << 14
    t = np.empty(n, dtype=np.int64)
    _lib.orc_sample_ternary(5, 1, t, n)
    assert set(np.unique(t)) == {-1, 0, 1}
    assert abs(t.mean()) < 0.03 and abs((t == 0).mean() - 1 / 3) < 0.02
    e = np.empty(n, dtype=np.int64)
    _lib.orc_sample_cbd(5, 3, e, n)
    assert abs(e.mean()) < 0.1 and abs(e.var() - 10.5) < 0.6 and np.abs(e).max() <= 21
    q = 1125899906826241
    u = np.empty(n, dtype=np.uint64)
    _lib.orc_sample_uniform(5, 2, q, u, n)
    assert u.max() < q and abs(u.astype(np.float64).mean() / q - 0.5) < 0.01
    # the generator itself, retyped: word = M(M(seed ^ M(tag)) + index)
    def M(z):
        z = (z + 0x9E3779B97F4A7C15) % 2**64
        z = ((z ^ (z >> 30)) * 0xBF58476D1CE4E5B9) % 2**64
        z = ((z ^ (z >> 27)) * 0x94D049BB133111EB) % 2**64
        return z ^ (z >> 31)
    for idx in (0, 1, 77):
        w = M((M(5 ^ M(2)) + idx) % 2**64)
        assert _lib.orc_draw(5, 2, idx) == w
        assert int(u[idx]) == (w * q) >> 64
    # tag packing keeps the fields apart
    assert len({ckks.make_tag(d, k, j, l) for d in (1, 2) for k in (0, 5) for j in (0, 3) for l in (0, 9)}) == 16


def test_fast_conversion_overshoot(toy_oracle):
    """ModUp form: result = [x]_S + u*S with integer 0 <= u < |src|; centred form:
    result = x (mod S) and |result| < |src|*S/2 (when the target modulus is large enough to see it)."""
    o = toy_oracle
    src, dst = [0, 1], [2, 3, 4, 5, 6, 7]
    a = S.uniform_residues_np(2, 0, [o.q[i] for i in src], o.N)
    Sm = prod(o.q[i] for i in src)
    Dm = prod(o.q[i] for i in dst)
    x = poly_from_rns(a, [o.q[i] for i in src])
    out = poly_from_rns(o.fast_conv(a, src, dst), [o.q[i] for i in dst])
    us = set()
    for xi, yi in zip(x, out):
        assert (yi - xi) % Sm == 0
        us.add((yi - xi) // Sm)
    assert us <= {0, 1} and len(us) == 2
    outc = poly_from_rns(o.fast_conv(a, src, dst, centred=True), [o.q[i] for i in dst])
    for xi, yi in zip(x, outc):
        yc = centre(yi, Dm)
        assert (yc - xi) % Sm == 0 and abs(yc) < len(src) * Sm / 2
    # one source limb, centred: the exact centred remainder
    one = poly_from_rns(o.fast_conv(a[:1], [0], dst, centred=True), [o.q[i] for i in dst])
    assert [centre(v, Dm) for v in one] == [centre(int(v), o.q[0]) for v in a[0]]


@pytest.mark.parametrize("level", [6, 5, 3])
def test_mod_down_is_rounded_division_by_P(toy_oracle, level):
    o = toy_oracle
    ext = list(range(level)) + o.special
    mods = [o.q[i] for i in ext]
    c = S.uniform_residues_np(3, level, mods, o.N)
    big = poly_from_rns(c, mods)
    Ql = prod(o.q[:level])
    got = poly_from_rns(o.intt(o.mod_down(o.ntt(c, ext), level), list(range(level))), o.q[:level])
    errs = set()
    for v, g in zip(big, got):
        exact = (2 * v + o.P) // (2 * o.P)  # round(v / P)
        errs.add(centre(g - exact, Ql))
    assert max(abs(e) for e in errs) <= o.K // 2 + 1 and 0 in errs
    assert abs(sum(errs)) <= 1  # symmetric, no bias


@pytest.mark.parametrize("level", [6, 2])
def test_rescale_is_exact_rounding(toy_oracle, level):
    o = toy_oracle
    mods = o.q[:level]
    data = list(range(level))
    c = np.stack([S.uniform_residues_np(4, p, mods, o.N) for p in range(2)])
    ct = np.stack([o.ntt(c[p], data) for p in range(2)])
    out = o.rescale(ct)
    ql, Qr = o.q[level - 1], prod(mods[:-1])
    for p in range(2):
        big = poly_from_rns(c[p], mods)
        got = poly_from_rns(o.intt(out[p], data[:-1]), mods[:-1])
        assert got == [((2 * v + ql) // (2 * ql)) % Qr for v in big]


def test_automorphism_forms_agree_and_compose(toy_oracle):
    o = toy_oracle
    idx = [0, 1]
    a = S.uniform_residues_np(5, 0, [o.q[i] for i in idx], o.N)
    ae = o.ntt(a, idx)
    for g in (5, 25, pow(5, 7, 2 * o.N), 2 * o.N - 1):
        via_coeff = o.ntt(o.automorphism_coeff(a, g, idx), idx)
        assert np.array_equal(o.automorphism(ae, g, 2), via_coeff)
    g, h = 5, pow(5, 11, 2 * o.N)
    assert np.array_equal(o.automorphism(o.automorphism(ae, g, 2), h, 2), o.automorphism(ae, g * h % (2 * o.N), 2))
    # coefficient form by hand on X: X -> X^g
    x = np.zeros((1, o.N), dtype=np.uint64)
    x[0, 1] = 1
    y = o.automorphism_coeff(x, 2 * o.N - 1, [0])  # X^(2N-1) = -X^(N-1)
    assert y[0, o.N - 1] == o.q[0] - 1 and y.sum() == o.q[0] - 1


def test_encode_decode_and_slot_semantics(toy_oracle):
    o = toy_oracle
    z = S.uniform_slots(6, 0, 1, o.n)[0] + 1j * S.uniform_slots(6, 1, 1, o.n)[0]
    m = o.encode_coeffs(z, 2.0**30).astype(np.float64) / 2.0**30
    assert np.abs(o.decode_coeffs(m) - z).max() < 1e-6
    # decoding is evaluation at zeta^(5^j)
    zeta = np.exp(1j * np.pi / o.N)
    for j in (0, 1, 7):
        root = zeta ** pow(5, j, 2 * o.N)
        assert abs(sum(m[i] * root**i for i in range(o.N)) - z[j]) < 1e-6


def test_evk_identity_bigint(toy_oracle):
    """b_j + a_j s - e_j = P * T_j * s' (mod P*Q) with T_j = 1 on digit j, 0 on the other data limbs."""
    o = toy_oracle
    o.add_galois_key(3, 11)
    g, evk = o.keys[11]
    allidx = list(range(o.n_q + o.K))
    mods = [o.q[i] for i in allidx]
    PQ = prod(mods)
    s = [int(v) for v in o.s_coeff]
    s_rot = poly_from_rns(o.intt(o.automorphism(o.s_eval, g, len(allidx)), allidx), mods)
    for j in range(o.beta_max):
        b = poly_from_rns(o.intt(evk[j, 0], allidx), mods)
        a = poly_from_rns(o.intt(evk[j, 1], allidx), mods)
        e = np.empty(o.N, dtype=np.int64)
        _lib.orc_sample_cbd(o.seed, ckks.make_tag(ckks.DOM_EVK_E, 11, j), e, o.N)
        lhs = [(bi + asi - int(ei)) % PQ for bi, asi, ei in zip(b, negacyclic_mul_int(a, s, PQ), e)]
        D = o.digit_limbs(j, o.n_q)
        Qj = prod(o.q[i] for i in D)
        Q = prod(o.q[:o.n_q])
        Tj = (Q // Qj) * pow(Q // Qj, -1, Qj)
        assert lhs == [(o.P * Tj * si) % PQ for si in s_rot]


@pytest.mark.parametrize("level", [6, 5])
def test_key_switch_identity_before_division(toy_oracle, level):
    """c'_0 + c'_1 s = P d s' + sum_j d~_j e_j  (mod P Q_l), with d~_j = [d]_{Q_j} + u Q_j."""
    o = toy_oracle
    o.add_galois_key(1, 12)
    g, _ = o.keys[12]
    data = list(range(level))
    ext = data + o.special
    mods = [o.q[i] for i in ext]
    PQ = prod(mods)
    d = S.uniform_residues_np(7, level, o.q[:level], o.N)
    d_eval = o.ntt(d, data)
    acc = o.key_switch_raw(d_eval, 12, level)
    c0 = poly_from_rns(o.intt(acc[0], ext), mods)
    c1 = poly_from_rns(o.intt(acc[1], ext), mods)
    s = [int(v) for v in o.s_coeff]
    lhs = [(x + y) % PQ for x, y in zip(c0, negacyclic_mul_int(c1, s, PQ))]
    d_big = poly_from_rns(d, o.q[:level])
    allidx = list(range(o.n_q + o.K))
    s_rot = [centre(v, prod(o.q)) for v in
             poly_from_rns(o.intt(o.automorphism(o.s_eval, g, len(allidx)), allidx), [o.q[i] for i in allidx])]
    rhs = [o.P * v for v in negacyclic_mul_int(d_big, s_rot, PQ)]
    for j in range(-(-level // o.alpha)):
        dt = poly_from_rns(o.intt(o.mod_up_digit(d, d_eval, j, level), ext), mods)
        D = o.digit_limbs(j, level)
        Qj = prod(o.q[i] for i in D)
        for v, x in zip(dt, d_big):
            assert (v - x % Qj) % Qj == 0 and 0 <= (v - x % Qj) // Qj < len(D)
        e = np.empty(o.N, dtype=np.int64)
        _lib.orc_sample_cbd(o.seed, ckks.make_tag(ckks.DOM_EVK_E, 12, j), e, o.N)
        rhs = [r + t for r, t in zip(rhs, negacyclic_mul_int(dt, [int(v) for v in e], PQ))]
    assert lhs == [r % PQ for r in rhs]


@pytest.mark.parametrize("r", [1, 5, 31, -2])
def test_rotation_is_cyclic_left_shift(toy_oracle, r):
    o = toy_oracle
    scale = 2.0**20
    z = S.uniform_slots(8, 0, 1, o.n)[0]
    ct = o.encrypt(o.encode(z, scale, 6), 1)
    o.add_galois_key(r, 20)
    got = o.decrypt(o.rotate(ct, 20), scale)
    assert np.abs(got - np.roll(z, -r)).max() < 2e-4


def test_conjugation_and_times_i(toy_oracle):
    o = toy_oracle
    scale = 2.0**20
    z = S.uniform_slots(9, 0, 1, o.n)[0] + 1j * S.uniform_slots(9, 1, 1, o.n)[0]
    ct = o.encrypt(o.encode(z, scale, 6), 2)
    o.add_galois_key(CONJ, 21)
    assert np.abs(o.decrypt(o.rotate(ct, 21), scale) - np.conj(z)).max() < 2e-4
    assert np.abs(o.decrypt(o.mul_monomial_half(ct), scale) - 1j * z).max() < 2e-4


def test_mac_ctmul_rescale_semantics(toy_oracle):
    o = toy_oracle
    scale = 2.0**20
    z, w, v = S.uniform_slots(10, 0, 3, o.n)
    ctz = o.encrypt(o.encode(z, scale, 6), 3)
    ctv = o.encrypt(o.encode(v, scale, 6), 4)
    pw = o.encode(w, scale, 6)
    # acc = ctz*w + ctv*w
    acc = o.ct_pt_mac(ctv, pw, o.ct_pt_mac(ctz, pw, np.zeros_like(ctz)))
    assert np.abs(o.decrypt(acc, scale * scale) - (z + v) * w).max() < 2e-4
    prod_ct = o.ct_ct_mul(ctz, ctv)
    assert np.abs(o.decrypt(prod_ct, scale * scale) - z * v).max() < 2e-4
    pw30 = o.encode(w, float(o.q[5]), 6)
    res = o.rescale(o.ct_pt_mac(ctz, pw30, np.zeros_like(ctz)))
    assert res.shape == (2, 5, o.N)
    assert np.abs(o.decrypt(res, scale) - z * w).max() < 2e-4


def test_tiny_workload_through_oracle():
    """Workload 1 end to end: 4 ciphertexts x plaintext vector, rotate by +1 and +5, decrypt."""
    p = S.params("tiny")
    o = Oracle(p["log_n"], p["primes"], p["n_q"], p["n_p"], p["dnum"], p["seed"])
    assert max(o.q[:3]) < o.q[3] and all(q.bit_length() == 36 for q in o.q)
    scale = 2.0**30
    z = S.uniform_slots(p["seed"], 0, 4, o.n)
    w = S.uniform_slots(p["seed"], 1, 4, o.n)
    o.add_galois_key(1, 1)
    o.add_galois_key(5, 2)
    for i in range(4):
        ct = o.encrypt(o.encode(z[i], scale, 3), i)
        pr = o.ct_pt_mac(ct, o.encode(w[i], scale, 3), np.zeros_like(ct))
        for kid, r in ((1, 1), (2, 5)):
            got = o.decrypt(o.rotate(pr, kid), scale * scale)
            assert np.abs(got - np.roll(z[i] * w[i], -r)).max() < 2.0**-16


def test_hoisted_rotations_are_rotations_and_share_noise_bound(toy_oracle):
    """The hoisted mode gives the same slot shift as `rotate`; its residues differ only by the permuted ModUp
    overshoot, so both decrypt to the shift within the same tolerance."""
    o = toy_oracle
    scale = 2.0**20
    z = S.uniform_slots(14, 0, 1, o.n)[0]
    ct = o.encrypt(o.encode(z, scale, 6), 5)
    for r, kid in ((1, 31), (4, 32), (-3, 33)):
        o.add_galois_key(r, kid)
    outs = o.rotate_hoisted(ct, [31, 32, 33])
    for (r, kid), got in zip(((1, 31), (4, 32), (-3, 33)), outs):
        assert np.abs(o.decrypt(got, scale) - np.roll(z, -r)).max() < 2e-4
        plain = o.rotate(ct, kid)
        assert got.shape == plain.shape
        # same c1-independent part: the difference of the two results decrypts to (almost) zero
        diff = np.stack([o.sub(got[p], plain[p], list(range(6))) for p in range(2)])
        assert np.abs(o.decrypt(diff, scale)).max() < 2e-4
    # at a level where the last digit is partial
    ct5 = np.ascontiguousarray(ct[:, :5])
    got = o.rotate_hoisted(ct5, [32])[0]
    assert np.abs(o.decrypt(got, scale) - np.roll(z, -4)).max() < 2e-4


def test_rotate_sum_hoisted_is_the_sum_of_rotations(toy_oracle):
    """ct + sum_k rot_k(ct) with one decomposition and one division by P: decrypts to z + sum_k roll(z, -r_k), and
    differs from the sum of separately hoisted rotations by at most one unit per rotation in every coefficient
    (big-integer check of the additivity of the division by P up to rounding)."""
    from oracle.ckks import crt_lift_centered
    o = toy_oracle
    scale = 2.0**20
    z = S.uniform_slots(15, 0, 1, o.n)[0]
    level = 5
    data = list(range(level))
    ct = np.ascontiguousarray(o.encrypt(o.encode(z, scale, 6), 9)[:, :level])
    rots = ((-1, 41), (-2, 42), (-3, 43))
    for r, kid in rots:
        o.add_galois_key(r, kid)
    got = o.rotate_sum_hoisted(ct, [k for _, k in rots])
    want = z + sum(np.roll(z, -r) for r, _ in rots)
    assert np.abs(o.decrypt(got, scale) - want).max() < 5e-4
    ref = ct
    for out in o.rotate_hoisted(ct, [k for _, k in rots]):
        ref = o.ct_add(ref, out)
    seen = 0
    for c in range(2):
        d = o.sub(got[c], ref[c], data)
        diff = crt_lift_centered(o.intt(d, data), [o.q[i] for i in data])
        assert max(abs(int(v)) for v in diff) <= len(rots)
        seen += sum(1 for v in diff if int(v) != 0)
    assert seen > 0
    # a single rotation: exactly ct + rotate_hoisted
    one = o.rotate_sum_hoisted(ct, [42])
    assert np.array_equal(one, o.ct_add(ct, o.rotate_hoisted(ct, [42])[0]))


def test_split_complex_returns_doubled_real_and_imaginary_parts(toy_oracle):
    o = toy_oracle
    scale = 2.0**20
    z = S.uniform_slots(16, 0, 2, o.n)
    o.add_galois_key(CONJ, 47)
    ct = o.encrypt(o.encode(z[0] + 1j * z[1], scale, 4), 21)
    re2, im2 = o.split_complex(ct, 47)
    assert np.abs(o.decrypt(re2, scale) - 2 * z[0]).max() < 3e-4
    assert np.abs(o.decrypt(im2, scale) - 2 * z[1]).max() < 3e-4
    assert np.abs(o.decrypt(re2, scale).imag).max() < 3e-4 and np.abs(o.decrypt(im2, scale).imag).max() < 3e-4
