"""CPU oracle for the RNS-CKKS linear hot path (TEST INFRASTRUCTURE, fp64 / exact integers).

Only tests, the smoke check and the benchmark's CPU-baseline leg may import this
module; the product path never does, and this module imports nothing from the
CUDA package.  It composes the C primitives of oracle/fesc_oracle.c into the
operations the library exports, in the order the definitions state them:

  * encode / decode / encrypt / decrypt (harness side; the paper's client holds
    the secret key, Sec. 3 threat model),
  * ct-pt multiply-accumulate  (Table "CKKS primitives": ptmul, add),
  * rotation / conjugation = Galois automorphism then hybrid key switch
    (Table "CKKS primitives": rot, conj; rho(v; r)_j = v_{(j+r) mod n}),
  * rescale, ct x ct with relinearisation (ctmul),
  * the BSGS plaintext-weight projection Y = XW (App. "Projection Kernel
    Breakdown": packing idx(r,c) = c*T + r, accumulators c_p, giant-step fold).

The paper uses its CKKS backend as a black box, so the internals follow the
standard hybrid (dnum) key switching with these readings: canonical residues in
[0, q); uncorrected fast basis conversion in ModUp; division by P with the CENTRED
fast conversion of the special-limb residues (no half-P shift; error at most K/2
units, exact rounding for K = 1); rescale = the same centred conversion with one
source limb, i.e. exact rounded division by the dropped prime.

Layouts: a polynomial on k limbs is a uint64 array [k, N]; a ciphertext at
level l is [2, l, N] (c0 then c1), evaluation form, bit-reversed order.
"""
from __future__ import annotations

import ctypes
import math

import numpy as np

from . import build as _build

_lib = ctypes.CDLL(_build.build())
_u64p = np.ctypeslib.ndpointer(dtype=np.uint64, flags="C_CONTIGUOUS")
_i64p = np.ctypeslib.ndpointer(dtype=np.int64, flags="C_CONTIGUOUS")
_c = ctypes
_lib.orc_powmod.restype = _c.c_uint64
_lib.orc_powmod.argtypes = [_c.c_uint64] * 3
_lib.orc_min_psi.restype = _c.c_uint64
_lib.orc_min_psi.argtypes = [_c.c_uint64, _c.c_uint32]
_lib.orc_draw.restype = _c.c_uint64
_lib.orc_draw.argtypes = [_c.c_uint64] * 3
_lib.orc_ntt.argtypes = [_u64p, _u64p, _c.c_uint32, _c.c_uint32]
_lib.orc_intt.argtypes = [_u64p, _u64p, _c.c_uint32, _c.c_uint32]
_lib.orc_ntt_direct.argtypes = [_u64p, _u64p, _c.c_uint64, _c.c_uint32]
for _n in ("orc_mul", "orc_muladd", "orc_add", "orc_sub", "orc_mul_scalar", "orc_add_scalar"):
    getattr(_lib, _n).argtypes = [_u64p, _u64p, _u64p, _u64p, _c.c_uint32, _c.c_uint64]
_lib.orc_autom_coeff.argtypes = [_u64p, _u64p, _u64p, _c.c_uint32, _c.c_uint32, _c.c_uint64]
_lib.orc_autom_eval.argtypes = [_u64p, _u64p, _c.c_uint32, _c.c_uint32, _c.c_uint64]
_lib.orc_fast_conv.argtypes = [_u64p, _u64p, _c.c_uint32, _u64p, _c.c_uint32, _u64p, _c.c_uint64, _c.c_int]
_lib.orc_sample_uniform.argtypes = [_c.c_uint64, _c.c_uint64, _c.c_uint64, _u64p, _c.c_uint64]
_lib.orc_sample_ternary.argtypes = [_c.c_uint64, _c.c_uint64, _i64p, _c.c_uint64]
_lib.orc_sample_cbd.argtypes = [_c.c_uint64, _c.c_uint64, _i64p, _c.c_uint64]
_lib.orc_signed_to_rns.argtypes = [_i64p, _u64p, _u64p, _c.c_uint32, _c.c_uint64]

# domains of the counter-based generator
DOM_SECRET, DOM_EVK_A, DOM_EVK_E, DOM_ENC_A, DOM_ENC_E = 1, 2, 3, 4, 5
RELIN_KEY_ID = 0          # key id reserved for the relinearisation key
CONJ = -(1 << 31)         # "rotation amount" that selects complex conjugation


def make_tag(domain: int, key_id: int = 0, digit: int = 0, limb: int = 0) -> int:
    return domain | (key_id << 8) | (digit << 40) | (limb << 48)


def _arr(x) -> np.ndarray:
    return np.ascontiguousarray(x, dtype=np.uint64)


class Oracle:
    """RNS-CKKS context: `n_q` data primes then `n_p` special primes (all = 1 mod 2N)."""

    def __init__(self, log_n: int, primes, n_q: int, n_p: int, dnum: int, seed: int):
        assert len(primes) == n_q + n_p and n_p >= 1 and dnum >= 1
        self.log_n, self.N, self.n = log_n, 1 << log_n, 1 << (log_n - 1)
        self.q = [int(p) for p in primes]
        self.n_q, self.K = n_q, n_p
        self.alpha = -(-n_q // dnum)
        self.beta_max = -(-n_q // self.alpha)
        self.seed = seed
        self.special = list(range(n_q, n_q + n_p))
        self.P = math.prod(self.q[i] for i in self.special)
        for p in self.q:
            assert _lib.orc_min_psi(p, log_n) != 0, "prime is not NTT friendly"
        # secret key: ternary coefficients from the seed, kept in EVAL form on every limb
        s = np.empty(self.N, dtype=np.int64)
        _lib.orc_sample_ternary(seed, make_tag(DOM_SECRET), s, self.N)
        self.s_coeff = s
        allidx = list(range(n_q + n_p))
        self.s_eval = self.ntt(self.signed_to_rns(s, allidx), allidx)
        self.keys: dict[int, tuple[int, np.ndarray]] = {}
        s2 = self.mul(self.s_eval, self.s_eval, allidx)
        self.keys[RELIN_KEY_ID] = (0, self._gen_evk(RELIN_KEY_ID, s2))

    # ---- limb-wise primitives ------------------------------------------------
    def _q(self, idx) -> np.ndarray:
        return np.array([self.q[i] for i in idx], dtype=np.uint64)

    def ntt(self, a, idx):
        a = _arr(a).copy().reshape(len(idx), self.N)
        _lib.orc_ntt(a, self._q(idx), len(idx), self.log_n)
        return a

    def intt(self, a, idx):
        a = _arr(a).copy().reshape(len(idx), self.N)
        _lib.orc_intt(a, self._q(idx), len(idx), self.log_n)
        return a

    def _bin(self, fn, a, b, idx):
        a, b = _arr(a), _arr(b)
        out = np.empty_like(a)
        fn(a, b, out, self._q(idx), len(idx), a.size // len(idx))
        return out

    def mul(self, a, b, idx):
        return self._bin(_lib.orc_mul, a, b, idx)

    def add(self, a, b, idx):
        return self._bin(_lib.orc_add, a, b, idx)

    def sub(self, a, b, idx):
        return self._bin(_lib.orc_sub, a, b, idx)

    def mul_scalar(self, a, scalars, idx):
        c = np.array([int(s) % self.q[i] for s, i in zip(scalars, idx)], dtype=np.uint64)
        return self._bin(_lib.orc_mul_scalar, a, c, idx)

    def add_scalar(self, a, scalars, idx):
        c = np.array([int(s) % self.q[i] for s, i in zip(scalars, idx)], dtype=np.uint64)
        return self._bin(_lib.orc_add_scalar, a, c, idx)

    def neg(self, a, idx):
        return self.sub(np.zeros_like(_arr(a)), a, idx)

    def signed_to_rns(self, v, idx):
        v = np.ascontiguousarray(v, dtype=np.int64)
        out = np.empty((len(idx), v.size), dtype=np.uint64)
        _lib.orc_signed_to_rns(v, out, self._q(idx), len(idx), v.size)
        return out

    def fast_conv(self, a, src_idx, dst_idx, centred: bool = False):
        a = _arr(a).reshape(len(src_idx), -1)
        out = np.empty((len(dst_idx), a.shape[1]), dtype=np.uint64)
        _lib.orc_fast_conv(a, self._q(src_idx), len(src_idx), self._q(dst_idx), len(dst_idx), out,
                           a.shape[1], int(centred))
        return out

    # ---- Galois maps ---------------------------------------------------------
    def galois_element(self, r: int) -> int:
        """g with sigma_g = rho(.; r) (cyclic LEFT shift by r slots), or conjugation."""
        if r == CONJ:
            return 2 * self.N - 1
        return pow(5, r % self.n, 2 * self.N)

    def automorphism(self, a, g: int, k: int):
        a = _arr(a).reshape(k, self.N)
        out = np.empty_like(a)
        _lib.orc_autom_eval(a, out, k, self.log_n, g)
        return out

    def automorphism_coeff(self, a, g: int, idx):
        a = _arr(a).reshape(len(idx), self.N)
        out = np.empty_like(a)
        _lib.orc_autom_coeff(a, out, self._q(idx), len(idx), self.log_n, g)
        return out

    # ---- keys ------------------------------------------------------------------
    def digit_limbs(self, j: int, level: int):
        return list(range(j * self.alpha, min((j + 1) * self.alpha, level)))

    def _gen_evk(self, key_id: int, s_prime_eval):
        """Switching key from s' to s: for digit j and every modulus t (data and special),
        a_j uniform (drawn in EVAL form), e_j centred binomial,
        b_j = -a_j s + e_j + [t in digit j] (P mod q_t) s'.   Shape [beta, 2, n_q+K, N]."""
        allidx = list(range(self.n_q + self.K))
        evk = np.empty((self.beta_max, 2, len(allidx), self.N), dtype=np.uint64)
        for j in range(self.beta_max):
            a = np.empty((len(allidx), self.N), dtype=np.uint64)
            for t in allidx:
                _lib.orc_sample_uniform(self.seed, make_tag(DOM_EVK_A, key_id, j, t), self.q[t], a[t], self.N)
            e = np.empty(self.N, dtype=np.int64)
            _lib.orc_sample_cbd(self.seed, make_tag(DOM_EVK_E, key_id, j), e, self.N)
            e_eval = self.ntt(self.signed_to_rns(e, allidx), allidx)
            b = self.add(self.neg(self.mul(a, self.s_eval, allidx), allidx), e_eval, allidx)
            dj = self.digit_limbs(j, self.n_q)
            b[dj] = self.add(b[dj], self.mul_scalar(s_prime_eval[dj], [self.P] * len(dj), dj), dj)
            evk[j, 0], evk[j, 1] = b, a
        return evk

    def add_galois_key(self, r: int, key_id: int):
        assert key_id != RELIN_KEY_ID
        g = self.galois_element(r)
        allidx = list(range(self.n_q + self.K))
        self.keys[key_id] = (g, self._gen_evk(key_id, self.automorphism(self.s_eval, g, len(allidx))))

    # ---- hybrid key switch -----------------------------------------------------
    def mod_up_digit(self, d_coeff, d_eval, j: int, level: int):
        """Digit j of d extended to all level+K moduli, EVAL form."""
        ext = list(range(level)) + self.special
        D = self.digit_limbs(j, level)
        others = [t for t in ext if t not in D]
        conv = self.ntt(self.fast_conv(d_coeff[D], D, others), others)
        out = np.empty((len(ext), self.N), dtype=np.uint64)
        for pos, t in enumerate(ext):
            out[pos] = d_eval[t] if t in D else conv[others.index(t)]
        return out

    def mod_down(self, c_ext, level: int):
        """Division by P with centred remainder: [level+K, N] EVAL -> [level, N] EVAL.
        c_i = (c'_i - Conv_i([c']_P)) * P^-1 mod q_i, Conv = centred fast conversion of the
        special-limb residues (COEFF form) to q_i.  Equals round(c'/P) + e, |e| <= K/2,
        e = 0 when K = 1."""
        data = list(range(level))
        r = self.intt(c_ext[level:], self.special)
        u = self.ntt(self.fast_conv(r, self.special, data, centred=True), data)
        pinv = [pow(self.P, -1, self.q[i]) for i in data]
        return self.mul_scalar(self.sub(c_ext[:level], u, data), pinv, data)

    def key_switch_raw(self, d_eval, key_id: int, level: int):
        """Steps 1-4: returns the two accumulators on level+K moduli before division by P."""
        evk = self.keys[key_id][1]
        data = list(range(level))
        ext = data + self.special
        d_eval = _arr(d_eval).reshape(level, self.N)
        d_coeff = self.intt(d_eval, data)
        acc = np.zeros((2, len(ext), self.N), dtype=np.uint64)
        for j in range(-(-level // self.alpha)):
            dt = self.mod_up_digit(d_coeff, d_eval, j, level)
            for p in range(2):
                _lib.orc_muladd(dt, _arr(evk[j, p][ext]), acc[p], self._q(ext), len(ext), self.N)
        return acc

    def key_switch(self, d_eval, key_id: int, level: int):
        acc = self.key_switch_raw(d_eval, key_id, level)
        return np.stack([self.mod_down(acc[0], level), self.mod_down(acc[1], level)])

    # ---- ciphertext operations ---------------------------------------------------
    def ct_pt_mac(self, ct, pt, acc):
        """acc_p += c_p (.) pt for p in {0,1}; returns the new accumulator."""
        level = ct.shape[1]
        data = list(range(level))
        out = _arr(acc).copy()
        for p in range(2):
            _lib.orc_muladd(_arr(ct[p]), _arr(pt), out[p], self._q(data), level, self.N)
        return out

    def ct_add(self, a, b):
        level = a.shape[1]
        data = list(range(level))
        return np.stack([self.add(a[p], b[p], data) for p in range(2)])

    def rotate(self, ct, key_id: int):
        """Automorphism FIRST, then key switch of the permuted c1:
        (c0, c1) -> (sigma_g c0 + ks_0, ks_1)."""
        level = ct.shape[1]
        g = self.keys[key_id][0]
        data = list(range(level))
        c0 = self.automorphism(ct[0], g, level)
        d = self.automorphism(ct[1], g, level)
        ks = self.key_switch(d, key_id, level)
        return np.stack([self.add(c0, ks[0], data), ks[1]])

    def rotate_hoisted(self, ct, key_ids):
        """Several rotations of ONE ciphertext that share the decomposition of c1 ("hoisting"; a second,
        separately defined mode).  c1 is brought to COEFF form, extended digit by digit (ModUp) and
        transformed back ONCE; for every key the automorphism is applied to the extended digits (in EVAL
        form a permutation), then inner product with the key and division by P as in `key_switch`:
            out_g = (sigma_g c0 + ks0, ks1),  ks = ModDown( sum_j sigma_g(d~_j) (.) evk_{g,j} ).
        The residues differ from `rotate` (the conversion overshoot is permuted instead of recomputed);
        the decrypted value is the same rotation."""
        level = ct.shape[1]
        data = list(range(level))
        ext = data + self.special
        d_eval = _arr(ct[1])
        d_coeff = self.intt(d_eval, data)
        digits = [self.mod_up_digit(d_coeff, d_eval, j, level) for j in range(-(-level // self.alpha))]
        outs = []
        for kid in key_ids:
            g, evk = self.keys[kid]
            acc = np.zeros((2, len(ext), self.N), dtype=np.uint64)
            for j, dj in enumerate(digits):
                dt = self.automorphism(dj, g, len(ext))
                for p in range(2):
                    _lib.orc_muladd(dt, _arr(evk[j, p][ext]), acc[p], self._q(ext), len(ext), self.N)
            c0 = self.automorphism(ct[0], g, level)
            outs.append(np.stack([self.add(c0, self.mod_down(acc[0], level), data), self.mod_down(acc[1], level)]))
        return outs

    def rotate_sum_hoisted(self, ct, key_ids):
        """ct + sum_k rot_k(ct): hoisted rotations (one decomposition of c1) whose key-switch accumulators are
        summed on the extended basis and divided by P ONCE (a separately defined mode, used by the radix-4
        rotate-and-add fills of the scan):
            out0 = c0 + sum_k sigma_k(c0) + ModDown( sum_k sum_j sigma_k(d~_j) (.) evk_{k,j}[0] ),
            out1 = c1                     + ModDown( sum_k sum_j sigma_k(d~_j) (.) evk_{k,j}[1] )."""
        level = ct.shape[1]
        data = list(range(level))
        ext = data + self.special
        d_eval = _arr(ct[1])
        d_coeff = self.intt(d_eval, data)
        digits = [self.mod_up_digit(d_coeff, d_eval, j, level) for j in range(-(-level // self.alpha))]
        acc = np.zeros((2, len(ext), self.N), dtype=np.uint64)
        y0 = _arr(ct[0]).copy()
        for kid in key_ids:
            g, evk = self.keys[kid]
            for j, dj in enumerate(digits):
                dt = self.automorphism(dj, g, len(ext))
                for p in range(2):
                    _lib.orc_muladd(dt, _arr(evk[j, p][ext]), acc[p], self._q(ext), len(ext), self.N)
            y0 = self.add(y0, self.automorphism(ct[0], g, level), data)
        return np.stack([self.add(y0, self.mod_down(acc[0], level), data),
                         self.add(_arr(ct[1]), self.mod_down(acc[1], level), data)])

    def rescale(self, ct):
        """Rounded division by the last prime, level l -> l-1:
        c_i <- (c_i - [c_last]_centred) * q_last^-1 mod q_i  (= round(c / q_last) exactly)."""
        level = ct.shape[1]
        last = level - 1
        rest = list(range(last))
        ql = self.q[last]
        out = np.empty((2, last, self.N), dtype=np.uint64)
        qinv = [pow(ql, -1, self.q[i]) for i in rest]
        for p in range(2):
            r = self.intt(ct[p, last:last + 1], [last])            # COEFF, modulo q_last
            u = self.ntt(self.fast_conv(r, [last], rest, centred=True), rest)
            out[p] = self.mul_scalar(self.sub(ct[p, :last], u, rest), qinv, rest)
        return out

    def ct_ct_mul(self, a, b):
        """(d0, d1, d2) = (a0 b0, a0 b1 + a1 b0, a1 b1); result (d0 + ks_0, d1 + ks_1) with
        ks = KeySwitch(d2, relinearisation key).  No rescale."""
        level = a.shape[1]
        data = list(range(level))
        d0 = self.mul(a[0], b[0], data)
        d1 = self.add(self.mul(a[0], b[1], data), self.mul(a[1], b[0], data), data)
        d2 = self.mul(a[1], b[1], data)
        ks = self.key_switch(d2, RELIN_KEY_ID, level)
        return np.stack([self.add(d0, ks[0], data), self.add(d1, ks[1], data)])

    def mul_monomial_half(self, ct):
        """Multiply both polynomials by X^(N/2) (every slot times i; exact)."""
        level = ct.shape[1]
        data = list(range(level))
        mono = np.zeros(self.N, dtype=np.int64)
        mono[self.N // 2] = 1
        m_eval = self.ntt(self.signed_to_rns(mono, data), data)
        return np.stack([self.mul(ct[p], m_eval, data) for p in range(2)])

    def split_complex(self, ct, conj_key_id: int):
        """Real and imaginary slot parts of a complex-packed ciphertext, each doubled (exact, no rescale):
            re2 = ct + conj(ct)            (slots 2 Re z)
            im2 = -i (ct - conj(ct))       (slots 2 Im z;  -i = X^(N/2) three times)
        with conj = the rotation under the conjugation key.  Used to run a real-weight projection on two token
        blocks at once (App. "Projection Kernel Breakdown": pairing in the real and imaginary channels)."""
        level = ct.shape[1]
        data = list(range(level))
        bar = self.rotate(ct, conj_key_id)
        re2 = self.ct_add(ct, bar)
        diff = np.stack([self.sub(ct[p], bar[p], data) for p in range(2)])
        im2 = self.mul_monomial_half(self.mul_monomial_half(self.mul_monomial_half(diff)))
        return re2, im2

    # ---- BSGS projection -----------------------------------------------------------
    def giant_sum_deferred(self, accs, giant_key_ids):
        """sum_p rot(acc_p, giant step p) with ONE division by P for the whole sum (a separately defined mode):
            y0 = acc_0[0] + sum_{p>=1} sigma_p(acc_p[0]) + ModDown( sum_{p>=1} raw_p[0] ),
            y1 = acc_0[1]                                 + ModDown( sum_{p>=1} raw_p[1] ),
        raw_p = the key-switch accumulators of sigma_p(acc_p[1]) on the extended basis, added limb-wise.
        Division by P is additive up to its rounding, so the value equals the sum of the separate rotations;
        the residues differ (one rounding instead of n2 - 1) unless there is a single giant step."""
        level = accs[0].shape[1]
        data = list(range(level))
        ext = data + self.special
        y0, y1 = _arr(accs[0][0]).copy(), _arr(accs[0][1]).copy()
        raw = np.zeros((2, len(ext), self.N), dtype=np.uint64)
        for p in range(1, len(accs)):
            kid = giant_key_ids[p]
            g = self.keys[kid][0]
            y0 = self.add(y0, self.automorphism(accs[p][0], g, level), data)
            r = self.key_switch_raw(self.automorphism(accs[p][1], g, level), kid, level)
            raw = np.stack([self.add(raw[c], r[c], ext) for c in range(2)])
        if len(accs) > 1:
            y0 = self.add(y0, self.mod_down(raw[0], level), data)
            y1 = self.add(y1, self.mod_down(raw[1], level), data)
        return np.stack([y0, y1])

    def linear(self, ct_in, diags, desc, baby_key_ids, giant_key_ids, hoist: bool = False, defer: bool = False):
        """Y = XW on packed ciphertexts (App. "Projection Kernel Breakdown", real packing).

        ct_in  [token_blocks, in_blocks, 2, l, N]
        diags  [out_blocks, n2, in_blocks, n1, l, N]  plaintext diagonals D^(b)_{g,p,q}
        returns [token_blocks, out_blocks, 2, l-1, N]:
          acc_p = sum_g sum_q rot(x^(g), q*T) (.) D^(b)_{g,p,q};
          y^(b) = sum_p rot(acc_p, p*n1*T);  then rescale.
        baby_key_ids[q] rotates by q*T (q >= 1), giant_key_ids[p] by p*n1*T (p >= 1).
        hoist=True: the baby rotations use `rotate_hoisted` (different residues, same values).
        defer=True: the giant-step sum uses `giant_sum_deferred` (one division by P per output)."""
        n1, n2 = desc["n1"], desc["n2"]
        tbs, gin = ct_in.shape[0], ct_in.shape[1]
        level = ct_in.shape[3]
        nout = diags.shape[0]
        out = np.empty((tbs, nout, 2, level - 1, self.N), dtype=np.uint64)
        for tb in range(tbs):
            if hoist:   # baby rotations of one input share its decomposition
                rot = [[ct_in[tb, g]] + self.rotate_hoisted(ct_in[tb, g], [baby_key_ids[q] for q in range(1, n1)])
                       for g in range(gin)]
            else:
                rot = [[ct_in[tb, g] if q == 0 else self.rotate(ct_in[tb, g], baby_key_ids[q])
                        for q in range(n1)] for g in range(gin)]
            for b in range(nout):
                y = None
                accs = []
                for p in range(n2):
                    acc = np.zeros((2, level, self.N), dtype=np.uint64)
                    for g in range(gin):
                        for q in range(n1):
                            acc = self.ct_pt_mac(rot[g][q], diags[b, p, g, q], acc)
                    if defer:
                        accs.append(acc)
                        continue
                    if p > 0:
                        acc = self.rotate(acc, giant_key_ids[p])
                    y = acc if y is None else self.ct_add(y, acc)
                if defer:
                    y = self.giant_sum_deferred(accs, giant_key_ids)
                out[tb, b] = self.rescale(y)
        return out

    # ---- causal depthwise convolution (Sec. "Causal Depthwise Convolution", Eq. conv1d_depthwise) ------------
    def conv(self, ct_in, masks, bias, d_conv: int, T: int, key_base: int):
        """eta = b + sum_r M_r (.) rho(q; delta_r) on the projection packing idx(token, channel) = channel*T + token.

        ct_in  [token_blocks, blocks, 2, l, N]   q of every (token block, channel block)
        masks  [blocks, 2*d_conv - 1, l, N]      M_0..M_{d-1}, then M'_1..M'_{d-1} (tap weight times causal mask)
        bias   [blocks, l, N]                    encoded at the scale of the products
        returns [token_blocks, blocks, 2, l-1, N].
        Tap r >= 1 of token k reads token k-r: inside the block that is rho(q; -r) masked to tokens k >= r (M_r); the
        first r tokens read the previous block's last tokens, rho(q_prev; T - r) masked to k < r (M'_r; absent for the
        first block: q_t = 0 for t < 0).  The 2(d_conv-1) rotations of one ciphertext use `rotate_hoisted`; key ids:
        key_base + r for -r, key_base + d_conv + r for T - r."""
        tbs, blocks = ct_in.shape[0], ct_in.shape[1]
        level = ct_in.shape[3]
        data = list(range(level))
        out = np.empty((tbs, blocks, 2, level - 1, self.N), dtype=np.uint64)
        taps = list(range(1, d_conv))
        prev = None
        for tb in range(tbs):
            ids = [key_base + r for r in taps] + ([key_base + d_conv + r for r in taps] if tb + 1 < tbs else [])
            cur = []
            for b in range(blocks):
                rots = self.rotate_hoisted(ct_in[tb, b], ids) if ids else []
                acc = self.ct_pt_mac(ct_in[tb, b], masks[b, 0], np.zeros((2, level, self.N), dtype=np.uint64))
                for i, r in enumerate(taps):
                    acc = self.ct_pt_mac(rots[i], masks[b, r], acc)
                    if prev is not None:
                        acc = self.ct_pt_mac(prev[b][i], masks[b, d_conv - 1 + r], acc)
                acc[0] = self.add(acc[0], _arr(bias[b]), data)
                out[tb, b] = self.rescale(acc)
                cur.append(rots[len(taps):])
            prev = cur if tb + 1 < tbs else None
        return out

    def norm_square(self, y):
        """u = y~ (.) y~ (Alg. "one Block", the squares that feed the NeRMS protocol): ciphertext product with
        relinearisation, then rescale.  y [batch, 2, l, N] -> [batch, 2, l-1, N]."""
        return np.stack([self.rescale(self.ct_ct_mul(c, c)) for c in y])

    def norm_scale(self, y, s, gamma, T: int, key_base: int):
        """y^ = gamma_RMS (.) (y~ (.) br(s_RMS)) (Alg. "one Block", the step before HEOutProj) on the projection
        packing idx(token, channel) = channel*T + token.

        y      [token_blocks, blocks, 2, l, N]   gated scan output of every (token block, channel block)
        s      [token_blocks, 2, l, N]           slot k < T = the inverse RMS of token k, all other slots 0
        gamma  [blocks, l-1, N]                  per-channel weights, slot c*T + k = gamma[channel c of the block]
        returns [token_blocks, blocks, 2, l-2, N].
        br(s): log2(n/T) rotate-right-and-add steps by T*2^b (the rotation by -(T << b) under key id key_base + b),
        shared by the channel blocks of a token block; then a ciphertext product (relinearised, rescaled) and a
        plaintext product (rescaled)."""
        tbs, blocks, level = y.shape[0], y.shape[1], y.shape[3]
        steps = (self.n // T).bit_length() - 1
        assert (T << steps) == self.n and level >= 3
        out = np.empty((tbs, blocks, 2, level - 2, self.N), dtype=np.uint64)
        for tb in range(tbs):
            f = _arr(s[tb])
            for b in range(steps):
                f = self.ct_add(f, self.rotate(f, key_base + b))
            for blk in range(blocks):
                prod = self.rescale(self.ct_ct_mul(y[tb, blk], f))
                zero = np.zeros((2, level - 1, self.N), dtype=np.uint64)
                out[tb, blk] = self.rescale(self.ct_pt_mac(prod, gamma[blk], zero))
        return out

    # ---- harness: encode / decode / encrypt / decrypt ---------------------------------
    def _slot_index(self):
        idx = np.empty(self.n, dtype=np.int64)
        g = 1
        for j in range(self.n):
            idx[j] = (g - 1) // 2
            g = g * 5 % (2 * self.N)
        return idx

    def encode_coeffs(self, z, scale: float) -> np.ndarray:
        """Integer coefficients round(scale * m_i) of the real polynomial m with
        m(zeta^(5^j)) = z_j, zeta = exp(i pi / N); float64 with exact rint."""
        z = np.asarray(z, dtype=np.complex128)
        N = self.N
        vals = np.zeros(N, dtype=np.complex128)
        idx = self._slot_index()
        vals[idx] = z
        vals[N - 1 - idx] = np.conj(z)          # exponent 2N - 5^j  <->  index N-1-(5^j-1)/2
        twist = np.exp(-1j * np.pi * np.arange(N) / N)
        m = np.real(np.fft.fft(vals) * twist) / N
        return np.rint(m * scale).astype(np.int64)

    def encode(self, z, scale: float, level: int) -> np.ndarray:
        data = list(range(level))
        return self.ntt(self.signed_to_rns(self.encode_coeffs(z, scale), data), data)

    def decode_coeffs(self, m) -> np.ndarray:
        """Slots of a real-coefficient polynomial given as float64 coefficients."""
        N = self.N
        twist = np.exp(1j * np.pi * np.arange(N) / N)
        vals = np.fft.ifft(np.asarray(m, dtype=np.float64) * twist) * N
        return vals[self._slot_index()]

    def encrypt(self, pt_eval, nonce: int) -> np.ndarray:
        """Symmetric encryption: c1 = a uniform (EVAL), c0 = -a s + e + m."""
        level = pt_eval.shape[0]
        data = list(range(level))
        a = np.empty((level, self.N), dtype=np.uint64)
        for t in data:
            _lib.orc_sample_uniform(self.seed, make_tag(DOM_ENC_A, nonce, 0, t), self.q[t], a[t], self.N)
        e = np.empty(self.N, dtype=np.int64)
        _lib.orc_sample_cbd(self.seed, make_tag(DOM_ENC_E, nonce), e, self.N)
        e_eval = self.ntt(self.signed_to_rns(e, data), data)
        c0 = self.add(self.add(self.neg(self.mul(a, self.s_eval[:level], data), data), e_eval, data), pt_eval, data)
        return np.stack([c0, a])

    def decrypt_coeffs(self, ct, use_limbs: int | None = None):
        """Centred integer coefficients of c0 + c1 s, CRT-lifted from the first `use_limbs` limbs."""
        level = ct.shape[1]
        k = min(level, use_limbs or level)
        data = list(range(k))
        m = self.add(_arr(ct[0, :k]), self.mul(_arr(ct[1, :k]), self.s_eval[:k], data), data)
        m = self.intt(m, data)
        return crt_lift_centered(m, [self.q[i] for i in data])

    def decrypt(self, ct, scale: float, use_limbs: int | None = None) -> np.ndarray:
        coeffs = self.decrypt_coeffs(ct, use_limbs)
        return self.decode_coeffs(np.array([float(c) for c in coeffs]) / scale)


def crt_lift_centered(res, moduli):
    """Residues [k, n] -> list of n Python ints in (-Q/2, Q/2]."""
    Q = math.prod(moduli)
    n = res.shape[1]
    acc = np.zeros(n, dtype=object)
    for i, q in enumerate(moduli):
        Qi = Q // q
        c = Qi * pow(Qi, -1, q)
        acc = acc + res[i].astype(object) * c
    acc = acc % Q
    return [int(v) - Q if int(v) > Q // 2 else int(v) for v in acc]


def pack_linear_input(x_block, T: int, C: int, n: int) -> np.ndarray:
    """Slots idx(r,c) = c*T + r hold X[r, c] for one (token block, input block)."""
    v = np.zeros(n)
    rows, cols = x_block.shape
    for c in range(cols):
        v[c * T:c * T + rows] = x_block[:, c]
    return v


def linear_diagonal(W, b: int, g: int, p: int, q: int, T: int, C: int, n1: int) -> np.ndarray:
    """D^(b)_{g,p,q}[idx(r,c)] = W[gC + (c+q) mod C, bC + (c - p*n1) mod C], zero outside W."""
    d_in, d_out = W.shape
    c = np.arange(C)
    rows = g * C + (c + q) % C
    cols = b * C + (c - p * n1) % C
    ok = (rows < d_in) & (cols < d_out)
    vals = np.zeros(C)
    vals[ok] = W[rows[ok], cols[ok]]
    return np.repeat(vals, T)


def conv_masks(w, b_conv, blk: int, T: int, C: int, n: int):
    """Slot vectors of one channel block for `Oracle.conv`: w [channels, d_conv] tap weights, b_conv [channels].
    Returns (M [2*d_conv-1, n], bias [n]): M_r[c*T+k] = w[c,r] for k >= r, M'_r[c*T+k] = w[c,r] for k < r."""
    channels, d_conv = w.shape
    M = np.zeros((2 * d_conv - 1, n))
    bias = np.zeros(n)
    for c in range(C):
        ch = blk * C + c
        if ch >= channels:
            break
        bias[c * T:(c + 1) * T] = b_conv[ch]
        for r in range(d_conv):
            M[r, c * T + r:(c + 1) * T] = w[ch, r]
            if r >= 1:
                M[d_conv - 1 + r, c * T:c * T + r] = w[ch, r]
    return M, bias


# ---- token-major packing with periodic diagonals --------------------------------------------------------------
# App. "Projection Kernel Breakdown" defines two slot shifts on the segment view idx(r, s) = s * l_seg + r: the
# whole-segment shift Phi^delta (one rotation) and the intra-segment shift
#   Psi^t(x) = M^stay_t (.) rho(x; t) + M^wrap_t (.) rho(x; t - l_seg)      (two rotations and public masks).
# The projection of this build packs features as segments and tokens inside a segment, so a feature shift is a Phi and
# needs one rotation.  The TRANSPOSED packing, slot r*C + c = X[r, gC + c] (one segment per token, l_seg = C features),
# needs Psi for a feature shift, i.e. two rotations, but every plaintext diagonal then depends on the feature index
# only: the slot vector has period C, the encoded polynomial lives in Z[X^(n/C)], and its evaluation form is constant on
# aligned runs of N/(2C) indices, so a diagonal is N/(2C) times smaller (128 x at N = 2^16, C = 256).
# With the masks folded into the diagonals the product is an ordinary baby-step / giant-step sum over the rotation sets
#   baby  {0} + {q, q - C : 1 <= q < n1},      giant {0} + {p n1, p n1 - C : 1 <= p < n2}
# (2 n1 - 1 and 2 n2 - 1 amounts), which is exactly what `Oracle.linear` evaluates when it is given those keys:
#   y^(b) = sum_G rho( sum_{g, beta} D^(b)_{G,g,beta} (.) rho(x^(g); beta) ; G ).
def token_major_amounts(C: int, n1: int, n2: int):
    """(baby amounts, giant amounts) in slot order: index 0 is the identity, 2q-1 / 2q are q and q - C (baby),
    2p-1 / 2p are p*n1 and p*n1 - C (giant)."""
    baby = [0] + [a for q in range(1, n1) for a in (q, q - C)]
    giant = [0] + [a for p in range(1, n2) for a in (p * n1, p * n1 - C)]
    return baby, giant


def pack_linear_input_token_major(x_block, T: int, C: int, n: int) -> np.ndarray:
    """Slots r*C + c hold X[r, c] for one (token block, input block)."""
    v = np.zeros((T, C))
    rows, cols = x_block.shape
    v[:rows, :cols] = x_block
    return v.reshape(n)


def linear_diagonal_token_major(W, b: int, g: int, gi: int, bi: int, T: int, C: int, n1: int) -> np.ndarray:
    """Diagonal of giant slot gi and baby slot bi (see token_major_amounts) for output block b and input block g.
    Output feature c' = c'' - P (stay) or c'' + C - P (wrap) is assembled at position c'' of the accumulator; it takes
    input feature (c'' + q) mod C, which the baby rotation by q delivers where c'' + q < C and the one by q - C where
    c'' + q >= C.  The vector depends on c'' only (period C)."""
    d_in, d_out = W.shape
    p, wrap_g = ((gi + 1) // 2, gi % 2 == 0) if gi else (0, False)
    q, wrap_b = ((bi + 1) // 2, bi % 2 == 0) if bi else (0, False)
    P = p * n1
    cpp = np.arange(C)
    support_g = (cpp < P) if wrap_g else (cpp >= P)              # positions this accumulator owns
    c_out = cpp + C - P if wrap_g else cpp - P
    support_b = (cpp + q >= C) if wrap_b else (cpp + q < C)      # positions this baby rotation serves
    c_in = (cpp + q) % C
    rows, cols = g * C + c_in, b * C + c_out
    ok = support_g & support_b & (rows < d_in) & (cols < d_out) & (cols >= b * C)
    vals = np.zeros(C)
    vals[ok] = W[rows[ok], cols[ok]]
    return np.tile(vals, T)


def periodic_eval_runs(pt_eval: np.ndarray, run: int) -> np.ndarray:
    """One word per aligned run of `run` evaluation indices of a plaintext whose slot vector is periodic (asserts that
    the runs are constant): the compressed form of a token-major diagonal, [limbs, N / run]."""
    k, N = pt_eval.shape
    v = pt_eval.reshape(k, N // run, run)
    assert np.all(v == v[:, :, :1]), "not constant on runs: the slot vector is not periodic"
    return np.ascontiguousarray(v[:, :, 0])
