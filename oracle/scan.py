"""CPU oracle for the factorized scan-contract (TEST INFRASTRUCTURE).

Ideal semantics (Sec. 5.4, Eqs. fesc_recurrence / fesc_contract):

    h_k = br(a_k) (.) h_{k-1} + x_k (x)_g B_k,   h_0 = 0,      m_k = Sigma_{d_s}( h_k (.) br(C_k) )

with x_k in R^{H x P}, a_k in R^H, B_k, C_k in R^{G x d_s} (G = 1 here).  `float_recurrence` evaluates this
definition with a sequential float64 loop; it is the reference every encrypted result is compared with.

Homomorphic realisation.  The paper fixes the contract, the affine composition
(Eq. compact_affine_compose:  T_R o T_L = (a_R (.) a_L, br(a_R) (.) s_L + s_R)), the on-demand build and
contraction (Eq. hescan-contract-output), the blocked schedule with carries (Eq. resident-block-schedule, in its
serialized-carry form of App. "longer sequences"), the Brent-Kung network (App. "Prefix-Network Selection") and
the complex-paired state reduction (App. "Complex-Packed Reduction Accounting"); it does not give the slot-level
broadcast maps.  The dataflow below is this build's reading, stated in full in this header; the CUDA library
implements the same graph independently and must reproduce every residue.

Geometry (all powers of two).  n slots = c_state * stride, stride >= max(d_s, B_blk); one state ciphertext of
chunk kappa holds coordinate (e = kappa*c_state + e', i) at slot e'*stride + i (i < d_s; the rest idle).
hpc = c_state / P heads per chunk, each owning a slot region of R = n / hpc = P*stride slots.
A block of B tokens is cut into segs = max(1, B/stride) segments of Bt = B/segs tokens; x, a and the output have one
ciphertext per segment (stride >= B, one segment, is the paper's deployed shape with half of the state slots idle;
stride = d_s < B uses every slot: s_state = n, half as many chunks).
Inputs per token block j (B = B_blk tokens, t = token within the block; for X, A and the output t is the offset inside
the segment and the arrays carry a segment axis after the chunk axis):
    X[j][kappa]: slot e'*stride + t      = x_{jB+t}[kappa*c_state + e']          scale S_s[l0]
    A[j][kappa]: slot hh*R + t*P          = a_{jB+t}[kappa*hpc + hh], else 0       scale S_p[l0]
    Bc[j], Cc[j]: slot t*d_s + i          = B_{jB+t}[i], C_{jB+t}[i]               scale S_p[l0]
Output per (j, kappa): slot e'*stride + t = m_{jB+t}[kappa*c_state + e'], level l_out, scale S_s[l_out].

Scales.  Two canonical families per level: S_s (state-like values) and S_p (multiplicands), with
S_s[l-1] = S_s[l] S_p[l] / q_{l-1},  S_p[l-1] = S_p[l]^2 / q_{l-1},  S_s[l0] = 2^log_scale, S_p[l0] = q_{l0-1}.
Every product is s x p or p x p of operands at the same level, followed by a rescale.  An operand that sits at a
higher level is brought down by `adjust`: keep its first l_dst+1 limbs, multiply by the integer
round(S[l_dst] q_{l_dst} / S[l_src]), rescale.  Masks are plaintexts at scale S_p of their level.

Level schedule (logB = log2 B):  inputs l0;  masked / filled factors l0-1 (br(C): masked at l0-1, brought to linj-1,
filled there);  leaves (p, s) at l1 = l0-2;
up-sweep stage s -> l1-s;  summaries at lS = l1-logB;  down-sweep stage number d (1..logB-1) works at
lS-(d-1) -> lS-d;  carries g_j (j >= 1) at lS-(j-1);  injection at linj = l1-2logB+1 -> states at linj-1;
contraction -> linj-2;  reduction, conjugation, unpacking there;  output mask -> l_out = linj-3.

Grouped leaf build (`group` = G > 0, a separately defined mode: other residues, same values).  Building br(x_t) and
br(a_t) token by token costs log2(d_s) and log2(R/P) rotate-and-add steps per token at the top levels.  With groups of
G consecutive tokens the group is extracted, masked (slots [0,G) of every stride for x, [0,GP) of every head region for
a) and filled ONCE for its G tokens (log2(d_s/G), log2(R/(GP)) steps: the pattern of G tokens repeats with period G
slots resp. G blocks of P slots).  The copies of token g of the group sit in class g of every period; class j of its
broadcast takes them from class g, i.e. from the group ciphertext rotated by (g - j) units, so

    br(token g of the group) = rescale( sum_{j<G} classmask_j (.) rot(group, (g - j) unit) ),   unit = 1 (x), P (a):

the 2(G-1) rotations by +-unit..+-(G-1) unit are taken ONCE per group (one decomposition in hoisted mode) and every
token is G plaintext multiply-accumulates and one rescale (no copy leaves its period, so nothing crosses a channel or
head boundary).  The class masks cost one level: leaves at l1 = l0-3.  br(B_t) is built the same way (groups of G
tokens = G d_s consecutive slots, mask [0, G d_s), log2(n/(G d_s)) steps, class shifts of d_s slots), which lands it
at l0-2 where the leaves need it; br(C_t) keeps the token-by-token build (its fill runs at the injection level, where
rotations are cheap).

Invariant families (App. "Invariant Families", "Shared HEScan Kernel Backend"; `plain` = (abar, Bbar, Cbar); S4D / S5 /
LRU rows of Table "cross_ssm_family").  The decay abar[i] (per state coordinate), the input factor Bbar[i] and the output
factor Cbar[i] are server-held plaintexts that do not depend on the token; only x_k is encrypted:
    h_k[e,i] = abar[i] h_{k-1}[e,i] + x_k[e] Bbar[i],     m_k[e] = sum_i h_k[e,i] Cbar[i].
The affine packet loses its decay component: the decay over a span of m tokens is the plaintext abar^m, so a composition
is  s <- abar^m (.) s_L + s_R  with ONE ct-pt product and no ciphertext product anywhere ("Affine relin." 0 in the
paper's table).  Everything else (layouts, br(x_t), Brent-Kung schedule, levels, carries, reduction) is the dataflow
above with plaintexts in place of br(a), br(B), br(C): leaf s_t = br(x_t) (.) Bbar; up-sweep stage s and the down-sweep
stage over the same span use abar^(2^(s-1)); the carry uses abar^B; the injection of token t uses abar^(t+1); the
contraction uses Cbar.  Every plaintext is a slot pattern e'*stride + i -> v[i] encoded at scale S_p of the level where
it is used.

Other prefix networks (App. "Prefix-Network Selection"; `network` = "ks" Kogge-Stone, "sk" Sklansky; "bk" above is the
default): stage s = 1..logB combines operands at l1-(s-1) into results at l1-s, every prefix is complete at lS and there
is no down-sweep, so linj = lS - max(K_blk-2, 0) (the carry before the last block still sits at or above linj).
"""
from __future__ import annotations

import math

import numpy as np

from .ckks import CONJ, Oracle


# ---------------------------------------------------------------------------------------------
# ideal semantics
# ---------------------------------------------------------------------------------------------
def float_recurrence(x, a, B, C):
    """m[k,h,p] = sum_i h_k[h,p,i] C_k[0,i],  h_k = a_k[h] h_{k-1} + x_k[h,p] B_k[0,i]  (float64, sequential)."""
    L, H, P = x.shape
    d_s = B.shape[2]
    h = np.zeros((H, P, d_s))
    m = np.zeros((L, H, P))
    for k in range(L):
        h = a[k][:, None, None] * h + x[k][:, :, None] * B[k, 0][None, None, :]
        m[k] = h @ C[k, 0]
    return m


def float_recurrence_invariant(x, abar, Bbar, Cbar):
    """Invariant families (App. "Invariant Families"): m[k,h,p] = sum_i h_k[h,p,i] Cbar[i],
    h_k[h,p,i] = abar[i] h_{k-1}[h,p,i] + x_k[h,p] Bbar[i]  (float64, sequential)."""
    L, H, P = x.shape
    h = np.zeros((H, P, len(abar)))
    m = np.zeros((L, H, P))
    for k in range(L):
        h = abar[None, None, :] * h + x[k][:, :, None] * Bbar[None, None, :]
        m[k] = h @ Cbar
    return m


class ScanShape:
    def __init__(self, n, L, H, P, d_s, B_blk, stride=None):
        self.n, self.L, self.H, self.P, self.d_s, self.B = n, L, H, P, d_s, B_blk
        self.stride = stride or max(d_s, B_blk)
        self.c_state = n // self.stride
        self.E = H * P
        assert self.c_state * self.stride == n and self.stride >= d_s
        assert self.stride >= B_blk or B_blk % self.stride == 0
        self.segs = max(1, B_blk // self.stride)      # token segments of a block: one x / a / output ciphertext each
        self.Bt = B_blk // self.segs                   # tokens per segment
        assert self.c_state % P == 0 and self.E % self.c_state == 0
        self.hpc = self.c_state // P
        self.R = n // self.hpc
        self.K_s = self.E // self.c_state
        self.K_blk = -(-L // B_blk)
        self.logB = int(math.log2(B_blk))
        assert 1 << self.logB == B_blk and B_blk >= 2
        assert B_blk * d_s <= n and self.Bt * P <= self.R
        self.dg = min(16, B_blk)                      # base of the two-digit token offset t = t_lo + dg*t_hi (B, C)
        self.dgt = min(16, self.Bt)                   # ... of the offset inside a segment (x, a, output)

    # rotation amounts (slot LEFT shifts, modulo n) the dataflow uses
    def chains(self):
        """(signed unit, steps) of every rotate-and-add chain ct += rot(ct, unit * 2^b), b = 0..steps-1."""
        lg = lambda v: int(math.log2(v))
        return [(-1, lg(self.P)), (-1, lg(self.d_s)), (-self.P, lg(self.R // self.P)),
                (-self.stride, lg(self.c_state)), (1, lg(self.d_s))]

    @staticmethod
    def class_shifts(G: int, unit: int):
        """Rotation amounts (LEFT positive) of the grouped leaf build, in the order the rotated copies are kept:
        +unit, .., +(G-1) unit, -unit, .., -(G-1) unit.  The copy for class difference g - j = k sits at index k - 1
        (k > 0) or G - 2 - k (k < 0)."""
        return [k * unit for k in range(1, G)] + [-k * unit for k in range(1, G)]

    def rotation_amounts(self, hoist: bool = False, group: int = 0):
        """hoist=True adds the amounts 3 * unit * 2^b of the radix-4 chains (b even, b + 1 < steps); group=G adds the
        group extraction amounts and the class shifts +-unit .. +-(G-1) unit."""
        n, dg, B, dgt, Bt = self.n, self.dg, self.B, self.dgt, self.Bt
        am = set()
        for unit in (1, self.P):                      # extraction of x, a (offsets inside a segment)
            am |= {unit * t % n for t in range(1, dgt)} | {unit * dgt * t % n for t in range(1, Bt // dgt)}
        am |= {self.d_s * t % n for t in range(1, dg)} | {self.d_s * dg * t % n for t in range(1, B // dg)}   # B, C
        am |= {(-t) % n for t in range(1, dgt)} | {(-dgt * t) % n for t in range(1, Bt // dgt)}   # output placement
        am |= {(-(1 << b)) % n for b in range(int(math.log2(max(self.d_s, self.P))))}    # x fill, a pre-fill
        am |= {(-self.P * (1 << b)) % n for b in range(int(math.log2(self.R // self.P)))}        # a fill
        am |= {(-self.stride * (1 << b)) % n for b in range(int(math.log2(self.c_state)))}       # B, C fill
        am |= {(1 << b) for b in range(int(math.log2(self.d_s)))}                        # state reduction
        if hoist:
            for unit, steps in self.chains():
                am |= {(3 * unit * (1 << b)) % n for b in range(0, steps - 1, 2)}
        if group:
            G = group
            cnt = Bt // G
            dgg = min(16, cnt)
            for unit in (G, G * self.P):                                                   # extraction of the groups
                am |= {unit * t % n for t in range(1, dgg)} | {unit * dgg * t % n for t in range(1, cnt // dgg)}
            if hoist:                                                                      # radix-4 group fills
                for unit, steps in ((-G, int(math.log2(self.d_s // G))), (-G * self.P, int(math.log2(self.R // (G * self.P))))):
                    am |= {(3 * unit * (1 << b)) % n for b in range(0, steps - 1, 2)}
            for unit in (1, self.P, self.d_s):
                am |= {v % n for v in self.class_shifts(G, unit)}
            cntB = B // G                                                                  # groups of br(B)
            dgB = min(16, cntB)
            unit = G * self.d_s
            am |= {unit * t % n for t in range(1, dgB)} | {unit * dgB * t % n for t in range(1, cntB // dgB)}
            if hoist:
                am |= {(-3 * unit * (1 << b)) % n for b in range(0, int(math.log2(n // unit)) - 1, 2)}
            am |= {(-unit * (1 << b)) % n for b in range(int(math.log2(n // unit)))}
        am.discard(0)
        return sorted(am)


NETWORKS = ("bk", "ks", "sk")


def levels(l0: int, logB: int, K_blk: int, network: str = "bk", group: int = 0):
    assert network in NETWORKS
    l1 = l0 - 3 if group else l0 - 2
    lS = l1 - logB
    linj = l1 - 2 * logB + 1 if network == "bk" else lS - max(K_blk - 2, 0)
    lout = linj - 3
    assert lout >= 1, "not enough levels"
    assert K_blk <= 1 or lS - (K_blk - 2) >= linj, "carry chain runs below the injection level"
    return dict(l0=l0, l1=l1, lS=lS, linj=linj, lout=lout)


class ScanConsts:
    """Harness-side constants: canonical scales, level-adjust integers, mask plaintexts."""

    def __init__(self, orc: Oracle, shape: ScanShape, l0: int, log_scale: int, network: str = "bk", group: int = 0,
                 plain=None):
        """plain = (abar, Bbar, Cbar), three float vectors of length d_s: the invariant-family mode (module header)."""
        q = orc.q
        self.network, self.group, self.plain = network, group, plain is not None
        self.lv = levels(l0, shape.logB, shape.K_blk, network, group)
        self.S_s = {l0: float(2**log_scale)}
        self.S_p = {l0: float(q[l0 - 1])}
        for l in range(l0, 1, -1):
            self.S_s[l - 1] = self.S_s[l] * self.S_p[l] / q[l - 1]
            self.S_p[l - 1] = self.S_p[l] ** 2 / q[l - 1]
        for l in range(2, l0 + 1):
            assert abs(self.S_p[l] / q[l - 1] - 1) < 0.25, "prime chain too uneven for the scale schedule"
        # adjust integers: [src][dst]
        self.adj_s = {(a, b): int(round(self.S_s[b] * q[b] / self.S_s[a])) for a in range(2, l0 + 1) for b in range(1, a)}
        self.adj_p = {(a, b): int(round(self.S_p[b] * q[b] / self.S_p[a])) for a in range(2, l0 + 1) for b in range(1, a)}
        n, st = shape.n, shape.stride
        mx = np.zeros(n)
        mx[::st] = 1.0
        mb = np.zeros(n)
        mb[:shape.d_s] = 1.0
        ma = np.zeros(n)
        for hh in range(shape.hpc):
            ma[hh * shape.R: hh * shape.R + shape.P] = 1.0
        self.mask_x = orc.encode(mx, self.S_p[l0], l0)
        self.mask_b = orc.encode(mb, self.S_p[l0], l0)
        self.mask_a = orc.encode(ma, self.S_p[l0], l0)
        if group:
            G, P, R, d_s = group, shape.P, shape.R, shape.d_s
            assert G >= 2 and G & (G - 1) == 0 and G <= min(shape.Bt, d_s) and G * P <= R
            slot = np.arange(n)
            in_stride, in_region = slot % st, slot % R
            self.mask_xg = orc.encode((in_stride < G).astype(float), self.S_p[l0], l0)
            self.mask_ag = orc.encode((in_region < G * P).astype(float), self.S_p[l0], l0)
            self.mask_x2 = np.stack([orc.encode(((in_stride < d_s) & (in_stride % G == g)).astype(float),
                                                self.S_p[l0 - 1], l0 - 1) for g in range(G)])
            self.mask_a2 = np.stack([orc.encode(((in_region // P) % G == g).astype(float), self.S_p[l0 - 1], l0 - 1)
                                     for g in range(G)])
            self.mask_bg = orc.encode((slot < G * d_s).astype(float), self.S_p[l0], l0)
            self.mask_b2 = np.stack([orc.encode(((slot // d_s) % G == g).astype(float), self.S_p[l0 - 1], l0 - 1)
                                     for g in range(G)])
        if plain is not None:
            assert network == "bk", "the invariant-family mode uses the Brent-Kung schedule"
            abar, Bbar, Cbar = (np.asarray(v, dtype=np.float64) for v in plain)
            assert abar.shape == Bbar.shape == Cbar.shape == (shape.d_s,)
            lv, B, logB = self.lv, shape.B, shape.logB

            def pt(vec, level):     # slot e'*stride + i -> vec[i], encoded where it multiplies
                slots = np.zeros((shape.c_state, st))
                slots[:, :shape.d_s] = vec[None, :]
                return orc.encode(slots.reshape(-1), self.S_p[level], level)

            lx = l0 - 2 if group else l0 - 1                       # level of br(x_t)
            self.pt_b = pt(Bbar, lx)
            self.pt_c = pt(Cbar, lv["linj"] - 1)
            self.pt_up = {s: pt(abar ** (1 << (s - 1)), lv["l1"] - (s - 1)) for s in range(1, logB + 1)}
            self.pt_down = {d: pt(abar ** (1 << (logB - d - 1)), lv["lS"] - (d - 1)) for d in range(1, logB)}
            self.pt_carry = {j: pt(abar ** B, lv["lS"] - (j - 1)) for j in range(1, shape.K_blk - 1)}
            self.pt_inj = [pt(abar ** (t + 1), lv["linj"]) for t in range(B)] if shape.K_blk > 1 else []
        lred, lout = self.lv["linj"] - 2, self.lv["lout"]
        # the unpacked reduction carries a factor 2 (Re*2, Im*2); the output mask removes it and lands on S_s[lout]
        self.out_mask_scale = self.S_s[lout] * q[lout] / (2.0 * self.S_s[lred])
        self.mask_out = orc.encode(mx, self.out_mask_scale, lred)
        self.out_scale = self.S_s[lout]


def key_id_for(shape: ScanShape, amount: int, base: int = 100000) -> int:
    return base + shape.n if amount == CONJ else base + amount % shape.n


def add_scan_keys(orc: Oracle, shape: ScanShape, base: int = 100000, hoist: bool = False, group: int = 0):
    for r in shape.rotation_amounts(hoist, group):
        if key_id_for(shape, r, base) not in orc.keys:
            orc.add_galois_key(r, key_id_for(shape, r, base))
    if key_id_for(shape, CONJ, base) not in orc.keys:
        orc.add_galois_key(CONJ, key_id_for(shape, CONJ, base))


def pack_inputs(shape: ScanShape, x, a, B, C):
    """Slot vectors of the compact factors: dict name -> array [K_blk, (K_s,) n]."""
    sh = shape
    X = np.zeros((sh.K_blk, sh.K_s, sh.segs, sh.n))
    A = np.zeros((sh.K_blk, sh.K_s, sh.segs, sh.n))
    Bc = np.zeros((sh.K_blk, sh.n))
    Cc = np.zeros((sh.K_blk, sh.n))
    xf = x.reshape(sh.L, sh.E)
    for k in range(sh.L):
        j, t = divmod(k, sh.B)
        Bc[j, t * sh.d_s:(t + 1) * sh.d_s] = B[k, 0]
        Cc[j, t * sh.d_s:(t + 1) * sh.d_s] = C[k, 0]
        seg, tt = divmod(t, sh.Bt)
        for kap in range(sh.K_s):
            X[j, kap, seg, np.arange(sh.c_state) * sh.stride + tt] = xf[k, kap * sh.c_state:(kap + 1) * sh.c_state]
            for hh in range(sh.hpc):
                A[j, kap, seg, hh * sh.R + tt * sh.P] = a[k, kap * sh.hpc + hh]
    return X, A, Bc, Cc


def encrypt_inputs(orc: Oracle, shape: ScanShape, consts: ScanConsts, x, a, B, C, nonce0: int = 50000):
    X, A, Bc, Cc = pack_inputs(shape, x, a, B, C)
    l0 = consts.lv["l0"]
    nonce = [nonce0]

    def enc(v, scale):
        nonce[0] += 1
        return orc.encrypt(orc.encode(v, scale, l0), nonce[0])

    segs = range(shape.segs)
    ctX = np.stack([np.stack([np.stack([enc(X[j, k, g], consts.S_s[l0]) for g in segs]) for k in range(shape.K_s)])
                    for j in range(shape.K_blk)])
    ctA = np.stack([np.stack([np.stack([enc(A[j, k, g], consts.S_p[l0]) for g in segs]) for k in range(shape.K_s)])
                    for j in range(shape.K_blk)])
    ctB = np.stack([enc(Bc[j], consts.S_p[l0]) for j in range(shape.K_blk)])
    ctC = np.stack([enc(Cc[j], consts.S_p[l0]) for j in range(shape.K_blk)])
    return ctX, ctA, ctB, ctC


def encrypt_x(orc: Oracle, shape: ScanShape, consts: ScanConsts, x, nonce0: int = 50000):
    """Invariant-family mode: only the scan input is encrypted.  [K_blk, K_s, segs, 2, l0, N], the layout of X above."""
    l0 = consts.lv["l0"]
    X, _, _, _ = pack_inputs(shape, x, np.zeros((shape.L, shape.H)), np.zeros((shape.L, 1, shape.d_s)),
                             np.zeros((shape.L, 1, shape.d_s)))
    nonce = nonce0
    rows = []
    for j in range(shape.K_blk):
        for k in range(shape.K_s):
            for g in range(shape.segs):
                nonce += 1
                rows.append(orc.encrypt(orc.encode(X[j, k, g], consts.S_s[l0], l0), nonce))
    return np.stack(rows).reshape(shape.K_blk, shape.K_s, shape.segs, 2, l0, orc.N)


def unpack_output(orc: Oracle, shape: ScanShape, consts: ScanConsts, out):
    """out [K_blk, K_s, segs, 2, l_out, N] -> m [L, H, P] (float64, decrypted)."""
    sh = shape
    m = np.zeros((sh.K_blk * sh.B, sh.E))
    for j in range(sh.K_blk):
        for kap in range(sh.K_s):
            for seg in range(sh.segs):
                slots = orc.decrypt(out[j, kap, seg], consts.out_scale, 2).real
                for tt in range(sh.Bt):
                    m[j * sh.B + seg * sh.Bt + tt, kap * sh.c_state:(kap + 1) * sh.c_state] = \
                        slots[np.arange(sh.c_state) * sh.stride + tt]
    return m[:sh.L].reshape(sh.L, sh.H, sh.P)


# ---------------------------------------------------------------------------------------------
# homomorphic evaluation
# ---------------------------------------------------------------------------------------------
class ScanEvaluator:
    def __init__(self, orc: Oracle, shape: ScanShape, consts: ScanConsts, key_base: int = 100000, hoist: bool = False):
        """hoist=True (a separately defined mode, other residues, same values): rotate-and-add chains take two
        steps at once as ct + rot(ct, d) + rot(ct, 2d) + rot(ct, 3d) with one decomposition and one division by P
        (`rotate_sum_hoisted`), and the low digit of the two-digit token offsets uses `rotate_hoisted`."""
        self.o, self.sh, self.c, self.kb, self.hoist = orc, shape, consts, key_base, hoist
        self.network = consts.network       # the level schedule in `consts` belongs to one network
        self.group = consts.group           # ... and to one leaf build
        self.count = dict(rot=0, conj=0, ctmul=0, adjust=0, ptmul=0, compose=0)

    # -- primitives ---------------------------------------------------------------------------
    def rot(self, ct, amount):
        amount %= self.sh.n
        if amount == 0:
            return ct
        self.count["rot"] += 1
        return self.o.rotate(ct, key_id_for(self.sh, amount, self.kb))

    def conj(self, ct):
        self.count["conj"] += 1
        return self.o.rotate(ct, key_id_for(self.sh, CONJ, self.kb))

    def add(self, a, b):
        return self.o.ct_add(a, b)

    def sub(self, a, b):
        lv = list(range(a.shape[1]))
        return np.stack([self.o.sub(a[p], b[p], lv) for p in range(2)])

    def ptmul_rescale(self, ct, pt):
        self.count["ptmul"] += 1
        return self.o.rescale(self.o.ct_pt_mac(ct, pt, np.zeros_like(ct)))

    def mul_rescale(self, a, b):
        self.count["ctmul"] += 1
        return self.o.rescale(self.o.ct_ct_mul(a, b))

    def adjust(self, ct, dst, kind):
        src = ct.shape[1]
        if src == dst:
            return ct
        self.count["adjust"] += 1
        k = (self.c.adj_s if kind == "s" else self.c.adj_p)[(src, dst)]
        lv = list(range(dst + 1))
        cut = np.ascontiguousarray(ct[:, :dst + 1])
        scaled = np.stack([self.o.mul_scalar(cut[p], [k] * (dst + 1), lv) for p in range(2)])
        return self.o.rescale(scaled)

    def chain(self, ct, unit, steps):
        """ct += rot(ct, unit*2^b) for b = 0..steps-1 (unit signed).  Hoisted mode: steps (b, b+1) together."""
        b = 0
        while b < steps:
            d = unit * (1 << b)
            if self.hoist and b + 1 < steps:
                self.count["rot"] += 3
                ct = self.o.rotate_sum_hoisted(ct, [key_id_for(self.sh, k * d, self.kb) for k in (1, 2, 3)])
                b += 2
            else:
                ct = self.add(ct, self.rot(ct, d))
                b += 1
        return ct

    def class_broadcasts(self, group_ct, masks, unit):
        """[rescale(sum_j masks[j] (.) rot(group_ct, (g - j) unit)) for g < G]: the broadcasts of the G tokens of one
        filled group ciphertext.  The 2(G-1) rotations are taken once (hoisted mode: one decomposition)."""
        G = self.group
        shifts = self.sh.class_shifts(G, unit)
        if self.hoist:
            self.count["rot"] += len(shifts)
            rots = self.o.rotate_hoisted(group_ct, [key_id_for(self.sh, d, self.kb) for d in shifts])
        else:
            rots = [self.rot(group_ct, d) for d in shifts]
        out = []
        for g in range(G):
            acc = np.zeros_like(group_ct)
            for j in range(G):
                k = g - j
                src = group_ct if k == 0 else rots[k - 1 if k > 0 else G - 2 - k]
                acc = self.o.ct_pt_mac(src, masks[j], acc)
            self.count["ptmul"] += G
            out.append(self.o.rescale(acc))
        return out

    def fill_right(self, ct, unit, steps):
        """ct += rot(ct, -unit*2^b) for b = 0..steps-1 (copies a block to 2^steps consecutive blocks)."""
        return self.chain(ct, -unit, steps)

    def extract_all(self, ct, unit, count=None):
        """[rot(ct, unit*t) for t < count (default B)] with t = t_lo + dg*t_hi, dg = min(16, count):
        rot(ct, unit*dg*t_hi) first, then the low digit (in hoisted mode the dg-1 low-digit rotations of one
        ciphertext share its decomposition)."""
        sh = self.sh
        count = sh.B if count is None else count
        dg = min(16, count)
        out = [None] * count
        for th in range(count // dg):
            g = ct if th == 0 else self.rot(ct, unit * dg * th)
            out[th * dg] = g
            if self.hoist and dg > 1:
                self.count["rot"] += dg - 1
                lows = self.o.rotate_hoisted(g, [key_id_for(sh, unit * tl, self.kb) for tl in range(1, dg)])
                for tl in range(1, dg):
                    out[th * dg + tl] = lows[tl - 1]
            else:
                for tl in range(1, dg):
                    out[th * dg + tl] = self.rot(g, unit * tl)
        return out

    def compose(self, left, right, lvl, need_p=True):
        """(p_L, s_L) then (p_R, s_R), all brought to level lvl; result at lvl-1:
        (p_R p_L,  p_R s_L + s_R)   (Eq. compact_affine_compose)."""
        self.count["compose"] += 1
        pL, sL = self.adjust(left[0], lvl, "p") if need_p else None, self.adjust(left[1], lvl, "s")
        pR, sR = self.adjust(right[0], lvl, "p"), self.adjust(right[1], lvl - 1, "s")
        p = self.mul_rescale(pR, pL) if need_p else None
        s = self.add(self.mul_rescale(pR, sL), sR)
        return (p, s)

    # -- one token block ----------------------------------------------------------------------
    def broadcast_bc(self, ct, level=None):
        """brB_t (or brC_t) for every token of the block, value B_t[i] at every (e', i): level l0-1, or brought down
        to `level` BEFORE the rotate-and-add fill (br(C) is only needed at the injection level, where a rotation
        costs a fraction of one at the top level)."""
        sh, c = self.sh, self.c
        ex = self.extract_all(ct, sh.d_s)
        out = []
        for t in range(sh.B):
            u = self.ptmul_rescale(ex[t], c.mask_b)
            if level is not None:
                u = self.adjust(u, level, "p")
            out.append(self.fill_right(u, sh.stride, int(math.log2(sh.c_state))))
        return out

    def broadcast_b_grouped(self, ct):
        """br(B_t) for every token of the block at l0-2, built for groups of G tokens (module header)."""
        sh, c, G = self.sh, self.c, self.group
        unit = G * sh.d_s
        ex = self.extract_all(ct, unit, sh.B // G)
        out = []
        for u in range(sh.B // G):
            gb = self.fill_right(self.ptmul_rescale(ex[u], c.mask_bg), unit, int(math.log2(sh.n // unit)))
            out += self.class_broadcasts(gb, c.mask_b2, sh.d_s)
        return out

    def leaves(self, ctX, ctA, brB):
        """ctX, ctA: the `segs` ciphertexts of one (block, chunk), segment g holding the tokens g*Bt .. (g+1)*Bt-1."""
        sh, c = self.sh, self.c
        l1 = c.lv["l1"]
        T = []
        for seg in range(sh.segs):
            apre = self.fill_right(ctA[seg], 1, int(math.log2(sh.P)))
            ex, ea = self.extract_all(ctX[seg], 1, sh.Bt), self.extract_all(apre, sh.P, sh.Bt)
            for tt in range(sh.Bt):
                xr = self.ptmul_rescale(ex[tt], c.mask_x)
                xr = self.fill_right(xr, 1, int(math.log2(sh.d_s)))
                ar = self.adjust(self.ptmul_rescale(ea[tt], c.mask_a), l1, "p")        # to the leaf level, then fill
                ar = self.fill_right(ar, sh.P, int(math.log2(sh.R // sh.P)))
                s = self.mul_rescale(xr, brB[seg * sh.Bt + tt])
                T.append((ar, s))
        return T

    def leaves_grouped(self, ctX, ctA, brB):
        """Leaves (br a_t, br x_t (.) br B_t) at l1 = l0-3 with the grouped build (module header): groups of G tokens
        are extracted, masked and filled once; masked sums of the group's 2(G-1) rotations separate the tokens."""
        sh, c, G = self.sh, self.c, self.group
        l1, lg = c.lv["l1"], lambda v: int(math.log2(v))
        T = []
        for seg in range(sh.segs):
            apre = self.fill_right(ctA[seg], 1, lg(sh.P))
            gx = self.extract_all(ctX[seg], G, sh.Bt // G)
            ga = self.extract_all(apre, G * sh.P, sh.Bt // G)
            for u in range(sh.Bt // G):
                xg = self.fill_right(self.ptmul_rescale(gx[u], c.mask_xg), G, lg(sh.d_s // G))
                ag = self.fill_right(self.ptmul_rescale(ga[u], c.mask_ag), G * sh.P, lg(sh.R // (G * sh.P)))
                bx, ba = self.class_broadcasts(xg, c.mask_x2, 1), self.class_broadcasts(ag, c.mask_a2, sh.P)
                for g in range(G):
                    ar = self.adjust(ba[g], l1, "p")
                    T.append((ar, self.mul_rescale(bx[g], brB[seg * sh.Bt + u * G + g])))
        return T

    def brent_kung(self, T, need_p_down):
        """In-place inclusive prefix over T[0..B-1] (1-based positions k <-> T[k-1]).
        Returns the summary (the last position after the up-sweep)."""
        sh, c = self.sh, self.c
        B, logB, l1, lS = sh.B, sh.logB, c.lv["l1"], c.lv["lS"]
        for s in range(1, logB + 1):
            for k in range(1 << s, B + 1, 1 << s):
                T[k - 1] = self.compose(T[k - (1 << (s - 1)) - 1], T[k - 1], l1 - (s - 1))
        summary = T[B - 1]
        d = 0
        for s in range(logB - 1, 0, -1):
            d += 1
            for k in range(1 << s, B, 1 << s):
                r = k + (1 << (s - 1))
                if r < B:
                    T[r - 1] = self.compose(T[k - 1], T[r - 1], lS - (d - 1), need_p=need_p_down)
        return summary

    def kogge_stone(self, T, last_p):
        """Kogge-Stone network (App. "Prefix-Network Selection"): at stage s every position k > 2^(s-1) (1-based)
        takes t_k <- t_{k - 2^(s-1)} o t_k with both operands from stage s-1.  B log2 B - (B-1) compositions."""
        sh, l1 = self.sh, self.c.lv["l1"]
        for s in range(1, sh.logB + 1):
            d = 1 << (s - 1)
            prev = list(T)
            for k in range(d + 1, sh.B + 1):
                T[k - 1] = self.compose(prev[k - d - 1], prev[k - 1], l1 - (s - 1), need_p=(s < sh.logB or last_p))
        return T[sh.B - 1]

    def sklansky(self, T, last_p):
        """Sklansky network: at stage s the positions of the upper half of every aligned block of 2^s (0-based
        k in [b 2^s + 2^(s-1), (b+1) 2^s)) take t_k <- t_{b 2^s + 2^(s-1) - 1} o t_k.  (B/2) log2 B compositions."""
        sh, l1 = self.sh, self.c.lv["l1"]
        for s in range(1, sh.logB + 1):
            half = 1 << (s - 1)
            prev = list(T)
            for b in range(sh.B >> s):
                src = (b << s) + half - 1
                for k in range(src + 1, (b + 1) << s):
                    T[k] = self.compose(prev[src], prev[k], l1 - (s - 1), need_p=(s < sh.logB or last_p))
        return T[sh.B - 1]

    def prefix_network(self, T, later_block):
        """In-place inclusive prefixes of the block's tuples; returns the block summary (at level lS).  The decay
        products that only an incoming state would use are not formed for the first block."""
        if self.network == "bk":
            return self.brent_kung(T, need_p_down=later_block)
        return (self.kogge_stone if self.network == "ks" else self.sklansky)(T, later_block)

    def run(self, ctX, ctA, ctB, ctC):
        """ctX, ctA [K_blk, K_s, segs, 2, l0, N]; ctB, ctC [K_blk, 2, l0, N] -> out [K_blk, K_s, segs, 2, l_out, N]."""
        sh, c, o = self.sh, self.c, self.o
        lv = c.lv
        linj, lout = lv["linj"], lv["lout"]
        out = np.zeros((sh.K_blk, sh.K_s, sh.segs, 2, lout, o.N), dtype=np.uint64)
        carry = [None] * sh.K_s                       # g_j per chunk: the state before block j
        for j in range(sh.K_blk):
            brB = self.broadcast_b_grouped(ctB[j]) if self.group else self.broadcast_bc(ctB[j])
            brC = self.broadcast_bc(ctC[j], linj - 1)
            v = [[None] * sh.K_s for _ in range(sh.B)]
            for kap in range(sh.K_s):
                T = (self.leaves_grouped if self.group else self.leaves)(ctX[j, kap], ctA[j, kap], brB)
                summary = self.prefix_network(T, j > 0)
                g = carry[kap]
                for t in range(sh.B):
                    sP = self.adjust(T[t][1], linj - 1, "s")
                    if g is None:
                        h = sP
                    else:
                        h = self.add(self.mul_rescale(self.adjust(T[t][0], linj, "p"), self.adjust(g, linj, "s")), sP)
                    v[t][kap] = self.mul_rescale(h, brC[t])              # level linj-2
                if j + 1 < sh.K_blk:                                   # serialized carry g_{j+1} = S_j(g_j)
                    if g is None:
                        carry[kap] = summary[1]
                    else:
                        lg = g.shape[1]
                        carry[kap] = self.add(self.mul_rescale(self.adjust(summary[0], lg, "p"), g),
                                              self.adjust(summary[1], lg - 1, "s"))
            self.contract_block(j, v, out)
        return out

    # -- invariant families: plaintext decay, input factor and output factor -----------------------
    def compose_plain(self, sL, sR, lvl, pt):
        """s <- abar^span (.) s_L + s_R with operands brought to lvl (one ct-pt product); result at lvl-1."""
        self.count["compose"] += 1
        return self.add(self.ptmul_rescale(self.adjust(sL, lvl, "s"), pt), self.adjust(sR, lvl - 1, "s"))

    def leaves_plain(self, ctX):
        """s_t = br(x_t) (.) Bbar at l1 for the tokens of one (block, chunk); br(x_t) as in `leaves` / `leaves_grouped`."""
        sh, c, G = self.sh, self.c, self.group
        lg = lambda v: int(math.log2(v))
        T = []
        for seg in range(sh.segs):
            if G:
                gx = self.extract_all(ctX[seg], G, sh.Bt // G)
                for u in range(sh.Bt // G):
                    xg = self.fill_right(self.ptmul_rescale(gx[u], c.mask_xg), G, lg(sh.d_s // G))
                    T += [self.ptmul_rescale(b, c.pt_b) for b in self.class_broadcasts(xg, c.mask_x2, 1)]
            else:
                ex = self.extract_all(ctX[seg], 1, sh.Bt)
                for tt in range(sh.Bt):
                    xr = self.fill_right(self.ptmul_rescale(ex[tt], c.mask_x), 1, lg(sh.d_s))
                    T.append(self.ptmul_rescale(xr, c.pt_b))
        return T

    def brent_kung_plain(self, T):
        """In-place inclusive prefixes of the state inputs T[0..B-1]; returns the block summary (level lS)."""
        sh, c = self.sh, self.c
        B, logB, l1, lS = sh.B, sh.logB, c.lv["l1"], c.lv["lS"]
        for s in range(1, logB + 1):
            for k in range(1 << s, B + 1, 1 << s):
                T[k - 1] = self.compose_plain(T[k - (1 << (s - 1)) - 1], T[k - 1], l1 - (s - 1), c.pt_up[s])
        summary = T[B - 1]
        d = 0
        for s in range(logB - 1, 0, -1):
            d += 1
            for k in range(1 << s, B, 1 << s):
                r = k + (1 << (s - 1))
                if r < B:
                    T[r - 1] = self.compose_plain(T[k - 1], T[r - 1], lS - (d - 1), c.pt_down[d])
        return summary

    def run_plain(self, ctX):
        """Invariant-family scan-contract (module header): ctX [K_blk, K_s, segs, 2, l0, N] -> out as in `run`."""
        sh, c, o = self.sh, self.c, self.o
        assert c.plain
        linj, lout = c.lv["linj"], c.lv["lout"]
        out = np.zeros((sh.K_blk, sh.K_s, sh.segs, 2, lout, o.N), dtype=np.uint64)
        carry = [None] * sh.K_s
        for j in range(sh.K_blk):
            v = [[None] * sh.K_s for _ in range(sh.B)]
            for kap in range(sh.K_s):
                T = self.leaves_plain(ctX[j, kap])
                summary = self.brent_kung_plain(T)
                g = carry[kap]
                for t in range(sh.B):
                    h = self.adjust(T[t], linj - 1, "s")
                    if g is not None:       # state = abar^(t+1) (.) g_j + s_t
                        h = self.add(self.ptmul_rescale(self.adjust(g, linj, "s"), c.pt_inj[t]), h)
                    v[t][kap] = self.ptmul_rescale(h, c.pt_c)              # level linj-2
                if j + 1 < sh.K_blk:                                       # serialized carry g_{j+1} = abar^B g_j + s_S
                    if g is None:
                        carry[kap] = summary
                    else:
                        lg = g.shape[1]
                        carry[kap] = self.add(self.ptmul_rescale(g, c.pt_carry[j]), self.adjust(summary, lg - 1, "s"))
            self.contract_block(j, v, out)
        return out

    def contract_block(self, j, v, out):
        """State-axis reduction of every token, chunks paired in the real / imaginary lanes."""
        sh, c, o = self.sh, self.c, self.o
        steps = int(math.log2(sh.d_s))
        for t in range(sh.B):
            for kap in range(0, sh.K_s, 2):
                paired = kap + 1 < sh.K_s
                chi = self.add(v[t][kap], o.mul_monomial_half(v[t][kap + 1])) if paired else v[t][kap]
                chi = self.chain(chi, 1, steps)
                if paired:
                    bar = self.conj(chi)
                    parts = [self.add(chi, bar), self.neg_times_i(self.sub(chi, bar))]   # 2 Re, 2 Im
                else:
                    parts = [self.add(chi, chi)]                                           # same factor 2
                for off, part in enumerate(parts):
                    y = self.ptmul_rescale(part, c.mask_out)
                    seg, tt = divmod(t, sh.Bt)                      # placement inside the token's segment
                    y = self.rot(self.rot(y, -(tt % sh.dgt)), -sh.dgt * (tt // sh.dgt))
                    out[j, kap + off, seg] = self.add(out[j, kap + off, seg], y)

    def neg_times_i(self, ct):
        """-i * ct  =  X^(N/2) applied three times (exact monomial products)."""
        o = self.o
        return o.mul_monomial_half(o.mul_monomial_half(o.mul_monomial_half(ct)))


def closed_form_counts(shape: ScanShape, network: str = "bk"):
    """Counts the dataflow must reproduce (pins against the paper's ledgers)."""
    sh = shape
    per_block = dict(bk=2 * (sh.B - 1) - sh.logB,                 # compositions of each network over B positions
                     ks=sh.B * sh.logB - (sh.B - 1),
                     sk=(sh.B // 2) * sh.logB)[network]
    return dict(
        compose=sh.K_blk * sh.K_s * per_block,
        reduce_rot=sh.K_blk * sh.B * (-(-sh.K_s // 2)) * int(math.log2(sh.d_s)),
        reduce_conj=sh.K_blk * sh.B * (sh.K_s // 2),
    )
