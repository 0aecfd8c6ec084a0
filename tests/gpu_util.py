"""Helpers shared by the GPU parity tests: context pairs (CUDA library + oracle) and array moves."""
from __future__ import annotations

import numpy as np


def to_dev(a: np.ndarray):
    import torch

    return torch.from_numpy(np.ascontiguousarray(a, dtype=np.uint64).view(np.int64)).cuda()


def to_host(t) -> np.ndarray:
    return t.cpu().numpy().view(np.uint64)


_PAIRS = {}


def ctx_pair(name: str):
    """(CUDA context, oracle) for a named parameter set, cached per process."""
    import fesc_synth as S
    import paper_2608_17442_b200 as fesc
    from oracle.ckks import Oracle

    if name not in _PAIRS:
        p = S.params(name)
        args = (p["log_n"], p["primes"], p["n_q"], p["n_p"], p["dnum"], p["seed"])
        _PAIRS[name] = (fesc.Context(*args), Oracle(*args), p)
    return _PAIRS[name]


def add_key(pair, rot: int, key_id: int):
    ctx, orc, _ = pair
    if key_id not in orc.keys:
        orc.add_galois_key(rot, key_id)
        ctx.add_galois_key(rot, key_id)


def random_ct(orc, seed: int, stream: int, level: int, batch: int) -> np.ndarray:
    """[batch, 2, level, N] uniform residues (a ciphertext-shaped input)."""
    import fesc_synth as S

    out = np.empty((batch, 2, level, orc.N), dtype=np.uint64)
    for b in range(batch):
        for p in range(2):
            out[b, p] = S.uniform_residues_np(seed, stream * 4096 + b * 2 + p, orc.q[:level], orc.N)
    return out


def run_scan_parity(name, hoist=0, network="bk", group=0, **kw):
    """fesc_scan_contract against ScanEvaluator.run on the named parameter set and shape: asserts that every output
    residue is equal and returns the largest deviation of the decrypted result from the float64 recurrence."""
    import torch
    import fesc_synth as S
    import paper_2608_17442_b200 as fesc
    from oracle.ckks import CONJ
    from oracle.scan import (ScanConsts, ScanEvaluator, ScanShape, add_scan_keys, encrypt_inputs, float_recurrence,
                             key_id_for, unpack_output)

    ctx, orc, p = ctx_pair(name)
    sh = ScanShape(orc.n, **kw)
    l0 = p["n_q"]
    x, a, B, C = S.scan_inputs(p["seed"] + sh.L, sh.L, sh.H, sh.P, 1, sh.d_s)
    c = ScanConsts(orc, sh, l0, p["log_scale"], network, group)
    add_scan_keys(orc, sh, hoist=bool(hoist), group=group)
    for r in sh.rotation_amounts(bool(hoist), group) + [CONJ]:
        ctx.add_galois_key(r, key_id_for(sh, r))
    ctX, ctA, ctB, ctC = encrypt_inputs(orc, sh, c, x, a, B, C)
    want = ScanEvaluator(orc, sh, c, hoist=bool(hoist)).run(ctX, ctA, ctB, ctC)
    adj_s = [c.adj_s.get((s, d), 0) for s in range(l0 + 1) for d in range(l0 + 1)]
    adj_p = [c.adj_p.get((s, d), 0) for s in range(l0 + 1) for d in range(l0 + 1)]
    out = torch.empty((sh.K_blk, sh.K_s, sh.segs, 2, c.lv["lout"], orc.N), dtype=torch.int64, device="cuda")
    desc = fesc.ScanDesc(sh.L, sh.H, sh.P, sh.d_s, sh.B, kw.get("stride", 0), l0, 100000, hoist,
                         {"bk": fesc.NET_BRENT_KUNG, "ks": fesc.NET_KOGGE_STONE, "sk": fesc.NET_SKLANSKY}[network], group)
    gm = [to_dev(m) for m in (c.mask_xg, c.mask_ag, c.mask_x2, c.mask_a2, c.mask_bg, c.mask_b2)] if group else None
    ctx.scan_contract(to_dev(ctX), to_dev(ctA), to_dev(ctB), to_dev(ctC), desc, to_dev(c.mask_x), to_dev(c.mask_b),
                      to_dev(c.mask_a), to_dev(c.mask_out), adj_s, adj_p, out, gm)
    ctx.sync()
    got = to_host(out)
    assert np.array_equal(got, want)
    m = unpack_output(orc, sh, c, got)
    return np.abs(m - float_recurrence(x, a, B, C)).max()


def run_scan_parity_invariant(name, hoist=0, group=0, seed_stream=300, **kw):
    """The invariant-family mode (plaintext decay, input and output factors): fesc_scan_contract with desc.plain = 1
    against ScanEvaluator.run_plain; asserts equal residues, returns the largest deviation of the decrypted result
    from the float64 recurrence and the library's key-switch count."""
    import torch
    import fesc_synth as S
    import paper_2608_17442_b200 as fesc
    from oracle.ckks import CONJ
    from oracle.scan import (ScanConsts, ScanEvaluator, ScanShape, add_scan_keys, encrypt_x, float_recurrence_invariant,
                             key_id_for, unpack_output)

    ctx, orc, p = ctx_pair(name)
    sh = ScanShape(orc.n, **kw)
    l0 = p["n_q"]
    x, _, _, _ = S.scan_inputs(p["seed"] + sh.L, sh.L, sh.H, sh.P, 1, sh.d_s)
    g = S.rng(p["seed"], seed_stream)
    fac = (g.uniform(0.9, 1.0, sh.d_s), g.standard_normal(sh.d_s) * 0.5, g.standard_normal(sh.d_s) * 0.5)
    c = ScanConsts(orc, sh, l0, p["log_scale"], "bk", group, plain=fac)
    add_scan_keys(orc, sh, hoist=bool(hoist), group=group)
    for r in sh.rotation_amounts(bool(hoist), group) + [CONJ]:
        ctx.add_galois_key(r, key_id_for(sh, r))
    ctX = encrypt_x(orc, sh, c, x)
    ev = ScanEvaluator(orc, sh, c, hoist=bool(hoist))
    want = ev.run_plain(ctX)
    assert ev.count["ctmul"] == 0

    def table(rows, count):       # {index: [level, N]} -> [count][l0][N], zero beyond each row's level
        out = np.zeros((max(count, 1), l0, orc.N), dtype=np.uint64)
        for i, v in rows.items():
            out[i, :v.shape[0]] = v
        return to_dev(out)

    lv = c.lv
    tables = (to_dev(c.pt_b), to_dev(c.pt_c), table({s - 1: v for s, v in c.pt_up.items()}, sh.logB),
              table({d - 1: v for d, v in c.pt_down.items()}, sh.logB - 1), table(dict(c.pt_carry), sh.K_blk),
              to_dev(np.stack(c.pt_inj)) if c.pt_inj else None)
    adj_s = [c.adj_s.get((s, d), 0) for s in range(l0 + 1) for d in range(l0 + 1)]
    out = torch.empty((sh.K_blk, sh.K_s, sh.segs, 2, lv["lout"], orc.N), dtype=torch.int64, device="cuda")
    desc = fesc.ScanDesc(sh.L, sh.H, sh.P, sh.d_s, sh.B, kw.get("stride", 0), l0, 100000, hoist, fesc.NET_BRENT_KUNG, group, 1)
    gm = [to_dev(c.mask_xg), None, to_dev(c.mask_x2), None, None, None] if group else None
    ks0 = ctx.counters()[1]
    ctx.scan_contract(to_dev(ctX), None, None, None, desc, to_dev(c.mask_x), None, None, to_dev(c.mask_out), adj_s, None,
                      out, gm, tables)
    ctx.sync()
    ks = ctx.counters()[1] - ks0
    got = to_host(out)
    assert np.array_equal(got, want)
    assert ks == ev.count["rot"] + ev.count["conj"]          # rotations and conjugations only: no relinearisation
    m = unpack_output(orc, sh, c, got)
    return np.abs(m - float_recurrence_invariant(x, *fac)).max()
