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
