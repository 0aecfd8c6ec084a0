"""The benchmark's launch configuration at full size: in_proj 768 -> 3352 at L = 2048 tokens (48 input
ciphertexts, 10 752 diagonals = 126 GiB as residues or 110 GiB as the packed byte-plane image the benchmark uses,
224 outputs, N = 2^16, 24 limbs).  Inputs are the benchmark's own
(counter-hash residues); one sampled output ciphertext is recomputed by the oracle from the same counters,
regenerated on the CPU, and must match bit for bit.  Properties that hold at any size are checked on all
outputs: canonical residues, and equality of outputs whose inputs are equal."""
import gc

import numpy as np
import pytest

import fesc_synth as S
from tests.gpu_util import ctx_pair, to_host

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("hoist,defer,packed", [(0, 0, 0), (1, 1, 1)])
def test_in_proj_full_size_sampled_against_oracle(hoist, defer, packed):
    """(1, 1, 1) is the benchmark's default launch configuration (hoisted baby steps, one division by P per output,
    packed diagonals: the tensor-core accumulate at its full size); (0, 0, 0) the plain definitions on residues."""
    import torch
    import bench
    import paper_2608_17442_b200 as fesc

    pair = ctx_pair("full")
    ctx, orc, p = pair
    ctx.trim()                     # an earlier test may have left a large scratch arena on this cached context
    gin, nout, tbs = bench.workload_dims()
    assert (gin, nout, tbs) == (3, 14, 16)
    n1, n2, T, level = bench.N1, bench.N2, bench.T_SEG, bench.LEVEL
    for q in range(1, n1):
        if bench.BABY_BASE + q not in orc.keys:
            orc.add_galois_key(q * T, bench.BABY_BASE + q)
            ctx.add_galois_key(q * T, bench.BABY_BASE + q)
    for g in range(1, n2):
        if bench.GIANT_BASE + g not in orc.keys:
            orc.add_galois_key(g * n1 * T, bench.GIANT_BASE + g)
            ctx.add_galois_key(g * n1 * T, bench.GIANT_BASE + g)
    seed = S.config_seed(4)
    desc = fesc.BsgsDesc(n1, n2, gin, nout, tbs, level, bench.BABY_BASE, bench.GIANT_BASE, hoist, defer, packed)
    ct, diags = bench.make_inputs(p["primes"], orc.N, gin, nout, tbs, seed, torch.device("cuda"), ctx, desc)
    out = torch.empty((tbs, nout, 2, level - 1, orc.N), dtype=torch.int64, device="cuda")
    torch.cuda.empty_cache()
    ctx.linear(ct, diags, desc, out)
    ctx.sync()
    # properties on every output: residues are canonical
    qs = torch.tensor(p["primes"][:level - 1], dtype=torch.int64, device="cuda").view(1, 1, 1, -1, 1)
    assert bool(((out >= 0) & (out < qs)).all())
    # sampled output (token block 5, last and partially filled output block 13), inputs regenerated on the CPU
    tb, b = 5, 13
    got = to_host(out[tb, b])
    del out, qs
    q24 = p["primes"][:level]
    ct_s = np.empty((1, gin, 2, level, orc.N), dtype=np.uint64)
    for g in range(gin):
        r = S.hashed_residues(seed, tb * gin + g, q24, 2 * orc.N, device="cpu")
        ct_s[0, g] = r.view(level, 2, orc.N).permute(1, 0, 2).numpy().view(np.uint64)
        assert np.array_equal(ct_s[0, g], to_host(ct[tb, g]))          # same generator on both devices
    dg_s = np.empty((1, n2, gin, n1, level, orc.N), dtype=np.uint64)
    for pp in range(n2):
        r = S.hashed_residues(seed, 100000 + b * n2 + pp, q24, gin * n1 * orc.N, device="cpu")
        dg_s[0, pp] = r.view(level, gin, n1, orc.N).permute(1, 2, 0, 3).numpy().view(np.uint64)
    if packed:      # the image is not comparable word by word: check the generator itself on one diagonal chunk
        r = S.hashed_residues(seed, 100000 + b * n2 + 3, q24, gin * n1 * orc.N, device="cuda")
        assert np.array_equal(dg_s[0, 3, 1, 7], to_host(r.view(level, gin, n1, orc.N)[:, 1, 7].contiguous()))
        del r
    else:
        assert np.array_equal(dg_s[0, 3, 1, 7], to_host(diags[b, 3, 1, 7]))
    del ct, diags
    gc.collect()
    torch.cuda.empty_cache()
    want = orc.linear(ct_s, dg_s, dict(n1=n1, n2=n2), {q: bench.BABY_BASE + q for q in range(1, n1)},
                      {g: bench.GIANT_BASE + g for g in range(1, n2)}, hoist=bool(hoist), defer=bool(defer))
    assert np.array_equal(got, want[0, 0])
