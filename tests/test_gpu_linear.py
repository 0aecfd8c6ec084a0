"""GPU parity for the BSGS projection: residues equal the oracle's bit for bit, and the decrypted
result equals X @ W in float64."""
import numpy as np
import pytest

import fesc_synth as S
from oracle.ckks import linear_diagonal, pack_linear_input
from tests.gpu_util import add_key, ctx_pair, to_dev, to_host

pytestmark = pytest.mark.gpu


def _setup(pair, T, C, n1, n2, tokens, d_in, d_out, level, scale, wscale=1.0, key_base=1000):
    ctx, orc, p = pair
    n = orc.n
    assert C * T == n and n1 * n2 == C
    X, W = S.linear_inputs(p["seed"] + 4, tokens, d_in, d_out)
    W = W * wscale
    gin, nout, tbs = -(-d_in // C), -(-d_out // C), -(-tokens // T)
    for q in range(1, n1):
        add_key(pair, q * T, key_base + q)
    for g in range(1, n2):
        add_key(pair, g * n1 * T, key_base + 500 + g)
    cts = np.empty((tbs, gin, 2, level, orc.N), dtype=np.uint64)
    for tb in range(tbs):
        for g in range(gin):
            v = pack_linear_input(X[tb * T:(tb + 1) * T, g * C:(g + 1) * C], T, C, n)
            cts[tb, g] = orc.encrypt(orc.encode(v, scale, level), 7000 + tb * gin + g)
    diags = np.empty((nout, n2, gin, n1, level, orc.N), dtype=np.uint64)
    for b in range(nout):
        for pp in range(n2):
            for g in range(gin):
                for q in range(n1):
                    diags[b, pp, g, q] = orc.encode(linear_diagonal(W, b, g, pp, q, T, C, n1), float(orc.q[level - 1]), level)
    return X, W, cts, diags, (gin, nout, tbs)


def _run_gpu(ctx, cts, diags, n1, n2, dims, level, key_base=1000, hoist=0, defer=0, packed=0):
    """packed=1: the diagonals go through fesc_linear_pack_diags first (two ranges when there are more than 8 (b,p)
    pairs, so that the placement of a later range is exercised) and fesc_linear runs on the byte-plane image."""
    import torch
    import paper_2608_17442_b200 as fesc

    gin, nout, tbs = dims
    desc = fesc.BsgsDesc(n1, n2, gin, nout, tbs, level, key_base, key_base + 500, hoist, defer, packed)
    out = torch.empty((tbs, nout, 2, level - 1, cts.shape[-1]), dtype=torch.int64, device="cuda")
    d = to_dev(diags)
    if packed:
        image = torch.full((ctx.linear_packed_bytes(desc),), 0xA5, dtype=torch.uint8, device="cuda")
        pairs = nout * n2
        flat = d.reshape(pairs, gin, n1, level, cts.shape[-1])
        cut = 8 if pairs > 8 else pairs
        ctx.linear_pack_diags(flat[:cut], desc, 0, cut, image)
        if cut < pairs:
            ctx.linear_pack_diags(flat[cut:].contiguous(), desc, cut, pairs - cut, image)
        d = image
    ctx.linear(to_dev(cts), d, desc, out)
    return to_host(out)


@pytest.mark.parametrize("shape", [(32, 16, 4, 4, 70, 40, 50, 5), (64, 8, 8, 1, 64, 8, 8, 3), (16, 32, 2, 16, 20, 33, 30, 24)])
def test_linear_small_ring(shape):
    T, C, n1, n2, tokens, d_in, d_out, level = shape
    pair = ctx_pair("small")
    ctx, orc, _ = pair
    scale = 2.0**40
    X, W, cts, diags, dims = _setup(pair, T, C, n1, n2, tokens, d_in, d_out, level, scale, wscale=10.0,
                                    key_base=1000 + 37 * T)
    got = _run_gpu(ctx, cts, diags, n1, n2, dims, level, key_base=1000 + 37 * T)
    kb = 1000 + 37 * T
    want = orc.linear(cts, diags, dict(n1=n1, n2=n2), {q: kb + q for q in range(1, n1)},
                      {g: kb + 500 + g for g in range(1, n2)})
    assert np.array_equal(got, want)
    assert np.array_equal(_run_gpu(ctx, cts, diags, n1, n2, dims, level, key_base=kb, packed=1), want)
    # hoisted baby rotations: other residues (own oracle mode), same values
    got_h = _run_gpu(ctx, cts, diags, n1, n2, dims, level, key_base=kb, hoist=1)
    want_h = orc.linear(cts, diags, dict(n1=n1, n2=n2), {q: kb + q for q in range(1, n1)},
                        {g: kb + 500 + g for g in range(1, n2)}, hoist=True)
    assert np.array_equal(got_h, want_h)
    assert n1 == 1 or not np.array_equal(got_h, got)
    # one division by P for the whole giant-step sum (own oracle mode), alone and with hoisting
    for hoist in (0, 1):
        got_d = _run_gpu(ctx, cts, diags, n1, n2, dims, level, key_base=kb, hoist=hoist, defer=1)
        want_d = orc.linear(cts, diags, dict(n1=n1, n2=n2), {q: kb + q for q in range(1, n1)},
                            {g: kb + 500 + g for g in range(1, n2)}, hoist=bool(hoist), defer=True)
        assert np.array_equal(got_d, want_d)
        assert np.array_equal(_run_gpu(ctx, cts, diags, n1, n2, dims, level, key_base=kb, hoist=hoist, defer=1, packed=1), want_d)
    gin, nout, tbs = dims
    for tb in range(tbs):
        for b in range(nout):
            yh = orc.decrypt(got_h[tb, b], scale, 2).real.reshape(C, T).T
            assert np.abs(yh[:min(T, tokens - tb * T), :min(C, d_out - b * C)]
                          - (X @ W)[tb * T:(tb + 1) * T, b * C:(b + 1) * C]).max() < 2.0**-18
    Y = np.zeros((tbs * T, nout * C))
    for tb in range(tbs):
        for b in range(nout):
            Y[tb * T:(tb + 1) * T, b * C:(b + 1) * C] = orc.decrypt(got[tb, b], scale, 2).real.reshape(C, T).T
    assert np.abs(Y[:tokens, :d_out] - X @ W).max() < 2.0**-18


def test_linear_accumulate_extreme_residues_256_terms():
    """Worst case for the mixed integer/FP64 sums: 256 terms per accumulator, every residue q-1 (largest products,
    largest rounding of the FP64 magnitude) in one half of the data and uniform residues in the other."""
    pair = ctx_pair("small")
    ctx, orc, p = pair
    T, C, n1, n2, level = 32, 16, 16, 1, 4
    gin, nout, tbs = 16, 2, 3
    kb = 5000
    for q in range(1, n1):
        add_key(pair, q * T, kb + q)
    qs = np.array(orc.q[:level], dtype=np.uint64)
    primes = [int(x) for x in qs]
    cts = np.stack([S.uniform_residues_np(p["seed"] + 91, i, primes, orc.N)
                    for i in range(tbs * gin * 2)]).reshape(tbs, gin, 2, level, orc.N)
    diags = np.stack([S.uniform_residues_np(p["seed"] + 92, i, primes, orc.N)
                      for i in range(nout * n2 * gin * n1)]).reshape(nout, n2, gin, n1, level, orc.N)
    cts[:, :, :, :, : orc.N // 2] = (qs - 1)[None, None, None, :, None]
    diags[:, :, :, :, :, : orc.N // 2] = (qs - 1)[None, None, None, None, :, None]
    for hoist in (0, 1):
        got = _run_gpu(ctx, cts, diags, n1, n2, (gin, nout, tbs), level, key_base=kb, hoist=hoist)
        want = orc.linear(cts, diags, dict(n1=n1, n2=n2), {q: kb + q for q in range(1, n1)}, {}, hoist=bool(hoist))
        assert np.array_equal(got, want)
        # the byte-plane products on the tensor cores: 256 terms of 255 x 255 per plane pair, 8 k-steps
        got = _run_gpu(ctx, cts, diags, n1, n2, (gin, nout, tbs), level, key_base=kb, hoist=hoist, packed=1)
        assert np.array_equal(got, want)


def test_linear_on_complex_paired_token_blocks():
    """Two token blocks in the real and imaginary channels of one ciphertext, real diagonals: one projection and one
    conjugation per output give both results (residues bit-exact against the oracle, values against X @ W)."""
    import torch
    from oracle.ckks import CONJ

    pair = ctx_pair("small")
    ctx, orc, p = pair
    T, C, n1, n2, level, scale = 32, 16, 4, 4, 5, 2.0**40
    tokens, d_in, d_out, kb = 4 * T, 40, 50, 8000
    n = orc.n
    X, W = S.linear_inputs(p["seed"] + 9, tokens, d_in, d_out)
    W = W * 10.0
    gin, nout, pairs = -(-d_in // C), -(-d_out // C), tokens // (2 * T)
    for q in range(1, n1):
        add_key(pair, q * T, kb + q)
    for g in range(1, n2):
        add_key(pair, g * n1 * T, kb + 500 + g)
    add_key(pair, CONJ, kb + 999)
    cts = np.empty((pairs, gin, 2, level, orc.N), dtype=np.uint64)
    for u in range(pairs):
        for g in range(gin):
            v0 = pack_linear_input(X[(2 * u) * T:(2 * u + 1) * T, g * C:(g + 1) * C], T, C, n)
            v1 = pack_linear_input(X[(2 * u + 1) * T:(2 * u + 2) * T, g * C:(g + 1) * C], T, C, n)
            cts[u, g] = orc.encrypt(orc.encode(v0 + 1j * v1, scale, level), 7700 + u * gin + g)
    diags = np.empty((nout, n2, gin, n1, level, orc.N), dtype=np.uint64)
    for b in range(nout):
        for pp in range(n2):
            for g in range(gin):
                for q in range(n1):
                    diags[b, pp, g, q] = orc.encode(linear_diagonal(W, b, g, pp, q, T, C, n1), float(orc.q[level - 1]), level)
    got = _run_gpu(ctx, cts, diags, n1, n2, (gin, nout, pairs), level, key_base=kb, hoist=1, defer=1)
    want = orc.linear(cts, diags, dict(n1=n1, n2=n2), {q: kb + q for q in range(1, n1)},
                      {g: kb + 500 + g for g in range(1, n2)}, hoist=True, defer=True)
    assert np.array_equal(got, want)
    batch = pairs * nout
    z = to_dev(got.reshape(batch, 2, level - 1, orc.N))
    re2, im2 = torch.empty_like(z), torch.empty_like(z)
    ctx.split_complex(z, re2, im2, batch, level - 1, kb + 999)
    re2, im2 = to_host(re2), to_host(im2)
    Y = X @ W
    for u in range(pairs):
        for b in range(nout):
            wr, wi = orc.split_complex(want[u, b], kb + 999)
            assert np.array_equal(re2[u * nout + b], wr) and np.array_equal(im2[u * nout + b], wi)
            cols = slice(b * C, min((b + 1) * C, d_out))
            for part, tb in ((wr, 2 * u), (wi, 2 * u + 1)):
                y = orc.decrypt(part, 2 * scale, 2).real.reshape(C, T).T
                assert np.abs(y[:, :cols.stop - cols.start] - Y[tb * T:(tb + 1) * T, cols]).max() < 2.0**-18


def test_linear_on_complex_paired_input_blocks():
    """The paper's pairing (App. "Projection Kernel Breakdown"): input blocks 2u and 2u+1 in the real and imaginary
    channels, complex diagonals D^(2u) - i D^(2u+1); the real part of the result is X @ W.  Three input blocks become
    two ciphertexts per token block; residues bit-exact against the oracle, values against X @ W."""
    import torch
    from oracle.ckks import CONJ

    pair = ctx_pair("small")
    ctx, orc, p = pair
    T, C, n1, n2, level, scale = 32, 16, 4, 4, 5, 2.0**40
    tokens, d_in, d_out, kb = 2 * T, 40, 50, 8200
    n = orc.n
    X, W = S.linear_inputs(p["seed"] + 10, tokens, d_in, d_out)
    W = W * 10.0
    gin, nout, tbs = -(-d_in // C), -(-d_out // C), tokens // T
    gpair = -(-gin // 2)
    for q in range(1, n1):
        add_key(pair, q * T, kb + q)
    for g in range(1, n2):
        add_key(pair, g * n1 * T, kb + 500 + g)
    add_key(pair, CONJ, kb + 999)
    blk = lambda tb, g: pack_linear_input(X[tb * T:(tb + 1) * T, g * C:(g + 1) * C], T, C, n) if g < gin else np.zeros(n)
    cts = np.empty((tbs, gpair, 2, level, orc.N), dtype=np.uint64)
    for tb in range(tbs):
        for u in range(gpair):
            cts[tb, u] = orc.encrypt(orc.encode(blk(tb, 2 * u) + 1j * blk(tb, 2 * u + 1), scale, level), 7800 + tb * gpair + u)
    dg = lambda b, g, pp, q: linear_diagonal(W, b, g, pp, q, T, C, n1) if g < gin else np.zeros(n)
    diags = np.empty((nout, n2, gpair, n1, level, orc.N), dtype=np.uint64)
    for b in range(nout):
        for pp in range(n2):
            for u in range(gpair):
                for q in range(n1):
                    diags[b, pp, u, q] = orc.encode(dg(b, 2 * u, pp, q) - 1j * dg(b, 2 * u + 1, pp, q),
                                                    float(orc.q[level - 1]), level)
    got = _run_gpu(ctx, cts, diags, n1, n2, (gpair, nout, tbs), level, key_base=kb, hoist=1, defer=1)
    want = orc.linear(cts, diags, dict(n1=n1, n2=n2), {q: kb + q for q in range(1, n1)},
                      {g: kb + 500 + g for g in range(1, n2)}, hoist=True, defer=True)
    assert np.array_equal(got, want)
    batch = tbs * nout
    z = to_dev(got.reshape(batch, 2, level - 1, orc.N))
    re2 = torch.empty_like(z)
    ctx.split_complex(z, re2, None, batch, level - 1, kb + 999)
    re2 = to_host(re2)
    Y = X @ W
    for tb in range(tbs):
        for b in range(nout):
            wr, _ = orc.split_complex(want[tb, b], kb + 999)
            assert np.array_equal(re2[tb * nout + b], wr)
            cols = slice(b * C, min((b + 1) * C, d_out))
            y = orc.decrypt(wr, 2 * scale, 2).real.reshape(C, T).T
            assert np.abs(y[:, :cols.stop - cols.start] - Y[tb * T:(tb + 1) * T, cols]).max() < 2.0**-18


def test_linear_integer_kernels_with_55_bit_primes():
    """Primes above 50 bits (the integer recombination of the tensor-core accumulate; the 128-bit integer kernel where
    that does not apply) against the oracle."""
    pair = ctx_pair("wide")
    ctx, orc, _ = pair
    T, C, n1, n2, level = 32, 16, 4, 4, 6
    X, W, cts, diags, dims = _setup(pair, T, C, n1, n2, 50, 30, 20, level, 2.0**40, wscale=10.0, key_base=3000)
    for hoist, defer in ((0, 0), (1, 0), (1, 1)):
        got = _run_gpu(ctx, cts, diags, n1, n2, dims, level, key_base=3000, hoist=hoist, defer=defer)
        want = orc.linear(cts, diags, dict(n1=n1, n2=n2), {q: 3000 + q for q in range(1, n1)},
                          {g: 3500 + g for g in range(1, n2)}, hoist=bool(hoist), defer=bool(defer))
        assert np.array_equal(got, want)
        # packed diagonals with 55-bit primes: the 128-bit integer recombination
        got = _run_gpu(ctx, cts, diags, n1, n2, dims, level, key_base=3000, hoist=hoist, defer=defer, packed=1)
        assert np.array_equal(got, want)


def test_linear_full_ring_one_block():
    """N = 2^16, 24 limbs, scale 2^40: one token block x one output block of the in_proj shape
    (768 inputs = 3 input blocks, C=256, T=128, n1=32, n2=8); bit-exact and within 2^-18 of X @ W."""
    pair = ctx_pair("full")
    ctx, orc, _ = pair
    T, C, n1, n2, level = 128, 256, 32, 8, 24
    scale = 2.0**40
    X, W, cts, diags, dims = _setup(pair, T, C, n1, n2, 128, 768, 256, level, scale, key_base=2000)
    got = _run_gpu(ctx, cts, diags, n1, n2, dims, level, key_base=2000)
    want = orc.linear(cts, diags, dict(n1=n1, n2=n2), {q: 2000 + q for q in range(1, n1)},
                      {g: 2500 + g for g in range(1, n2)})
    assert np.array_equal(got, want)
    Y = orc.decrypt(got[0, 0], scale, 2).real.reshape(C, T).T
    err = np.abs(Y - X @ W).max()
    print("max |decrypt - X@W| = 2^%.2f" % np.log2(err))
    assert err < 2.0**-18
    # the benchmark's default modes (hoisted baby steps, one division by P per output): own residues, same values
    got_m = _run_gpu(ctx, cts, diags, n1, n2, dims, level, key_base=2000, hoist=1, defer=1)
    want_m = orc.linear(cts, diags, dict(n1=n1, n2=n2), {q: 2000 + q for q in range(1, n1)},
                        {g: 2500 + g for g in range(1, n2)}, hoist=True, defer=True)
    assert np.array_equal(got_m, want_m)
    assert np.array_equal(_run_gpu(ctx, cts, diags, n1, n2, dims, level, key_base=2000, hoist=1, defer=1, packed=1), want_m)
    err_m = np.abs(orc.decrypt(got_m[0, 0], scale, 2).real.reshape(C, T).T - X @ W).max()
    print("hoisted + deferred: max |decrypt - X@W| = 2^%.2f" % np.log2(err_m))
    assert err_m < 2.0**-18


def test_linear_token_major_packing_with_periodic_diagonals():
    """Token-major packing (slot r*C + c): the projection runs through the same fesc_linear with 2 n1 - 1 baby and
    2 n2 - 1 giant rotation amounts, and its diagonals are periodic, so the packed image holds one operand per aligned
    run of N/(2C) evaluation indices (desc.diag_run_log2 = 5 here: 32 times smaller).  Residues equal the oracle's
    (which multiplies the full-size diagonals), values equal X @ W."""
    import torch
    import paper_2608_17442_b200 as fesc
    from oracle.ckks import (linear_diagonal_token_major, pack_linear_input_token_major, periodic_eval_runs,
                             token_major_amounts)

    pair = ctx_pair("small")
    ctx, orc, p = pair
    n = orc.n
    T, C, n1, n2, level, scale, kb = 32, 16, 4, 4, 5, 2.0**40, 9000
    tokens, d_in, d_out = 150, 40, 20            # 5 token blocks (two groups), 3 input blocks, 2 output blocks
    X, W = S.linear_inputs(p["seed"] + 14, tokens, d_in, d_out)
    W = W * 10
    gin, nout, tbs = -(-d_in // C), -(-d_out // C), -(-tokens // T)
    baby, giant = token_major_amounts(C, n1, n2)
    nb, ng, run = len(baby), len(giant), orc.N // (2 * C)
    for i, a in enumerate(baby[1:], 1):
        add_key(pair, a, kb + i)
    for i, a in enumerate(giant[1:], 1):
        add_key(pair, a, kb + 500 + i)
    cts = np.empty((tbs, gin, 2, level, orc.N), dtype=np.uint64)
    for tb in range(tbs):
        for g in range(gin):
            v = pack_linear_input_token_major(X[tb * T:(tb + 1) * T, g * C:(g + 1) * C], T, C, n)
            cts[tb, g] = orc.encrypt(orc.encode(v, scale, level), 7900 + tb * gin + g)
    diags = np.empty((nout, ng, gin, nb, level, orc.N), dtype=np.uint64)
    small = np.empty((nout, ng, gin, nb, level, orc.N // run), dtype=np.uint64)
    for b in range(nout):
        for gi in range(ng):
            for g in range(gin):
                for bi in range(nb):
                    diags[b, gi, g, bi] = orc.encode(linear_diagonal_token_major(W, b, g, gi, bi, T, C, n1),
                                                     float(orc.q[level - 1]), level)
                    small[b, gi, g, bi] = periodic_eval_runs(diags[b, gi, g, bi], run)
    shift = run.bit_length() - 1
    desc = fesc.BsgsDesc(nb, ng, gin, nout, tbs, level, kb, kb + 500, 1, 1, 1, shift)
    image = torch.full((ctx.linear_packed_bytes(desc),), 0x5A, dtype=torch.uint8, device="cuda")
    full_desc = fesc.BsgsDesc(nb, ng, gin, nout, tbs, level, kb, kb + 500, 1, 1, 1, 0)
    assert ctx.linear_packed_bytes(desc) * run == ctx.linear_packed_bytes(full_desc)
    pairs = nout * ng
    flat = to_dev(small.reshape(pairs, gin, nb, level, orc.N // run))
    ctx.linear_pack_diags(flat[:8], desc, 0, 8, image)
    ctx.linear_pack_diags(flat[8:].contiguous(), desc, 8, pairs - 8, image)
    out = torch.empty((tbs, nout, 2, level - 1, orc.N), dtype=torch.int64, device="cuda")
    ctx.linear(to_dev(cts), image, desc, out)
    got = to_host(out)
    want = orc.linear(cts, diags, dict(n1=nb, n2=ng), {i: kb + i for i in range(1, nb)},
                      {i: kb + 500 + i for i in range(1, ng)}, hoist=True, defer=True)
    assert np.array_equal(got, want)
    Y = np.zeros((tbs * T, nout * C))
    for tb in range(tbs):
        for b in range(nout):
            Y[tb * T:(tb + 1) * T, b * C:(b + 1) * C] = orc.decrypt(got[tb, b], scale, 2).real.reshape(T, C)
    assert np.abs(Y[:tokens, :d_out] - X @ W).max() < 2.0**-18
    # periodic diagonals are a property of the packed image
    with pytest.raises(fesc.FescError) as e:
        ctx.linear(to_dev(cts), to_dev(diags), fesc.BsgsDesc(nb, ng, gin, nout, tbs, level, kb, kb + 500, 1, 1, 0, shift), out)
    assert e.value.code == fesc.EINVAL


@pytest.mark.parametrize("packed", [0, 1])
def test_linear_falls_back_to_smaller_groups_when_scratch_cannot_be_had(packed):
    """The projection sizes its token-block group from a scratch budget; when the arena cannot be reserved (failure
    injected on the host, no driver call) it halves the group and tries again.  Same residues, smaller group; a failure
    on every attempt comes back as FESC_ENOMEM and the context computes correctly afterwards."""
    import paper_2608_17442_b200 as fesc

    T, C, n1, n2, tokens, d_in, d_out, level = 32, 16, 4, 4, 8 * 32, 16, 32, 4       # 8 token blocks
    pair = ctx_pair("small")
    ctx, orc, _ = pair
    kb = 1000 + 37 * T
    X, W, cts, diags, dims = _setup(pair, T, C, n1, n2, tokens, d_in, d_out, level, 2.0**40, wscale=10.0, key_base=kb)
    want = orc.linear(cts, diags, dict(n1=n1, n2=n2), {q: kb + q for q in range(1, n1)}, {g: kb + 500 + g for g in range(1, n2)})
    ctx.trim()
    assert np.array_equal(_run_gpu(ctx, cts, diags, n1, n2, dims, level, key_base=kb, packed=packed), want)
    full_group = ctx.counters()[5]
    assert full_group == 8
    ctx.trim()
    ctx.test_fail_allocs(1)                    # the first reservation fails: one halving
    assert np.array_equal(_run_gpu(ctx, cts, diags, n1, n2, dims, level, key_base=kb, packed=packed), want)
    assert ctx.counters()[5] == 4
    ctx.trim()
    ctx.test_fail_allocs(16)                   # every attempt fails, down to a group of one
    with pytest.raises(fesc.FescError) as e:
        _run_gpu(ctx, cts, diags, n1, n2, dims, level, key_base=kb, packed=packed)
    assert e.value.code == fesc.ENOMEM
    ctx.test_fail_allocs(0)
    assert np.array_equal(_run_gpu(ctx, cts, diags, n1, n2, dims, level, key_base=kb, packed=packed), want)


@pytest.mark.parametrize("gin", [7, 9, 11])
def test_linear_packed_input_fragments_of_4_to_6_ksteps(gin):
    """Sums of 112, 144 and 176 terms: the packed accumulate keeps the input fragments of 4, 5 and 6 k-steps in shared
    memory beside a shorter ring (the token-major in_proj has 189 terms); residues against the oracle, both operand forms."""
    T, C, n1, n2, tokens, d_out, level = 16, 32, 16, 2, 40, 40, 3
    pair = ctx_pair("small")
    ctx, orc, _ = pair
    kb = 20000                      # key ids of its own (the cached context keeps every key of every test)
    X, W, cts, diags, dims = _setup(pair, T, C, n1, n2, tokens, gin * C - 3, d_out, level, 2.0**40, wscale=10.0, key_base=kb)
    assert dims[0] == gin
    want = orc.linear(cts, diags, dict(n1=n1, n2=n2), {q: kb + q for q in range(1, n1)}, {g: kb + 500 + g for g in range(1, n2)})
    assert np.array_equal(_run_gpu(ctx, cts, diags, n1, n2, dims, level, key_base=kb, packed=1), want)
    assert np.array_equal(_run_gpu(ctx, cts, diags, n1, n2, dims, level, key_base=kb, packed=0), want)
