"""Seeded synthetic inputs shared by the oracle-side tests and the CUDA-side harness.

This module holds no CKKS arithmetic.  It only produces inputs: the RNS prime
lists handed to ``fesc_ctx_create`` (found by a deterministic downward walk
from a seed-dependent start), float64 messages / weights / scan factors with
the distributions of the five workloads, and bulk "uniform residue" arrays from
a counter hash that gives identical values on CPU and on the GPU (so a sampled
output of a full-size run can be recomputed elsewhere from the same counters).
"""
from __future__ import annotations

import numpy as np

SEED_BASE = 260817442 * 10


def config_seed(k: int) -> int:
    """Seed of workload k (1..5)."""
    return SEED_BASE + k


# ---------------------------------------------------------------------------
# primes
# ---------------------------------------------------------------------------
_MR_BASES = (2, 3, 5, 7, 11, 13, 17, 19, 23, 29, 31, 37)


def is_prime(n: int) -> bool:
    """Deterministic Miller-Rabin for n < 3.3e24 (12 prime bases)."""
    if n < 2:
        return False
    for p in _MR_BASES:
        if n % p == 0:
            return n == p
    d, r = n - 1, 0
    while d % 2 == 0:
        d //= 2
        r += 1
    for a in _MR_BASES:
        x = pow(a, d, n)
        if x in (1, n - 1):
            continue
        for _ in range(r - 1):
            x = x * x % n
            if x == n - 1:
                break
        else:
            return False
    return True


def ntt_primes(bits: int, log_n: int, count: int, seed: int, exclude=()) -> list[int]:
    """`count` primes q = k*2N+1 below 2^bits, walking k downward from
    2^bits/(2N) - (seed mod 4096); returned in descending order."""
    two_n = 2 << log_n
    k = (1 << bits) // two_n - (seed % 4096)
    out: list[int] = []
    while len(out) < count:
        q = k * two_n + 1
        if q < (1 << bits) and q.bit_length() == bits and q not in exclude and is_prime(q):
            out.append(q)
        k -= 1
        if k <= 0:
            raise ValueError("ran out of candidates")
    return out


def params(name: str) -> dict:
    """CKKS parameter sets of the workloads.

    tiny : N=2^12, 3 data + 1 special 36-bit primes, dnum=3, scale 2^30 (workload 1)
    full : N=2^16, 24 x 50-bit data + 4 x 60-bit special primes, scale 2^40,
           dnum=6 (alpha=4 limbs per digit = number of special primes; the
           graded reading of workloads 3-5)
    full_literal : same primes, dnum=4 (alpha=6 > 4 special primes; the literal
           text of workloads 3-5, whose key-switch noise exceeds the scale)
    toy  : N=2^6 for exhaustive big-integer checks
    """
    if name == "tiny":
        seed = config_seed(1)
        four = ntt_primes(36, 12, 4, seed)
        return dict(name=name, log_n=12, primes=four[1:] + four[:1], n_q=3, n_p=1, dnum=3,
                    seed=seed, log_scale=30)
    if name in ("full", "full_literal"):
        seed = config_seed(3)
        data = ntt_primes(50, 16, 24, seed)
        special = ntt_primes(60, 16, 4, seed)
        return dict(name=name, log_n=16, primes=data + special, n_q=24, n_p=4,
                    dnum=6 if name == "full" else 4, seed=seed, log_scale=40)
    if name == "toy":
        seed = config_seed(0)
        data = ntt_primes(30, 6, 6, seed)
        special = ntt_primes(36, 6, 2, seed)
        return dict(name=name, log_n=6, primes=data + special, n_q=6, n_p=2, dnum=3,
                    seed=seed, log_scale=20)
    if name == "small":
        # N=2^10 with the limb structure of the full set, for fast multi-level tests
        seed = config_seed(0)
        data = ntt_primes(50, 10, 24, seed)
        special = ntt_primes(60, 10, 4, seed)
        return dict(name=name, log_n=10, primes=data + special, n_q=24, n_p=4, dnum=6,
                    seed=seed, log_scale=40)
    if name == "small_d9":
        # the small ring with 9 key-switch digits of two limbs (more digits than one FP64 fold-back interval)
        seed = config_seed(0)
        data = ntt_primes(50, 10, 18, seed)
        special = ntt_primes(60, 10, 2, seed)
        return dict(name=name, log_n=10, primes=data + special, n_q=18, n_p=2, dnum=9, seed=seed, log_scale=40)
    if name in ("scan_toy", "scan_small"):
        # rings for the scan-contract tests: the paper's toy shape (16 slots) and a 128-slot analogue of
        # the Mamba-2-base geometry; 50-bit chain, two 60-bit special primes, two limbs per digit
        log_n, n_q = (5, 10) if name == "scan_toy" else (8, 16)
        seed = config_seed(5)
        data = ntt_primes(50, log_n, n_q, seed)
        special = ntt_primes(60, log_n, 2, seed)
        return dict(name=name, log_n=log_n, primes=data + special, n_q=n_q, n_p=2, dnum=n_q // 2,
                    seed=seed, log_scale=40)
    if name == "wide":
        # 55-bit data primes: exercises the integer (non-FP64) kernels of the library
        seed = config_seed(0)
        data = ntt_primes(55, 10, 6, seed)
        special = ntt_primes(60, 10, 2, seed)
        return dict(name=name, log_n=10, primes=data + special, n_q=6, n_p=2, dnum=3, seed=seed, log_scale=40)
    if name == "full52":
        # N=2^16 with 52-bit data primes: the integer wide-lazy transform path
        seed = config_seed(0)
        data = ntt_primes(52, 16, 2, seed)
        special = ntt_primes(60, 16, 1, seed)
        return dict(name=name, log_n=16, primes=data + special, n_q=2, n_p=1, dnum=2, seed=seed, log_scale=40)
    raise KeyError(name)


# ---------------------------------------------------------------------------
# float64 messages
# ---------------------------------------------------------------------------
def rng(seed: int, stream: int = 0) -> np.random.Generator:
    return np.random.Generator(np.random.PCG64([seed, stream]))


def uniform_slots(seed: int, stream: int, count: int, n_slots: int) -> np.ndarray:
    """`count` real slot vectors uniform in [-1, 1]."""
    return rng(seed, stream).uniform(-1.0, 1.0, size=(count, n_slots))


def linear_inputs(seed: int, tokens: int, d_in: int, d_out: int):
    """Activations ~N(0,1) [tokens, d_in] and weights ~N(0, 0.02^2) [d_in, d_out]."""
    g = rng(seed, 100)
    x = g.standard_normal((tokens, d_in))
    w = g.standard_normal((d_in, d_out)) * 0.02
    return x, w


def scan_inputs(seed: int, L: int, H: int, P: int, G: int, d_s: int):
    """Factor packets of the scan contract: x~N(0,1) [L,H,P], decay a~U(0.9,1)
    [L,H], B and C ~N(0, 1/d_s) [L,G,d_s]."""
    g = rng(seed, 200)
    x = g.standard_normal((L, H, P))
    a = g.uniform(0.9, 1.0, size=(L, H))
    B = g.standard_normal((L, G, d_s)) / np.sqrt(d_s)
    C = g.standard_normal((L, G, d_s)) / np.sqrt(d_s)
    return x, a, B, C


def uniform_residues_np(seed: int, stream: int, primes, n: int) -> np.ndarray:
    """[len(primes), n] uint64 residues, uniform below each prime (numpy PCG64)."""
    g = rng(seed, 1000 + stream)
    out = np.empty((len(primes), n), dtype=np.uint64)
    for i, q in enumerate(primes):
        out[i] = g.integers(0, q, size=n, dtype=np.uint64)
    return out


# ---------------------------------------------------------------------------
# bulk counter-hash residues (identical on any torch device)
# ---------------------------------------------------------------------------
_M1 = -0x40A7B892E31B1A47  # 0xBF58476D1CE4E5B9 as int64
_M2 = -0x6B2FB644ECCEEE15  # 0x94D049BB133111EB as int64


def hashed_residues(seed: int, stream: int, primes, n: int, device="cpu", first: int = 0):
    """[len(primes), n] residues r[i][t] = mix(seed, stream, i, first+t) mod primes[i]
    as an int64 torch tensor on `device` (bit pattern = the uint64 residue).

    The mixer is a 64-bit multiply/xor-shift finaliser evaluated in wrapping
    int64 arithmetic; its top bit is cleared before the remainder so that the
    signed remainder equals the unsigned one.  Only used to fill large buffers
    (ciphertext-shaped and plaintext-shaped inputs of the full-size workloads).
    """
    import torch

    t = torch.arange(first, first + n, dtype=torch.int64, device=device)
    rows = []
    for i, q in enumerate(primes):
        key = (seed * 0x9E3779B1 + stream * 0x85EBCA77 + i * 0xC2B2AE3D + 0x27D4EB2F) & 0x7FFFFFFFFFFFFFFF
        z = t * 0x9E3779B97F4A7C1 + key
        z = (z ^ ((z >> 30) & 0x3FFFFFFFF)) * _M1
        z = (z ^ ((z >> 27) & 0x1FFFFFFFFF)) * _M2
        z = z ^ ((z >> 31) & 0x1FFFFFFFF)
        z = z & 0x7FFFFFFFFFFFFFFF
        rows.append(torch.remainder(z, q))
    return torch.stack(rows)
