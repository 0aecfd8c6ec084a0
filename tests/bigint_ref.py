"""Big-integer helpers for pinning the oracle: plain Python ints, no shared code with
either implementation."""
from __future__ import annotations

import math


def brev(x: int, bits: int) -> int:
    r = 0
    for _ in range(bits):
        r = (r << 1) | (x & 1)
        x >>= 1
    return r


def crt(residues, moduli) -> int:
    """The integer in [0, prod moduli) with the given residues (Garner / incremental)."""
    x, m = 0, 1
    for r, q in zip(residues, moduli):
        t = ((int(r) - x) * pow(m, -1, q)) % q
        x += m * t
        m *= q
    return x


def centre(x: int, m: int) -> int:
    x %= m
    return x - m if x > m // 2 else x


def negacyclic_schoolbook(a, b, q):
    n = len(a)
    c = [0] * n
    for i in range(n):
        for j in range(n):
            k = i + j
            if k < n:
                c[k] = (c[k] + int(a[i]) * int(b[j])) % q
            else:
                c[k - n] = (c[k - n] - int(a[i]) * int(b[j])) % q
    return c


def is_primitive_root_2n(psi: int, q: int, n: int) -> bool:
    return pow(psi, n, q) == q - 1


def poly_from_rns(rows, moduli):
    """[k][N] residues -> list of N big ints in [0, Q)."""
    n = len(rows[0])
    return [crt([rows[i][c] for i in range(len(moduli))], moduli) for c in range(n)]


def negacyclic_mul_int(a, b, modulus):
    n = len(a)
    c = [0] * n
    for i in range(n):
        if a[i] == 0:
            continue
        for j in range(n):
            k = i + j
            if k < n:
                c[k] += a[i] * b[j]
            else:
                c[k - n] -= a[i] * b[j]
    return [x % modulus for x in c]


def prod(xs):
    return math.prod(int(x) for x in xs)
