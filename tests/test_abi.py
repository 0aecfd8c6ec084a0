"""The C-ABI library builds, loads and exports every symbol that include/fesc.h declares
(no GPU needed: nothing is launched)."""
import ctypes
import os
import re

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def test_library_exports_every_declared_symbol():
    from paper_2608_17442_b200 import build

    path = build.build()
    lib = ctypes.CDLL(path)
    header = open(os.path.join(ROOT, "include", "fesc.h")).read()
    header = re.sub(r"/\*.*?\*/", "", header, flags=re.S)
    names = set(re.findall(r"\b(fesc_[a-z0-9_]+)\s*\(", header))
    assert {"fesc_ctx_create", "fesc_ntt", "fesc_intt", "fesc_ct_pt_mac", "fesc_rotate", "fesc_linear"} <= names
    for n in names:
        assert hasattr(lib, n), n


def test_binding_names_match_header():
    import paper_2608_17442_b200 as fesc

    for n in ("ntt", "intt", "ct_pt_mac", "rotate", "rescale", "ct_ct_mul", "linear", "add_galois_key"):
        assert hasattr(fesc.Context, n)


def test_product_does_not_import_oracle():
    pkg = os.path.join(ROOT, "paper_2608_17442_b200")
    for dirpath, _, files in os.walk(pkg):
        for f in files:
            if f.endswith((".py", ".cu", ".cuh", ".h")):
                text = open(os.path.join(dirpath, f)).read()
                assert "oracle" not in text.replace("no CPU fallback", ""), f


def test_params_info_flags_a_special_modulus_below_the_digit_modulus():
    """fesc_params_info runs on the host alone.  The graded reading of workloads 3-5 (6 digits of 4 limbs, P = four
    60-bit primes) has P above every digit modulus; the literal dnum = 4 set (digits of 6 x 50 bits against the same
    240-bit P) does not, and is flagged."""
    import fesc_synth as S
    import paper_2608_17442_b200 as fesc

    p = S.params("full")
    info = fesc.params_info(p["log_n"], p["primes"], p["n_q"], p["n_p"], p["dnum"])
    assert (info.alpha, info.digits, info.flags) == (4, 6, 0)
    assert 239.9 < info.log2_P < 240.0 and 199.9 < info.log2_Qmax < 200.0
    p = S.params("full_literal")
    info = fesc.params_info(p["log_n"], p["primes"], p["n_q"], p["n_p"], p["dnum"])
    assert (info.alpha, info.digits) == (6, 4)
    assert info.flags & fesc.INFO_KEYSWITCH_NOISE and info.log2_Qmax > info.log2_P
    # the exact comparison decides, not the rounded logarithms: P one prime short of the digit modulus
    p = S.params("tiny")
    info = fesc.params_info(p["log_n"], p["primes"], p["n_q"], p["n_p"], 1)       # one digit of 3 limbs, one special prime
    assert info.flags & fesc.INFO_KEYSWITCH_NOISE
    info = fesc.params_info(p["log_n"], p["primes"], p["n_q"], p["n_p"], 3)       # digits of one limb; special = largest prime
    assert info.flags == 0
