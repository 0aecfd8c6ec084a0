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
