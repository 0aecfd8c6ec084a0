"""Thin Python binding of the sm_100a RNS-CKKS library (argument marshalling only).

Every function below forwards to the C-ABI entry point of the same name in
libfesc_b200.so (declared in include/fesc.h); all arithmetic runs in the CUDA kernels.
Tensors are torch CUDA tensors of dtype int64 (bit pattern = the uint64 residue); the
binding passes their data pointers and the current torch stream.  There is no CPU
fallback: importing succeeds without the library, but the first call raises.
"""
from __future__ import annotations

import ctypes
import os

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.environ.get("FESC_LIB", os.path.join(_HERE, "libfesc_b200.so"))

OK, EINVAL, ENOMEM, ECUDA, ELEVEL, ENOKEY, ETIMEOUT, EBOUNDS = 0, -1, -2, -3, -4, -5, -6, -7
CONJ = -(1 << 31)
NET_BRENT_KUNG, NET_KOGGE_STONE, NET_SKLANSKY = 0, 1, 2     # fesc_scan_desc.network
RELIN_KEY_ID = 0

_lib = None
_debug_bounds = False      # the loaded library is the bounds-checking debug build


class FescError(RuntimeError):
    def __init__(self, code: int, msg: str):
        super().__init__(f"fesc error {code}: {msg}")
        self.code = code


class BsgsDesc(ctypes.Structure):
    _fields_ = [(n, ctypes.c_uint32) for n in
                ("n1", "n2", "in_blocks", "out_blocks", "token_blocks", "n_limbs", "baby_key_base", "giant_key_base",
                 "hoist", "defer", "packed", "diag_run_log2")]


class Info(ctypes.Structure):
    _fields_ = ([(n, ctypes.c_uint32) for n in ("log_n", "n_q", "n_p", "dnum", "alpha", "digits", "flags", "reserved")]
                + [("log2_P", ctypes.c_double), ("log2_Qmax", ctypes.c_double)])


INFO_KEYSWITCH_NOISE = 1


class ConvDesc(ctypes.Structure):
    _fields_ = [(n, ctypes.c_uint32) for n in ("d_conv", "T", "blocks", "token_blocks", "n_limbs", "key_base")]


class NormDesc(ctypes.Structure):
    _fields_ = [(n, ctypes.c_uint32) for n in ("T", "blocks", "token_blocks", "n_limbs", "key_base")]


class ScanDesc(ctypes.Structure):
    _fields_ = [(n, ctypes.c_uint32) for n in ("L", "H", "P", "d_s", "B_blk", "stride", "n_limbs", "key_base",
                                                       "hoist", "network", "group", "plain")]


class ScanConsts(ctypes.Structure):
    _fields_ = [(n, ctypes.c_void_p) for n in ("d_mask_x", "d_mask_b", "d_mask_a", "d_mask_out", "adj_s", "adj_p",
                                               "d_mask_xg", "d_mask_ag", "d_mask_x2", "d_mask_a2", "d_mask_bg", "d_mask_b2",
                                               "d_pt_b", "d_pt_c", "d_pt_up", "d_pt_down", "d_pt_carry", "d_pt_inj")]


def lib():
    """Load libfesc_b200.so (built by paper_2608_17442_b200.build); raise if it is missing."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise RuntimeError(f"{LIB_PATH} is missing: run `python -m paper_2608_17442_b200.build` "
                               "(there is no CPU fallback)")
        L = ctypes.CDLL(LIB_PATH)
        c = ctypes
        vp, u32, u64, i32, sz = c.c_void_p, c.c_uint32, c.c_uint64, c.c_int32, c.c_size_t
        sig = {
            "fesc_ctx_create": [c.POINTER(vp), u32, c.POINTER(u64), u32, u32, u32, u64],
            "fesc_ctx_destroy": [vp],
            "fesc_sync": [vp, vp],
            "fesc_ctx_trim": [vp],
            "fesc_selftest_wait_limit": [vp, vp],
            "fesc_ctx_add_galois_key": [vp, i32, u32],
            "fesc_ctx_export_key": [vp, u32, vp, vp],
            "fesc_ctx_export_secret": [vp, vp, vp],
            "fesc_ctx_counters": [vp, c.POINTER(u64)],
            "fesc_profile_enable": [vp, c.c_int, u32],
            "fesc_profile_read": [vp, c.POINTER(c.c_float), c.POINTER(u64)],
            "fesc_ntt": [vp, vp, u32, u32, u32, vp],
            "fesc_intt": [vp, vp, u32, u32, u32, vp],
            "fesc_ct_pt_mac": [vp, vp, vp, sz, vp, u32, u32, vp],
            "fesc_rotate": [vp, vp, vp, u32, u32, u32, vp],
            "fesc_rotate_hoisted": [vp, vp, vp, u32, u32, c.POINTER(u32), u32, vp],
            "fesc_rotate_sum_hoisted": [vp, vp, vp, u32, u32, c.POINTER(u32), u32, vp],
            "fesc_conv": [vp, vp, vp, vp, c.POINTER(ConvDesc), vp, vp],
            "fesc_norm_square": [vp, vp, vp, c.c_uint32, c.c_uint32, vp],
            "fesc_norm_scale": [vp, vp, vp, vp, c.POINTER(NormDesc), vp, vp],
            "fesc_split_complex": [vp, vp, vp, vp, u32, u32, u32, vp],
            "fesc_rescale": [vp, vp, vp, u32, u32, vp],
            "fesc_rescale_static": [vp, vp, vp, u32, u32, vp],
            "fesc_ct_ct_mul": [vp, vp, vp, vp, u32, u32, vp],
            "fesc_linear": [vp, vp, vp, c.POINTER(BsgsDesc), vp, vp],
            "fesc_linear_pack_diags": [vp, vp, c.POINTER(BsgsDesc), u32, u32, vp, vp],
            "fesc_params_info": [u32, c.POINTER(u64), u32, u32, u32, c.POINTER(Info)],
            "fesc_ctx_info": [vp, c.POINTER(Info)],
            "fesc_ctx_test_fail_allocs": [vp, u32],
            "fesc_scan_contract": [vp, vp, vp, vp, vp, c.POINTER(ScanDesc), c.POINTER(ScanConsts), vp, vp],
            "fesc_debug_bounds_register": [vp, sz],
            "fesc_debug_bounds_clear": [],
            "fesc_debug_bounds_report": [c.POINTER(u32), c.POINTER(u32), c.POINTER(u64), c.POINTER(u64)],
        }
        for name, args in sig.items():
            f = getattr(L, name)
            f.argtypes = args
            f.restype = c.c_int
        L.fesc_last_error.argtypes = [vp]
        L.fesc_last_error.restype = c.c_char_p
        L.fesc_linear_packed_bytes.argtypes = [vp, c.POINTER(BsgsDesc)]
        L.fesc_linear_packed_bytes.restype = sz
        L.fesc_ctx_num_digits.argtypes = [vp]
        L.fesc_ctx_num_digits.restype = u32
        _lib = L
    return _lib


def debug_bounds() -> bool:
    """True when the loaded library is the bounds-checking debug build (FESC_LIB pointing at libfesc_b200_dbg.so):
    the binding then registers the extent of every tensor it passes, and Context.sync raises FescError(EBOUNDS) after
    a kernel skipped a region outside every known extent.  The first call needs a GPU."""
    global _debug_bounds
    if not getattr(debug_bounds, "asked", False):
        _debug_bounds = lib().fesc_debug_bounds_clear() == OK
        debug_bounds.asked = True
    return _debug_bounds


def debug_bounds_clear():
    if lib().fesc_debug_bounds_clear() != OK:
        raise FescError(EINVAL, "not a debug build")


def debug_bounds_report():
    """(skipped regions since the last report, first site = file id << 16 | line, first address, its size in bytes)."""
    c = ctypes
    h, s, a, b = c.c_uint32(), c.c_uint32(), c.c_uint64(), c.c_uint64()
    if lib().fesc_debug_bounds_report(c.byref(h), c.byref(s), c.byref(a), c.byref(b)) != OK:
        raise FescError(EINVAL, "not a debug build")
    return h.value, s.value, a.value, b.value


def params_info(log_n: int, primes, n_q: int, n_p: int, dnum: int) -> Info:
    """fesc_params_info: derived parameters and flags of a parameter set; runs on the host alone (no GPU needed)."""
    arr = (ctypes.c_uint64 * len(primes))(*[int(p) for p in primes])
    out = Info()
    rc = lib().fesc_params_info(log_n, arr, n_q, n_p, dnum, ctypes.byref(out))
    if rc != OK:
        raise FescError(rc, "bad parameter set")
    return out


def _stream():
    import torch

    return ctypes.c_void_p(torch.cuda.current_stream().cuda_stream)


def _raw(t):
    """Data pointer of a contiguous CUDA tensor (None passes through); a debug build learns the tensor's extent."""
    if t is None:
        return None
    assert t.is_cuda and t.is_contiguous()
    if debug_bounds():
        lib().fesc_debug_bounds_register(t.data_ptr(), t.numel() * t.element_size())
    return t.data_ptr()


def _ptr(t):
    assert t.element_size() == 8
    return ctypes.c_void_p(_raw(t))


class Context:
    """Owner of a fesc_ctx handle; methods mirror the C entry points."""

    def __init__(self, log_n: int, primes, n_q: int, n_p: int, dnum: int, seed: int):
        self.log_n, self.N = log_n, 1 << log_n
        self.n_q, self.n_p, self.dnum, self.seed = n_q, n_p, dnum, seed
        self.primes = [int(p) for p in primes]
        arr = (ctypes.c_uint64 * len(self.primes))(*self.primes)
        h = ctypes.c_void_p()
        rc = lib().fesc_ctx_create(ctypes.byref(h), log_n, arr, n_q, n_p, dnum, seed)
        if rc != OK:
            raise FescError(rc, "fesc_ctx_create failed")
        self.h = h

    def _chk(self, rc: int):
        if rc != OK:
            raise FescError(rc, lib().fesc_last_error(self.h).decode())

    def close(self):
        if getattr(self, "h", None) and _lib is not None:
            _lib.fesc_ctx_destroy(self.h)
            self.h = None

    def __del__(self):
        try:
            self.close()
        except Exception:      # interpreter shutdown: module globals may already be gone
            pass

    def trim(self):
        """Release the scratch arena (it is reserved again on demand)."""
        self._chk(lib().fesc_ctx_trim(self.h))

    def selftest_wait_limit(self):
        self._chk(lib().fesc_selftest_wait_limit(self.h, _stream()))

    def sync(self):
        self._chk(lib().fesc_sync(self.h, _stream()))

    @property
    def num_digits(self) -> int:
        return lib().fesc_ctx_num_digits(self.h)

    def counters(self):
        out = (ctypes.c_uint64 * 8)()
        self._chk(lib().fesc_ctx_counters(self.h, out))
        return list(out)

    PROFILE_FAMILIES = ("ntt", "modup", "inner", "moddown", "autom", "bsgs", "rescale", "pointwise")

    def profile_enable(self, families, max_records: int = 65536):
        """Time the named kernel families (iterable of PROFILE_FAMILIES names; empty = off)."""
        mask = 0
        for f in families:
            mask |= 1 << self.PROFILE_FAMILIES.index(f)
        self._chk(lib().fesc_profile_enable(self.h, mask, max_records))

    def profile_read(self):
        """{family: (milliseconds, records)} since the last read."""
        ms = (ctypes.c_float * 8)()
        rec = (ctypes.c_uint64 * 8)()
        self._chk(lib().fesc_profile_read(self.h, ms, rec))
        return {n: (float(ms[i]), int(rec[i])) for i, n in enumerate(self.PROFILE_FAMILIES)}

    def add_galois_key(self, rot: int, key_id: int):
        self._chk(lib().fesc_ctx_add_galois_key(self.h, rot, key_id))

    def export_key(self, key_id: int):
        import torch

        out = torch.empty((self.num_digits, 2, self.n_q + self.n_p, self.N), dtype=torch.int64, device="cuda")
        self._chk(lib().fesc_ctx_export_key(self.h, key_id, _ptr(out), _stream()))
        return out

    def export_secret(self):
        import torch

        out = torch.empty((self.n_q + self.n_p, self.N), dtype=torch.int64, device="cuda")
        self._chk(lib().fesc_ctx_export_secret(self.h, _ptr(out), _stream()))
        return out

    def ntt(self, data, batch: int, first_limb: int, n_limbs: int):
        self._chk(lib().fesc_ntt(self.h, _ptr(data), batch, first_limb, n_limbs, _stream()))

    def intt(self, data, batch: int, first_limb: int, n_limbs: int):
        self._chk(lib().fesc_intt(self.h, _ptr(data), batch, first_limb, n_limbs, _stream()))

    def ct_pt_mac(self, ct, pt, acc, batch: int, n_limbs: int, pt_stride=None):
        if pt_stride is None:
            pt_stride = n_limbs * self.N
        self._chk(lib().fesc_ct_pt_mac(self.h, _ptr(ct), _ptr(pt), pt_stride, _ptr(acc), batch, n_limbs, _stream()))

    def rotate(self, ct_in, ct_out, batch: int, n_limbs: int, key_id: int):
        self._chk(lib().fesc_rotate(self.h, _ptr(ct_in), _ptr(ct_out), batch, n_limbs, key_id, _stream()))

    def split_complex(self, ct_in, re2, im2, batch: int, n_limbs: int, conj_key_id: int):
        self._chk(lib().fesc_split_complex(self.h, _ptr(ct_in), _ptr(re2), _ptr(im2) if im2 is not None else None, batch,
                                           n_limbs, conj_key_id, _stream()))

    def norm_square(self, y, out, batch, n_limbs):
        self._chk(lib().fesc_norm_square(self.h, _ptr(y), _ptr(out), batch, n_limbs, _stream()))

    def norm_scale(self, y, s, gamma, desc: "NormDesc", out):
        self._chk(lib().fesc_norm_scale(self.h, _ptr(y), _ptr(s), _ptr(gamma), ctypes.byref(desc), _ptr(out), _stream()))

    def conv(self, ct_in, masks, bias, desc: "ConvDesc", ct_out):
        self._chk(lib().fesc_conv(self.h, _ptr(ct_in), _ptr(masks), _ptr(bias), ctypes.byref(desc), _ptr(ct_out), _stream()))

    def rotate_sum_hoisted(self, ct_in, ct_out, batch: int, n_limbs: int, key_ids):
        ids = (ctypes.c_uint32 * len(key_ids))(*key_ids)
        self._chk(lib().fesc_rotate_sum_hoisted(self.h, _ptr(ct_in), _ptr(ct_out), batch, n_limbs, ids, len(key_ids), _stream()))

    def rotate_hoisted(self, ct_in, ct_out, batch: int, n_limbs: int, key_ids):
        ids = (ctypes.c_uint32 * len(key_ids))(*key_ids)
        self._chk(lib().fesc_rotate_hoisted(self.h, _ptr(ct_in), _ptr(ct_out), batch, n_limbs, ids, len(key_ids), _stream()))

    def rescale(self, ct_in, ct_out, batch: int, n_limbs: int):
        self._chk(lib().fesc_rescale(self.h, _ptr(ct_in), _ptr(ct_out), batch, n_limbs, _stream()))

    def rescale_static(self, ct_in, ct_out, batch: int, n_limbs: int):
        """fesc_rescale without any device allocation: scratch lives in a fixed 4 MiB array of the library
        (batch * 2 * N <= 524 288 words).  For callers that cannot reach cudaMalloc (fixed memory budgets
        owned by another allocator, latency-critical loops, hosts that forbid allocator calls).  The first
        call on a device looks up the array's address; make it before any stream capture.  Calls share the
        array: do not overlap them on the GPU."""
        self._chk(lib().fesc_rescale_static(self.h, _ptr(ct_in), _ptr(ct_out), batch, n_limbs, _stream()))

    def ct_ct_mul(self, a, b, out, batch: int, n_limbs: int):
        self._chk(lib().fesc_ct_ct_mul(self.h, _ptr(a), _ptr(b), _ptr(out), batch, n_limbs, _stream()))

    def linear(self, ct_in, diags, desc: BsgsDesc, ct_out):
        """diags: the residue tensor, or (desc.packed = 1) the uint8 image filled by linear_pack_diags."""
        assert diags.is_cuda and diags.is_contiguous()
        self._chk(lib().fesc_linear(self.h, _ptr(ct_in), ctypes.c_void_p(_raw(diags)), ctypes.byref(desc),
                                    _ptr(ct_out), _stream()))

    def linear_packed_bytes(self, desc: BsgsDesc) -> int:
        return int(lib().fesc_linear_packed_bytes(self.h, ctypes.byref(desc)))

    def linear_pack_diags(self, diags, desc: BsgsDesc, first: int, count: int, packed):
        """Packs the (b,p) pairs [first, first+count) from `diags` ([count][in_blocks][n1][n_limbs][N] residues) into
        their place inside the uint8 CUDA tensor `packed` (linear_packed_bytes(desc) bytes)."""
        assert packed.is_cuda and packed.is_contiguous() and packed.element_size() == 1
        self._chk(lib().fesc_linear_pack_diags(self.h, _ptr(diags), ctypes.byref(desc), first, count,
                                               ctypes.c_void_p(_raw(packed)), _stream()))

    def info(self) -> Info:
        out = Info()
        self._chk(lib().fesc_ctx_info(self.h, ctypes.byref(out)))
        return out

    def test_fail_allocs(self, count: int):
        self._chk(lib().fesc_ctx_test_fail_allocs(self.h, count))

    def scan_contract(self, x, a, B, C, desc: ScanDesc, mask_x, mask_b, mask_a, mask_out, adj_s, adj_p, m_out,
                      group_masks=None, plain_tables=None):
        """adj_s / adj_p: sequences of (n_limbs+1)^2 Python ints (host tables); masks: CUDA tensors (None where the
        mode does not use one); group_masks = (mask_xg, mask_ag, mask_x2, mask_a2, mask_bg, mask_b2) for desc.group > 0;
        plain_tables = (pt_b, pt_c, pt_up, pt_down, pt_carry, pt_inj) for desc.plain = 1 (a, B, C may then be None)."""
        n = (desc.n_limbs + 1) ** 2
        hs = (ctypes.c_uint64 * n)(*[int(v) for v in adj_s])
        hp = (ctypes.c_uint64 * n)(*[int(v) for v in (adj_p if adj_p is not None else [0] * n)])
        ptr = _raw
        cs = ScanConsts(ptr(mask_x), ptr(mask_b), ptr(mask_a), ptr(mask_out),
                        ctypes.cast(hs, ctypes.c_void_p).value, ctypes.cast(hp, ctypes.c_void_p).value,
                        *([ptr(t) for t in group_masks] if group_masks else [None] * 6),
                        *([ptr(t) for t in plain_tables] if plain_tables else [None] * 6))
        opt = lambda t: _ptr(t) if t is not None else None
        self._chk(lib().fesc_scan_contract(self.h, _ptr(x), opt(a), opt(B), opt(C), ctypes.byref(desc),
                                           ctypes.byref(cs), _ptr(m_out), _stream()))
