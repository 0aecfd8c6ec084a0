#!/usr/bin/env python
"""Benchmark of the encrypted Mamba-2-base in_proj projection (768 -> 3352 at L = 2048 tokens)
on B200, through the C-ABI library.

One "step" = one fesc_linear call on the full workload: 48 input ciphertexts (16 token blocks x
3 input blocks, N = 2^16, 24 limbs), 10 752 pre-encoded plaintext diagonals (126 GiB, resident),
1 488 baby + 1 568 giant rotations (hybrid key switch, 6 digits), 172 032 ct-pt MACs, 224
rescales.  Inputs are seeded synthetic residues (uniform below each prime) of exactly those
shapes; arithmetic is data-independent, so timing equals that of real encodings.

  python bench.py [--gpus N] [--steps K] [--warmup W] [--impl reference]
  python bench.py --workload out_proj | conv | norm | scan_slice | scan_layer  (the other stages of a layer)
  python bench.py --workload rotations                                      (512 plain rotations, both digit layouts)

Prints ONE JSON line (rank 0).  `value` = key switches per second over the whole step, summed
over ranks (each rank runs its own 2048-token batch: weak scaling, no data-path collective);
`latency_ms` is the projection latency the metric names.  The default step uses hoisted baby
rotations and one division by P per output (--hoist 0 --defer 0: the plain definitions); beside
the headline the line carries `roofline`, `kernel_breakdown`, `e2e`, `clocks`, `cpu_baseline`,
`isolated` (ct-pt MAC and key-switch inner product alone) and `variants` (token blocks paired in
the real and imaginary channels).
"""
from __future__ import annotations

import argparse
import json
import os
import subprocess
import sys
import tempfile
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

METRIC = "encrypted 768->3352 projection latency at L=2048; key-switches/s; HBM GB/s vs peak"
T_SEG, C_SEG, N1, N2 = 128, 256, 32, 8
D_IN, D_OUT, TOKENS = 768, 3352, 2048
PROJ = "in_proj"            # "out_proj" (1536 -> 768) is selected by --workload out_proj
LEVEL = 24
BABY_BASE, GIANT_BASE = 1000, 1500
DIAG_SHIFT = 0              # log2 of the run length of periodic diagonals (token-major packing): 7 at C = 256
KEY_AMOUNTS = None          # (baby amounts, giant amounts) in slots when they are not q*T and p*n1*T


def workload_dims(scale_down: int = 1):
    gin = -(-D_IN // C_SEG)
    nout = -(-D_OUT // C_SEG)
    tbs = -(-TOKENS // T_SEG)
    if scale_down > 1:   # debugging aid only; never used for a reported number
        nout = max(1, nout // scale_down)
        tbs = max(1, tbs // scale_down)
    return gin, nout, tbs


def key_switches_per_step(gin, nout, tbs):
    return tbs * (gin * (N1 - 1) + nout * (N2 - 1))


# ---------------------------------------------------------------------------------------------
# distributed plumbing (one process per GPU; only a barrier and a max over ranks)
# ---------------------------------------------------------------------------------------------
def dist_setup(backend: str):
    import torch.distributed as dist

    world = int(os.environ.get("WORLD_SIZE", "1"))
    if world > 1 and not dist.is_initialized():
        dist.init_process_group(backend=backend)
    return int(os.environ.get("RANK", "0")), world


def max_over_ranks(value: float, device="cpu") -> float:
    import torch
    import torch.distributed as dist

    if not (dist.is_available() and dist.is_initialized()):
        return value
    t = torch.tensor([value], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def barrier():
    import torch.distributed as dist

    if dist.is_available() and dist.is_initialized():
        dist.barrier()


# ---------------------------------------------------------------------------------------------
# clocks
# ---------------------------------------------------------------------------------------------
class ClockSampler:
    QUERY = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
             "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
             "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index: int):
        self.gpu = gpu_index
        self.f = tempfile.NamedTemporaryFile("w+", suffix=".csv", delete=False)
        self.p = None

    def start(self):
        try:
            self.p = subprocess.Popen(["nvidia-smi", "-i", str(self.gpu), f"--query-gpu={self.QUERY}",
                                       "--format=csv,noheader,nounits", "-lms", "100"], stdout=self.f,
                                      stderr=subprocess.DEVNULL)
        except OSError:
            self.p = None

    def stop(self) -> dict:
        if self.p is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        self.p.terminate()
        try:
            self.p.wait(timeout=5)
        except subprocess.TimeoutExpired:
            self.p.kill()
        self.f.flush()
        self.f.seek(0)
        sm, mx, power, reasons = [], [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for line in self.f.read().splitlines():
            parts = [x.strip() for x in line.split(",")]
            if len(parts) < 9:
                continue
            try:
                sm.append(float(parts[1]))
                mx.append(float(parts[2]))
                power.append(float(parts[3]))
            except ValueError:
                continue
            for n, v in zip(names, parts[5:9]):
                if v.lower().startswith("active"):
                    reasons.add(n)
        os.unlink(self.f.name)
        if not sm:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["no samples"]}
        sm.sort()
        return {"sm_mhz": sm[len(sm) // 2], "sm_max_mhz": max(mx), "power_w_max": max(power),
                "samples": len(sm), "reasons": sorted(reasons)}


# ---------------------------------------------------------------------------------------------
# synthetic inputs
# ---------------------------------------------------------------------------------------------
def make_inputs(primes, n, gin, nout, tbs, seed, device, ctx=None, desc=None):
    """ct_in [tbs][gin][2][LEVEL][N] and the diagonals [nout][N2][gin][N1][LEVEL][N] filled with hashed
    residues; stream ids: ciphertext (tb,g) -> tb*gin+g, diagonal chunk (b,p) -> 100000 + b*N2+p.
    With desc.packed the diagonals of one output block at a time are generated and handed to
    fesc_linear_pack_diags (the one-off weight preparation, like the encoding itself outside the timed region);
    the byte-plane image (uint8) is returned instead of the residues."""
    import torch
    import fesc_synth as S

    q = primes[:LEVEL]
    ct = torch.empty((tbs, gin, 2, LEVEL, n), dtype=torch.int64, device=device)
    for tb in range(tbs):
        for g in range(gin):
            r = S.hashed_residues(seed, tb * gin + g, q, 2 * n, device=device)      # [LEVEL, 2n]
            ct[tb, g] = r.view(LEVEL, 2, n).permute(1, 0, 2)
    packed = bool(desc is not None and desc.packed)
    nd = n >> (desc.diag_run_log2 if desc is not None else 0)      # words per limb of a diagonal (periodic: one per run)
    per = 1                         # output blocks per pack call: a range must start at a multiple of 8 (b,p) pairs
    while (per * N2) % 8 and per < nout:
        per += 1
    if packed:
        assert (per * N2) % 8 == 0 or per == nout
        diags = torch.empty((ctx.linear_packed_bytes(desc),), dtype=torch.uint8, device=device)
        one = torch.empty((per, N2, gin, N1, LEVEL, nd), dtype=torch.int64, device=device)
    else:
        diags = torch.empty((nout, N2, gin, N1, LEVEL, n), dtype=torch.int64, device=device)
    for b in range(nout):
        for p in range(N2):
            r = S.hashed_residues(seed, 100000 + b * N2 + p, q, gin * N1 * nd, device=device)
            (one[b % per] if packed else diags[b])[p] = r.view(LEVEL, gin, N1, nd).permute(1, 2, 0, 3)
            del r
        if packed and (b % per == per - 1 or b == nout - 1):
            first, cnt = (b // per) * per, b % per + 1
            ctx.linear_pack_diags(one[:cnt], desc, first * N2, cnt * N2, diags)
    if packed:
        ctx.sync()
        del one
    return ct, diags


def peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        d = json.load(open(path))
        return float(d["hbm_gbs"]), "measured"
    return 6650.0, "fallback"


# ALU ceilings: issue rates per SM per clock (measured with register-only chains) and operations per unit of work.
SM_COUNT = 148
IMAD_PER_CLK_PER_SM = 64          # 32-bit multiply-adds per SM per clock (measured 63 with a register chain)
FP64_PER_CLK_PER_SM = 64          # FP64 FMAs per SM per clock (measured 63 with a register chain)
BFLY_IMAD = 20                    # integer Shoup butterfly (primes >= 2^50): 10 products of 32x32->64
BFLY_FP64 = 8.5                   # FP64 butterfly (primes < 2^50): 5 ops product + 2 adds + ~1.5 fold-back / conversion share
                                  # (counted per pass: 8.25 forward strided, 8.75 forward contiguous, 8.5-9.5 inverse)
MAC_FP64 = 6                      # FP64 multiply-accumulate: 5 ops exact product + 1 add
MAC_MIXED_CYCLES = 8              # mixed-pipe multiply-accumulate: multiplier-pipe cycles per warp (one 32x32+64 = 4,
                                  # two 32-bit multiply-adds = 2 each) on each of the 4 sub-partitions of an SM
# DRAM traffic of one accumulate launch is not captured at full size: a small-case capture of the same kernel
# (a few GB, inputs larger than L2) gives measured DRAM bytes / algorithmic bytes, and because every operand byte is
# read once per launch and every output byte written once, traffic grows in proportion to the algorithmic bytes.
BSGS_TRAFFIC_RATIO = {"packed": 1.000, "residues": 1.001}     # measured DRAM bytes / algorithmic bytes (small case)
PACKED_BYTES_PER_WORD = 7                                     # a residue below 2^56 as byte planes
NTT_DISPATCH_CYCLES = 27.1        # dispatch-port cycles per warp-butterfly of the FP64 transforms: 9.5 x 2 + 8.1 (ncu opcode mix)
NTT_TRAFFIC_RATIO = 1.0           # the transforms read and write every word of both passes through DRAM once
INT_LIMB_SHARE = 32.0 / 224.0     # transforms on the 60-bit special primes per key switch (integer path)


def isolated_kernels(ctx, fesc, torch, ct, out, hbm_peak, n):
    """The memory-bound kernels timed alone (CUDA events / the library's family timers), untimed part of the run:
    the plain ct-pt multiply-accumulate and one batch of 32 plain rotations by one key (key-switch inner product,
    limb transforms)."""
    res = {}
    word = 8
    batch = 32
    x = ct.reshape(-1, 2, LEVEL, n)[:batch]                          # 32 input ciphertexts of the step
    acc = out.reshape(-1)[: batch * 2 * LEVEL * n].view(batch, 2, LEVEL, n)
    pt = torch.empty((batch, LEVEL, n), dtype=torch.int64, device=ct.device)
    pt.copy_(x[:, 0])
    acc.zero_()
    for _ in range(3):
        ctx.ct_pt_mac(x, pt, acc, batch, LEVEL)
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    reps = 10
    e0.record()
    for _ in range(reps):
        ctx.ct_pt_mac(x, pt, acc, batch, LEVEL)
    e1.record()
    torch.cuda.synchronize()
    t = e0.elapsed_time(e1) * 1e-3 / reps
    by = batch * (2 + 1 + 2 + 2) * LEVEL * n * word                  # ct, pt, acc read, acc written
    res["ct_pt_mac"] = {"achieved": by / t / 1e9, "peak": hbm_peak, "unit": "GB/s", "frac": by / t / 1e9 / hbm_peak,
                        "bytes_per_launch": by, "macs_per_s": batch / t,
                        "l2": "operands of one launch 2.8 GB, larger than L2"}
    del pt
    # 32 rotations by one key (batches of 8 inside the library)
    ctx.rotate(x, acc, batch, LEVEL, BABY_BASE + 1)
    ctx.profile_enable(["ntt", "inner", "modup", "moddown", "autom"], 4096)
    c0 = ctx.counters()
    e0.record()
    ctx.rotate(x, acc, batch, LEVEL, BABY_BASE + 1)
    e1.record()
    torch.cuda.synchronize()
    fam = ctx.profile_read()
    ctx.profile_enable([])
    c1 = ctx.counters()
    t = e0.elapsed_time(e1) * 1e-3
    beta = ctx.num_digits
    rows = LEVEL + ctx.n_p
    launches = max(1, fam["inner"][1])
    by = batch * (beta + 2) * rows * n * word + launches * beta * 2 * rows * n * word   # digits in, sums out, key per launch
    ti = fam["inner"][0] * 1e-3
    res["evk_inner_product"] = {"achieved": by / ti / 1e9, "peak": hbm_peak, "unit": "GB/s", "frac": by / ti / 1e9 / hbm_peak,
                                "bytes": by, "launches": launches, "ms": fam["inner"][0]}
    res["rotation_batch32"] = {"key_switches_per_s": batch / t, "ms": t * 1e3,
                               "limb_transforms": c1[0] - c0[0],
                               "limb_transforms_per_s": (c1[0] - c0[0]) / (fam["ntt"][0] * 1e-3),
                               "family_ms": {k: round(v[0], 3) for k, v in fam.items() if v[1]}}
    return res


# ---------------------------------------------------------------------------------------------
# reference arm and CPU baseline: the oracle, timed as it stands on a bounded sample
# ---------------------------------------------------------------------------------------------
def oracle_sample(steps: int, warmup: int, hoist: bool = True, defer: bool = True):
    """One token block x one output block x ONE input block of the projection through the
    oracle: 31 baby + 7 giant rotations, 256 MACs, 1 rescale.  Returns (key-switches/s, ms/step, cores)."""
    import numpy as np
    import fesc_synth as S
    from oracle.ckks import Oracle

    p = S.params("full")
    orc = Oracle(p["log_n"], p["primes"], p["n_q"], p["n_p"], p["dnum"], p["seed"])
    for q in range(1, N1):
        orc.add_galois_key(q * T_SEG, BABY_BASE + q)
    for g in range(1, N2):
        orc.add_galois_key(g * N1 * T_SEG, GIANT_BASE + g)
    seed = S.config_seed(4)
    ct = np.empty((1, 1, 2, LEVEL, orc.N), dtype=np.uint64)
    for pp in range(2):
        ct[0, 0, pp] = S.uniform_residues_np(seed, pp, orc.q[:LEVEL], orc.N)
    diags = np.empty((1, N2, 1, N1, LEVEL, orc.N), dtype=np.uint64)
    for pp in range(N2):
        for q in range(N1):
            diags[0, pp, 0, q] = S.uniform_residues_np(seed, 10 + pp * N1 + q, orc.q[:LEVEL], orc.N)
    desc = dict(n1=N1, n2=N2)
    bk = {q: BABY_BASE + q for q in range(1, N1)}
    gk = {g: GIANT_BASE + g for g in range(1, N2)}
    for _ in range(warmup):
        orc.linear(ct, diags, desc, bk, gk, hoist=hoist, defer=defer)
    t0 = time.perf_counter()
    for _ in range(max(1, steps)):
        orc.linear(ct, diags, desc, bk, gk, hoist=hoist, defer=defer)
    dt = (time.perf_counter() - t0) / max(1, steps)
    ks = (N1 - 1) + (N2 - 1)
    cores = int(os.environ.get("OMP_NUM_THREADS", os.cpu_count() or 1))
    return ks / dt, dt * 1e3, cores


def workload_text(args):
    """config.workload of both arms (the reference arm times a bounded sample of this workload)."""
    return ("%s %d->%d, L=2048 tokens, N=2^16, 24x50-bit limbs + 4x60-bit special primes, "
            "6 key-switch digits, C=256 T=128 n1=%d n2=%d, baby rotations %s"
            % (PROJ, D_IN, D_OUT, N1, N2, "hoisted (one decomposition per input ciphertext)" if args.hoist else "by plain rotations")
            + (", one division by P per output for the giant-step sum" if args.defer else ""))


SAMPLE_TEXT = ("1 token block x 1 output block x 1 input block of the projection "
               "(31 baby + 7 giant rotations, 256 ct-pt MACs, 1 rescale; 1/672 of the step's MACs)")


def oracle_rates():
    """Per-operation rates of the oracle as it stands at N = 2^16 and 24 limbs (a few seconds of host time):
    limb transforms, ct-pt multiply-accumulates and plain rotations per second."""
    import numpy as np
    import fesc_synth as S
    from oracle.ckks import Oracle

    p = S.params("full")
    orc = Oracle(p["log_n"], p["primes"], p["n_q"], p["n_p"], p["dnum"], p["seed"])
    orc.add_galois_key(1, 7)
    seed = S.config_seed(3)
    idx = list(range(LEVEL))
    ct = np.stack([S.uniform_residues_np(seed, 50 + i, orc.q[:LEVEL], orc.N) for i in range(2)])
    pt = S.uniform_residues_np(seed, 60, orc.q[:LEVEL], orc.N)

    def rate(fn, units, min_s=1.5):
        fn()
        n, t0 = 0, time.perf_counter()
        while time.perf_counter() - t0 < min_s:
            fn()
            n += 1
        return units * n / (time.perf_counter() - t0)

    return {"limb_transforms_per_s": rate(lambda: orc.intt(orc.ntt(ct[0], idx), idx), 2 * LEVEL),
            "ct_pt_macs_per_s": rate(lambda: orc.ct_pt_mac(ct, pt, ct), 1),
            "rotations_per_s": rate(lambda: orc.rotate(ct, 7), 1, 3.0),
            "at": "N=2^16, 24 limbs (a ciphertext-level unit each; rotation = automorphism + hybrid key switch, 6 digits)"}


def measure_projection(args, ctx, dev, rank, world, key_base):
    """One projection workload (the module's D_IN, D_OUT, N1, N2) timed on `ctx`: keys, synthetic inputs, packed or
    residue diagonals, 3 warm-up steps, one profiled step, `args.steps` timed steps with the clocks sampled."""
    import torch
    import fesc_synth as S
    import paper_2608_17442_b200 as fesc

    p = S.params("full")
    n = ctx.N
    bb, gb = key_base
    baby = KEY_AMOUNTS[0] if KEY_AMOUNTS else [q * T_SEG for q in range(N1)]
    giant = KEY_AMOUNTS[1] if KEY_AMOUNTS else [g * N1 * T_SEG for g in range(N2)]
    assert len(baby) == N1 and len(giant) == N2
    for q in range(1, N1):
        ctx.add_galois_key(baby[q], bb + q)
    for g in range(1, N2):
        ctx.add_galois_key(giant[g], gb + g)
    gin, nout, tbs = workload_dims(1)
    desc = fesc.BsgsDesc(N1, N2, gin, nout, tbs, LEVEL, bb, gb, int(args.hoist), int(args.defer), int(args.packed),
                         DIAG_SHIFT if args.packed else 0)
    ct, diags = make_inputs(p["primes"], n, gin, nout, tbs, S.config_seed(5) + rank, dev, ctx, desc)
    out = torch.empty((tbs, nout, 2, LEVEL - 1, n), dtype=torch.int64, device=dev)
    torch.cuda.empty_cache()
    for _ in range(3):
        ctx.linear(ct, diags, desc, out)
    ctx.profile_enable(fesc.Context.PROFILE_FAMILIES, 120000)
    ctx.linear(ct, diags, desc, out)
    fam = ctx.profile_read()
    ctx.profile_enable([])
    c0 = ctx.counters()
    sampler = ClockSampler(torch.cuda.current_device())
    sampler.start()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(args.steps):
        ctx.linear(ct, diags, desc, out)
    e1.record()
    ctx.sync()
    clocks = sampler.stop()
    c1 = ctx.counters()
    ms = e0.elapsed_time(e1) / args.steps
    ks = (c1[1] - c0[1]) // args.steps
    res = {"ms": ms, "key_switches": ks, "key_switches_per_s": ks / (ms * 1e-3), "gpu_launches": (c1[4] - c0[4]) // args.steps,
           "clocks": clocks, "kernel_breakdown": {k: {"ms": round(v[0], 2), "records": v[1]} for k, v in fam.items() if v[1]},
           "workload": workload_text(args), "input_cts": tbs * gin, "output_cts": tbs * nout,
           "diagonals": nout * N2 * gin * N1, "diagonals_gib": diags.numel() * diags.element_size() / 2**30,
           "token_blocks_per_group": int(c1[5])}
    del ct, diags, out
    return res


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    value, ms, cores = oracle_sample(args.steps, args.warmup, bool(args.hoist), bool(args.defer))
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": "key-switches/s",
        "n_gpus": args.gpus, "steps": args.steps, "warmup": args.warmup, "ms_per_step": ms,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "u64", "data": "synthetic",
        "config": {"workload": workload_text(args), "sample_per_step": SAMPLE_TEXT},
        "cpu_baseline": {"value": value, "unit": "key-switches/s", "cores": cores, "kind": "oracle",
                         "sample": SAMPLE_TEXT, "rates": oracle_rates()},
        "e2e": {"value": value, "unit": "key-switches/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line), flush=True)


def measure_variants(args, ctx, ct, diags, out, gin, nout, tbs, n, dev):
    """The same 2048 x 768 -> 3352 job with two real blocks in the real and imaginary channels of one ciphertext
    (token blocks, or the paper's input blocks); reported beside the headline."""
    import torch
    import paper_2608_17442_b200 as fesc

    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    # the same 2048 x 768 -> 3352 job with token blocks (2u, 2u+1) paired in the real and imaginary channels:
    # half the ciphertexts go through fesc_linear (real diagonals act on complex slots), then one conjugation
    # per output separates the two results.  Reported beside the headline, which keeps one block per ciphertext.
    conj_id = GIANT_BASE + 400
    ctx.add_galois_key(fesc.CONJ, conj_id)
    half = tbs // 2
    desc2 = fesc.BsgsDesc(N1, N2, gin, nout, half, LEVEL, BABY_BASE, GIANT_BASE, int(args.hoist), int(args.defer),
                          int(args.packed))
    zc = torch.empty((half * nout, 2, LEVEL - 1, n), dtype=torch.int64, device=dev)
    o2 = out.reshape(2, half * nout, 2, LEVEL - 1, n)

    def paired():
        ctx.linear(ct[:half], diags, desc2, zc)
        ctx.split_complex(zc, o2[0], o2[1], half * nout, LEVEL - 1, conj_id)

    paired()
    c0 = ctx.counters()
    torch.cuda.synchronize()
    e0.record()
    for _ in range(args.steps):
        paired()
    e1.record()
    torch.cuda.synchronize()
    c1 = ctx.counters()
    v_ms = e0.elapsed_time(e1) / args.steps
    variants = {"paired_token_blocks": {"latency_ms": v_ms, "key_switches_per_step": (c1[1] - c0[1]) // args.steps,
                                        "input_cts": half * gin, "output_cts": 2 * half * nout,
                                        "note": "token blocks 2u and 2u+1 in the real and imaginary channels; "
                                                "fesc_linear on 8 complex token blocks + fesc_split_complex"}}
    del zc
    # the paper's own pairing (App. "Projection Kernel Breakdown"): input blocks 2u and 2u+1 in the real and
    # imaginary channels with complex diagonals, real part of every output by one conjugation.  Timed on the same
    # buffers reinterpreted as ceil(gin/2) input blocks (residues are random either way).
    gp = -(-gin // 2)
    if gp < gin:
        desc3 = fesc.BsgsDesc(N1, N2, gp, nout, tbs, LEVEL, BABY_BASE, GIANT_BASE, int(args.hoist), int(args.defer),
                              int(args.packed))
        ct3 = ct.reshape(-1)[: tbs * gp * 2 * LEVEL * n].view(tbs, gp, 2, LEVEL, n)
        if args.packed:      # any bytes are valid byte planes: the head of the image serves as the smaller image
            dg3 = diags[: ctx.linear_packed_bytes(desc3)]
        else:
            dg3 = diags.reshape(-1)[: nout * N2 * gp * N1 * LEVEL * n].view(nout, N2, gp, N1, LEVEL, n)
        z3 = torch.empty((tbs * nout, 2, LEVEL - 1, n), dtype=torch.int64, device=dev)
        o3 = out.reshape(tbs * nout, 2, LEVEL - 1, n)

        def paired_in():
            ctx.linear(ct3, dg3, desc3, z3)
            ctx.split_complex(z3, o3, None, tbs * nout, LEVEL - 1, conj_id)

        paired_in()
        c0 = ctx.counters()
        torch.cuda.synchronize()
        e0.record()
        for _ in range(args.steps):
            paired_in()
        e1.record()
        torch.cuda.synchronize()
        c1 = ctx.counters()
        variants["paired_input_blocks"] = {
            "latency_ms": e0.elapsed_time(e1) / args.steps, "key_switches_per_step": (c1[1] - c0[1]) // args.steps,
            "input_cts": tbs * gp, "output_cts": tbs * nout,
            "note": "input blocks 2u and 2u+1 in the real and imaginary channels, complex diagonals; "
                    "fesc_linear on %d input blocks + real part by fesc_split_complex" % gp}
        del z3
    return variants


def bsgs_roofline(args, gin, nout, n, tb_per_launch, timed, hbm_peak, sm_mhz):
    """Roofline of the accumulate family from (milliseconds, launches).  Packed operands: the kernel streams the
    byte-plane image once per launch (7 bytes per diagonal word), the packed inputs of its token blocks and writes the
    partial sums: HBM-bound; the tensor-core ceiling (u8 mma.sync m16n8k32 at 8 cycles per scheduler, measured) is
    reported beside it.  Residue operands: the multiplier-pipe bound of the mixed-pipe kernel."""
    ms, launches = timed
    t = ms * 1e-3 / max(1, launches)
    ctw = 2 * LEVEL * n * 8
    terms, bp = gin * N1, nout * N2
    macs = tb_per_launch * bp * terms * 2 * LEVEL * n
    if args.packed:
        ksteps = -(-terms // 32)
        image = -(-bp // 8) * LEVEL * n * ksteps * 1792                      # bytes: 8 rows x 32 terms x 7 planes per image
        xpk = -(-2 * tb_per_launch // 8) * LEVEL * n * ksteps * 1792
        alg = image + xpk + tb_per_launch * bp * ctw
        mma = -(-bp // 8) * ksteps * 28 * LEVEL * n * -(-tb_per_launch // 4)      # m16n8k32 instructions per launch
        tensor_peak = SM_COUNT * 4 * sm_mhz * 1e6 / 8                            # instructions / s
        return {"kernel": "bsgs", "variant": "k_bsgs_accumulate_packed (byte planes on the tensor cores)", "bound": "hbm",
                "achieved": alg / t / 1e9, "peak": hbm_peak, "unit": "GB/s", "frac": alg / t / 1e9 / hbm_peak,
                "traffic": alg * BSGS_TRAFFIC_RATIO["packed"], "algorithmic_bytes_per_launch": alg,
                "avg_launch_ms": t * 1e3, "launches": launches, "token_blocks_per_launch": tb_per_launch,
                "modular_macs_per_s": macs / t,
                "tensor": {"achieved": mma / t, "peak": tensor_peak, "unit": "u8 m16n8k32 mma.sync / s", "frac": mma / t / tensor_peak}}
    alg = tb_per_launch * terms * ctw + bp * terms * (ctw // 2) + tb_per_launch * bp * ctw
    alu_peak = SM_COUNT * 4 * 32 * sm_mhz * 1e6 / MAC_MIXED_CYCLES / 1e12
    return {"kernel": "bsgs", "variant": "residue operands", "bound": "alu", "achieved": macs / t / 1e12, "peak": alu_peak,
            "unit": "T modular mac/s (integer multiplier pipe, 8 cycles per warp-mac)", "frac": macs / t / 1e12 / alu_peak,
            "traffic": alg * BSGS_TRAFFIC_RATIO["residues"], "avg_launch_ms": t * 1e3, "launches": launches,
            "token_blocks_per_launch": tb_per_launch,
            "hbm": {"achieved": alg / t / 1e9, "peak": hbm_peak, "unit": "GB/s", "frac": alg / t / 1e9 / hbm_peak,
                    "algorithmic_bytes_per_launch": alg}}


def ntt_roofline(p, n, timed, limb_ntts, hbm_peak, sm_mhz):
    """All transform launches of the measured steps: butterflies per second against the FP64 / integer issue ceiling,
    and the bytes the two passes of a limb transform move against the HBM peak."""
    ms, launches = timed
    bfly = limb_ntts * (n // 2) * p["log_n"]
    peak_fp = SM_COUNT * FP64_PER_CLK_PER_SM * sm_mhz * 1e6 / BFLY_FP64 / 1e12
    peak_int = SM_COUNT * IMAD_PER_CLK_PER_SM * sm_mhz * 1e6 / BFLY_IMAD / 1e12
    alu_peak = 1.0 / ((1.0 - INT_LIMB_SHARE) / peak_fp + INT_LIMB_SHARE / peak_int)
    ach = bfly / (ms * 1e-3) / 1e12
    moved = limb_ntts * 2 * 2 * n * 8           # two passes, each reads and writes the limb
    # What the dispatch port allows with the measured instruction mix of the FP64 path (ncu opcode counts: 17.6 warp
    # instructions per warp-butterfly, 9.5 of them FP64, which hold the port for two cycles): 27.1 cycles per
    # warp-butterfly on each of the 4 schedulers of an SM.  The kernels also have to load, exchange and store, so this,
    # not the FP64-pipe figure above, is the ceiling they can approach.
    issue_peak = SM_COUNT * 4 * 32 * sm_mhz * 1e6 / NTT_DISPATCH_CYCLES / 1e12
    return {"kernel": "ntt", "variant": "ntt16_strided + ntt16_contig (two passes per limb transform)", "bound": "alu",
            "achieved": ach, "peak": alu_peak, "unit": "T butterflies/s (FP64 pipe for 50-bit primes, integer pipe for 60-bit)",
            "peak_fp64_path": peak_fp, "peak_integer_path": peak_int, "frac": ach / alu_peak,
            "traffic": moved / max(1, launches) * NTT_TRAFFIC_RATIO, "launches": launches, "limb_transforms": limb_ntts,
            "us_per_limb_transform": ms * 1e3 / max(1, limb_ntts), "family_ms": ms,
            "dispatch": {"achieved": ach, "peak": issue_peak, "unit": "T butterflies/s", "frac": ach / issue_peak,
                         "cycles_per_warp_butterfly": NTT_DISPATCH_CYCLES},
            "hbm": {"achieved": moved / (ms * 1e-3) / 1e9, "peak": hbm_peak, "unit": "GB/s",
                    "frac": moved / (ms * 1e-3) / 1e9 / hbm_peak, "bytes_moved_per_limb_transform": 4 * n * 8}}


# ---------------------------------------------------------------------------------------------
def run_ours(args):
    import torch
    import fesc_synth as S
    import paper_2608_17442_b200 as fesc

    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device (there is no CPU fallback)")
    local = int(os.environ.get("LOCAL_RANK", "0"))
    torch.cuda.set_device(local)
    rank, world = dist_setup("nccl")
    dev = torch.device("cuda", local)

    p = S.params("full")
    ctx = fesc.Context(p["log_n"], p["primes"], p["n_q"], p["n_p"], p["dnum"], p["seed"])
    n = ctx.N
    gin, nout, tbs = workload_dims(args.scale_down)
    if args.profile_case:
        # small case for profiler captures, a few GB on the device, inputs larger than L2: the accumulate keeps its
        # full-size structure (96 terms = 3 k-steps, 4 tiles of 8 (b,p) outputs, 4 token blocks) at 4 limbs, and the
        # rotations run on batches of 48 and 32 ciphertexts; 10 Galois keys instead of 38
        global N1, N2, LEVEL
        N1, N2, LEVEL = 8, 4, 4
        gin, nout, tbs = 12, 8, 4
    for q in range(1, N1):
        ctx.add_galois_key(q * T_SEG, BABY_BASE + q)
    for g in range(1, N2):
        ctx.add_galois_key(g * N1 * T_SEG, GIANT_BASE + g)
    ks_per_step = key_switches_per_step(gin, nout, tbs)
    desc = fesc.BsgsDesc(N1, N2, gin, nout, tbs, LEVEL, BABY_BASE, GIANT_BASE, int(args.hoist), int(args.defer),
                         int(args.packed))
    ct, diags = make_inputs(p["primes"], n, gin, nout, tbs, S.config_seed(4) + rank, dev, ctx, desc)
    out = torch.empty((tbs, nout, 2, LEVEL - 1, n), dtype=torch.int64, device=dev)
    torch.cuda.empty_cache()

    def step():
        ctx.linear(ct, diags, desc, out)

    if args.profile_case or args.profile_step:
        # one bare step for a profiler capture (no warm-up, no timing claims)
        step()
        torch.cuda.synchronize()
        print(json.dumps({"profile_run": True, "gpu_launches": ctx.counters()[4],
                          "dims": {"in_blocks": gin, "out_blocks": nout, "token_blocks": tbs}}), flush=True)
        return

    # warm-up (also sizes the scratch arena) and a family breakdown on one untimed step
    for _ in range(max(3, args.warmup) - 1):
        step()
    ctx.profile_enable(fesc.Context.PROFILE_FAMILIES, 120000)
    limb_ntts_profiled = ctx.counters()[0]
    step()
    fam = ctx.profile_read()
    limb_ntts_profiled = ctx.counters()[0] - limb_ntts_profiled
    ctx.profile_enable([])
    total_fam = sum(v[0] for v in fam.values()) or 1.0
    breakdown = {k: {"ms": round(v[0], 3), "records": v[1], "share": round(v[0] / total_fam, 4)} for k, v in fam.items()}
    dominant = max(fam, key=lambda k: fam[k][0])

    # timed region
    ctx.profile_enable([dominant], 120000)
    launches0 = ctx.counters()[4]
    limb_ntts0 = ctx.counters()[0]
    sampler = ClockSampler(local)
    torch.cuda.synchronize()
    barrier()
    sampler.start()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(args.steps):
        step()
    e1.record()
    torch.cuda.synchronize()
    barrier()
    clocks = sampler.stop()
    ms_total = max_over_ranks(e0.elapsed_time(e1), dev)
    launches = ctx.counters()[4] - launches0
    limb_ntts = ctx.counters()[0] - limb_ntts0
    dom_ms, dom_records = ctx.profile_read()[dominant]
    ctx.profile_enable([])
    ms_per_step = ms_total / args.steps
    value = world * ks_per_step / (ms_per_step * 1e-3)

    # rooflines of the two heavy kernel families; `roofline` is the dominant one
    hbm_peak, peak_kind = peaks()
    sm_mhz = clocks.get("sm_mhz") or 1350.0
    tb_per_launch = int(ctx.counters()[5]) or tbs
    fam_roofs = {"bsgs": bsgs_roofline(args, gin, nout, n, tb_per_launch, fam["bsgs"], hbm_peak, sm_mhz),
                 "ntt": ntt_roofline(p, n, fam["ntt"], limb_ntts_profiled, hbm_peak, sm_mhz)}
    if dominant in fam_roofs:
        # the dominant family was event-timed over the whole timed region: use those launches
        if dominant == "bsgs":
            fam_roofs["bsgs"] = bsgs_roofline(args, gin, nout, n, tb_per_launch, (dom_ms, dom_records), hbm_peak, sm_mhz)
        else:
            fam_roofs["ntt"] = ntt_roofline(p, n, (dom_ms, dom_records), limb_ntts, hbm_peak, sm_mhz)
        roof = dict(fam_roofs[dominant], timed="all launches of the timed steps")
    else:
        roof = {"kernel": dominant, "bound": "alu", "achieved": None, "peak": None, "unit": "ms/launch", "frac": None,
                "traffic": None, "avg_launch_ms": dom_ms / max(1, dom_records)}
    roof["peak_source"] = peak_kind
    others = {k: dict(v, timed="one profiled step") for k, v in fam_roofs.items() if k != dominant}

    # end to end: pinned host inputs -> device, projection, result -> pinned host, every step, all inside the timed
    # region.  The copies run on their own streams with double-buffered device tensors, so the upload of step i+1
    # and the download of step i-1 overlap the projection of step i (what a caller streaming batches would do).
    h_in = torch.empty(ct.shape, dtype=torch.int64, pin_memory=True)
    h_in.copy_(ct)
    h_out = torch.empty(out.shape, dtype=torch.int64, pin_memory=True)
    e2e_steps = max(1, min(args.steps, 3))
    cts, outs = [ct, torch.empty_like(ct)], [out, torch.empty_like(out)]
    s_comp = torch.cuda.current_stream()
    s_in, s_out = torch.cuda.Stream(), torch.cuda.Stream()
    ev_in = [torch.cuda.Event() for _ in range(2)]
    ev_comp = [torch.cuda.Event() for _ in range(2)]
    ev_d2h = [torch.cuda.Event() for _ in range(2)]
    torch.cuda.synchronize()
    barrier()
    e0.record()
    s_in.wait_stream(s_comp)
    s_out.wait_stream(s_comp)
    for i in range(e2e_steps):
        b = i & 1
        with torch.cuda.stream(s_in):
            if i >= 2:
                s_in.wait_event(ev_comp[b])          # the projection that read this input buffer is done
            cts[b].copy_(h_in, non_blocking=True)
            ev_in[b].record(s_in)
        s_comp.wait_event(ev_in[b])
        if i >= 2:
            s_comp.wait_event(ev_d2h[b])             # the download of this output buffer is done
        ctx.linear(cts[b], diags, desc, outs[b])
        ev_comp[b].record(s_comp)
        with torch.cuda.stream(s_out):
            s_out.wait_event(ev_comp[b])
            h_out.copy_(outs[b], non_blocking=True)
            ev_d2h[b].record(s_out)
    s_comp.wait_stream(s_out)
    s_comp.wait_stream(s_in)
    e1.record()
    torch.cuda.synchronize()
    barrier()
    e2e_ms = max_over_ranks(e0.elapsed_time(e1), dev) / e2e_steps
    # one request on its own: upload, projection, download on ONE stream, nothing overlapped
    torch.cuda.synchronize()
    barrier()
    e0.record()
    cts[0].copy_(h_in, non_blocking=True)
    ctx.linear(cts[0], diags, desc, outs[0])
    h_out.copy_(outs[0], non_blocking=True)
    e1.record()
    torch.cuda.synchronize()
    barrier()
    single_ms = max_over_ranks(e0.elapsed_time(e1), dev)
    e2e = {"value": world * ks_per_step / (e2e_ms * 1e-3), "unit": "key-switches/s", "latency_ms": e2e_ms,
           "h2d_bytes_per_step": ct.numel() * 8, "d2h_bytes_per_step": out.numel() * 8,
           "overlap": "copies on separate streams, double-buffered device tensors (throughput of a stream of requests)",
           "single_shot_ms": single_ms,
           "single_shot": "one upload -> projection -> download on one stream, nothing overlapped (latency of one request)"}
    del cts, outs
    torch.cuda.empty_cache()

    isolated = isolated_kernels(ctx, fesc, torch, ct, out, hbm_peak, n) if (rank == 0 and args.scale_down == 1) else None
    variants = None
    if rank == 0 and args.scale_down == 1 and tbs % 2 == 0:
        variants = measure_variants(args, ctx, ct, diags, out, gin, nout, tbs, n, dev)
    stages = None
    config_extra = {"l2": "inputs larger than L2 (diagonals %.1f GiB stream every step)" % (diags.numel() * diags.element_size() / 2**30),
                    "diagonals_as": ("byte-plane image, %.1f GiB, packed once outside the timed region" % (diags.numel() / 2**30)
                                     if args.packed else "residues")}
    if rank == 0 and world == 1 and args.scale_down == 1 and args.stages and PROJ == "in_proj":
        del ct, diags, out, h_in, h_out
        torch.cuda.empty_cache()
        ctx.trim()
        stages = run_stages(args, ctx, dev)
    line = {
        "metric": METRIC, "value": value, "unit": "key-switches/s", "n_gpus": world, "steps": args.steps,
        "warmup": max(3, args.warmup), "ms_per_step": ms_per_step, "latency_ms": ms_per_step,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "u64", "data": "synthetic",
        "config": {"workload": workload_text(args),
                   "input_cts": tbs * gin, "diagonals": nout * N2 * gin * N1, "output_cts": tbs * nout,
                   "key_switches_per_step": ks_per_step, "macs_per_step": tbs * nout * N2 * gin * N1,
                   "l2": config_extra["l2"], "diagonals_as": config_extra["diagonals_as"],
                   "token_blocks_per_group": tb_per_launch,
                   "parallelism": "replicas x%d (independent 2048-token batches)" % world},
        "clocks": clocks, "e2e": e2e, "gpu_launches": int(launches),
        "roofline": roof, "roofline_other": others, "kernel_breakdown": breakdown,
    }
    if isolated:
        line["isolated"] = isolated
    if variants:
        line["variants"] = variants
    if stages:
        line["stages"] = stages
    if args.scale_down > 1:
        line["config"]["workload"] += " [DEBUG scale_down=%d: not a reportable number]" % args.scale_down
    if rank == 0 and world == 1 and not args.no_cpu:
        v, ms, cores = oracle_sample(1, 0, bool(args.hoist), bool(args.defer))
        line["cpu_baseline"] = {"value": v, "unit": "key-switches/s", "cores": cores, "kind": "oracle",
                                "sample": SAMPLE_TEXT, "ms": ms, "rates": oracle_rates()}
    if rank == 0:
        print(json.dumps(line), flush=True)
    del ctx


# ---------------------------------------------------------------------------------------------
# optional second workload: the scan-contract of one Mamba-2-base layer (or a slice of it)
# ---------------------------------------------------------------------------------------------
def scan_rotation_amounts(n, P, d_s, B, stride, hoist=False, group=0):
    """Slot rotations the scan-contract uses (see include/fesc.h), as left shifts modulo n."""
    import math

    dg = min(16, B)
    Bt = B // max(1, B // stride)                 # tokens per segment
    dgt = min(16, Bt)
    c_state = n // stride
    R = P * stride
    am = set()
    for unit in (1, P):                           # x, a: offsets inside a segment
        am |= {unit * t % n for t in range(1, dgt)} | {unit * dgt * t % n for t in range(1, Bt // dgt)}
    am |= {d_s * t % n for t in range(1, dg)} | {d_s * dg * t % n for t in range(1, B // dg)}      # B, C
    am |= {(-t) % n for t in range(1, dgt)} | {(-dgt * t) % n for t in range(1, Bt // dgt)}        # output placement
    am |= {(-(1 << b)) % n for b in range(int(math.log2(max(d_s, P))))}
    am |= {(-P * (1 << b)) % n for b in range(int(math.log2(R // P)))}
    am |= {(-stride * (1 << b)) % n for b in range(int(math.log2(c_state)))}
    am |= {(1 << b) for b in range(int(math.log2(d_s)))}
    if hoist:    # radix-4 rotate-and-add chains also rotate by 3 * unit * 2^b (b even, b + 1 < steps)
        lg = lambda v: int(math.log2(v))
        for unit, steps in ((-1, lg(P)), (-1, lg(d_s)), (-P, lg(R // P)), (-stride, lg(c_state)), (1, lg(d_s))):
            am |= {(3 * unit * (1 << b)) % n for b in range(0, steps - 1, 2)}
    if group:    # grouped leaf build: group offsets (two digits) and the class shifts +-unit .. +-(G-1) unit
        cnt = Bt // group
        dgg = min(16, cnt)
        for unit in (group, group * P):
            am |= {unit * t % n for t in range(1, dgg)} | {unit * dgg * t % n for t in range(1, cnt // dgg)}
        if hoist:
            for unit, steps in ((-group, int(math.log2(d_s // group))), (-group * P, int(math.log2(R // (group * P))))):
                am |= {(3 * unit * (1 << b)) % n for b in range(0, steps - 1, 2)}
        for unit in (1, P, d_s):
            am |= {(k * unit) % n for k in range(1, group)} | {(-k * unit) % n for k in range(1, group)}
        cnt_b, unit = B // group, group * d_s                   # br(B): groups of `group` tokens = unit slots
        dg_b = min(16, cnt_b)
        am |= {unit * t % n for t in range(1, dg_b)} | {unit * dg_b * t % n for t in range(1, cnt_b // dg_b)}
        am |= {(-unit * (1 << b)) % n for b in range(int(math.log2(n // unit)))}
        if hoist:
            am |= {(-3 * unit * (1 << b)) % n for b in range(0, int(math.log2(n // unit)) - 1, 2)}
    am.discard(0)
    return sorted(am)


def scan_partition(K_s: int, world: int):
    """State chunks of every rank: chunk PAIRS (2l, 2l+1) stay together (they are reduced in the real and imaginary
    lanes of one ciphertext); pairs are dealt out in contiguous, near-equal runs.  Returns [(first chunk, count)]."""
    pairs = -(-K_s // 2)
    out = []
    for r in range(world):
        lo, hi = pairs * r // world, pairs * (r + 1) // world
        first, end = 2 * lo, min(2 * hi, K_s)
        out.append((first, max(0, end - first)))
    return out


def gather_chunk_outputs(local, parts, rank, world, K_blk, K_s):
    """The one exchange of the sharded scan: every rank contributes the output ciphertexts of its chunks
    ([K_blk, chunks, ...]); all ranks end with the full [K_blk, K_s, ...] tensor.  One all_gather of equal-sized
    buffers (ranks with fewer chunks pad), NCCL on GPUs, gloo in the CPU test."""
    import torch
    import torch.distributed as dist

    width = max(c for _, c in parts)
    tail = tuple(local.shape[2:])
    buf = torch.zeros((K_blk, width) + tail, dtype=local.dtype, device=local.device)
    buf[:, : local.shape[1]] = local
    if world > 1:
        bufs = [torch.empty_like(buf) for _ in range(world)]
        dist.all_gather(bufs, buf)
    else:
        bufs = [buf]
    full = torch.empty((K_blk, K_s) + tail, dtype=local.dtype, device=local.device)
    for r, (first, count) in enumerate(parts):
        if count:
            full[:, first:first + count] = bufs[r][:, :count]
    return full


def run_scan(args, ctx=None, quiet=False):
    """Times fesc_scan_contract on synthetic residues of the deployed geometry (N=2^16, 24 limbs, stride 256,
    B_blk=256, d_s=128, P=64).  --workload scan_slice: 4 heads x 512 tokens; scan_layer: 24 heads x 2048 tokens.
    With --gpus N (one process per GPU) the state chunks are dealt out to the ranks in pairs (Alg. 7: chunks are
    independent; the compact factors B, C are replicated) and the outputs are exchanged ONCE at the end by an
    all-gather, inside the timed region: strong scaling, time = max over ranks."""
    import torch
    import fesc_synth as S
    import paper_2608_17442_b200 as fesc

    rank, world = dist_setup("nccl")
    local = int(os.environ.get("LOCAL_RANK", "0"))
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    p = S.params("full")
    if ctx is None:
        ctx = fesc.Context(p["log_n"], p["primes"], p["n_q"], p["n_p"], p["dnum"], p["seed"])
    n, N = ctx.N // 2, ctx.N
    H, L = (4, 512) if args.workload == "scan_slice" else (24, 2048)
    P, d_s, B, stride, l0 = 64, 128, 256, int(args.stride), int(args.scan_limbs)
    if stride == 128 and args.workload == "scan_slice":
        H = 8                                                  # one chunk pair of 4 heads per chunk
    K_s, K_blk = H * P // (n // stride), L // B
    segs = max(1, B // stride)
    hpc = (n // stride) // P                                   # heads per chunk
    parts = scan_partition(K_s, world)
    first, mine = parts[rank]
    base = 100000
    G = int(args.group)
    for r in scan_rotation_amounts(n, P, d_s, B, stride, bool(args.hoist), G):
        ctx.add_galois_key(r, base + r)
    ctx.add_galois_key(fesc.CONJ, base + n)
    seed = S.config_seed(5)
    q = p["primes"][:l0]

    def cts(count, stream):
        r = S.hashed_residues(seed, stream, q, count * 2 * N, device=dev)
        return r.view(l0, count, 2, N).permute(1, 2, 0, 3).contiguous()

    def chunk_cts(stream):                                     # [K_blk][mine][segs] ciphertexts of this rank's chunks only
        out_c = torch.empty((K_blk, max(mine, 1), segs, 2, l0, N), dtype=torch.int64, device=dev)
        for j in range(K_blk):                                 # ciphertext (block j, chunk k, segment g) = index (j*K_s + k)*segs + g
            for k in range(mine):
                lo = ((j * K_s + first + k) * segs) * 2 * N
                r = S.hashed_residues(seed, stream, q, segs * 2 * N, device=dev, first=lo)
                out_c[j, k] = r.view(l0, segs, 2, N).permute(1, 2, 0, 3)
        return out_c

    x, a = chunk_cts(1), chunk_cts(2)
    Bc, Cc = cts(K_blk, 3), cts(K_blk, 4)
    masks = [S.hashed_residues(seed, 10 + i, q, N, device=dev).contiguous() for i in range(4)]
    net = {"bk": fesc.NET_BRENT_KUNG, "ks": fesc.NET_KOGGE_STONE, "sk": fesc.NET_SKLANSKY}[args.network]
    # injection level: 2 log2(B) - 1 network stages below the leaves (Brent-Kung), or log2(B) stages and the carries
    l1 = l0 - 3 if G else l0 - 2                               # the grouped leaf build spends one more level
    linj = l1 - 2 * 8 + 1 if args.network == "bk" else l1 - 8 - max(K_blk - 2, 0)
    gm = None
    if G:
        gm = [S.hashed_residues(seed, 20, q, N, device=dev).contiguous(),
              S.hashed_residues(seed, 21, q, N, device=dev).contiguous(),
              S.hashed_residues(seed, 22, q[:l0 - 1], G * N, device=dev).view(l0 - 1, G, N).permute(1, 0, 2).contiguous(),
              S.hashed_residues(seed, 23, q[:l0 - 1], G * N, device=dev).view(l0 - 1, G, N).permute(1, 0, 2).contiguous(),
              S.hashed_residues(seed, 24, q, N, device=dev).contiguous(),
              S.hashed_residues(seed, 25, q[:l0 - 1], G * N, device=dev).view(l0 - 1, G, N).permute(1, 0, 2).contiguous()]
    out = torch.empty((K_blk, max(mine, 1), segs, 2, linj - 3, N), dtype=torch.int64, device=dev)
    adj = [(1 << 49) + 12345 * i for i in range((l0 + 1) ** 2)]
    plain = int(getattr(args, "plain", 0))
    pts = None
    if plain:       # invariant families: plaintext tables (abar powers, Bbar, Cbar) in place of the a, B, C ciphertexts
        rows = lambda stream, count, lim: S.hashed_residues(seed, stream, q[:lim], count * N, device=dev).view(lim, count, N).permute(1, 0, 2).contiguous()
        pts = [rows(30, 1, l0 - 2 if G else l0 - 1)[0], rows(31, 1, linj - 1)[0], rows(32, 8, l0), rows(33, 7, l0),
               rows(34, K_blk, l0), rows(35, B, linj)]
    desc = fesc.ScanDesc(L, mine * hpc, P, d_s, B, stride, l0, base, int(args.hoist), net, G, plain)
    torch.cuda.empty_cache()

    def step():
        if mine:
            ctx.scan_contract(x, a, Bc, Cc, desc, masks[0], masks[1], masks[2], masks[3][:linj - 2], adj, adj, out, gm, pts)
        return gather_chunk_outputs(out[:, :mine], parts, rank, world, K_blk, K_s) if world > 1 else out

    if args.profile_step:           # one bare step for a profiler's launch list (no warm-up, no timing claims)
        step()
        ctx.sync()
        if rank == 0:
            print(json.dumps({"profile_run": True, "gpu_launches": ctx.counters()[4], "key_switches": ctx.counters()[1]}),
                  flush=True)
        return
    breakdown = None
    if args.workload == "scan_slice":
        step()                      # warm-up (sizes the scratch arena)
        ctx.sync()
        ctx.profile_enable(fesc.Context.PROFILE_FAMILIES, 600000)
        step()                      # family breakdown on an untimed step
        fam = ctx.profile_read()
        ctx.profile_enable([])
        breakdown = {k: {"ms": round(v[0], 1), "records": v[1]} for k, v in fam.items() if v[1]}
    ctx.sync()
    barrier()
    c0 = ctx.counters()
    sampler = ClockSampler(local)
    sampler.start()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    step()
    e1.record()
    ctx.sync()
    barrier()
    clocks = sampler.stop()
    c1 = ctx.counters()
    ms = max_over_ranks(e0.elapsed_time(e1), dev)
    ks_local = torch.tensor([float(c1[1] - c0[1])], dtype=torch.float64, device=dev)
    if world > 1:
        import torch.distributed as dist
        dist.all_reduce(ks_local)
    ks = int(ks_local.item())
    res = None
    if rank == 0:
        res = ({"metric": "scan-contract key-switches/s", "value": ks / (ms * 1e-3), "unit": "key-switches/s",
                          "n_gpus": world, "steps": 1, "warmup": 1 if args.workload == "scan_slice" else 0,
                          "ms_per_step": ms, "higher_is_better": True, "scaling": "strong", "dtype": "u64",
                          "data": "synthetic",
                          "config": {"workload": "%s: L=%d, H=%d, P=64, d_s=128, B_blk=256, stride=%d, K_s=%d, N=2^16, %d limbs, %s network, %s"
                                                 % (args.workload, L, H, stride, K_s, l0,
                                                    {"bk": "Brent-Kung", "ks": "Kogge-Stone", "sk": "Sklansky"}[args.network],
                                                    ("radix-4 hoisted rotate-and-add chains" if args.hoist else "plain rotations")
                                                    + (", leaves built in groups of %d tokens" % G if G else "")
                                                    + (", invariant-family mode (plaintext decay, B, C)" if plain else "")),
                                     "parallelism": "state chunks in pairs over %d rank(s): %s; one all-gather of the outputs"
                                                    % (world, [c for _, c in parts])},
                          "key_switches": ks, "limb_transforms": c1[0] - c0[0], "gpu_launches": c1[4] - c0[4],
                          "scratch_gib": c1[3] / 2**30, "clocks": clocks, "kernel_breakdown": breakdown})
        if not quiet:
            print(json.dumps(res), flush=True)
    return res


def run_rotations(args):
    """Key-switch / rotation workload: 32 ciphertexts (N = 2^16, 24 limbs), 16 key slots (rotations 1..8 and 8*{1..8}),
    512 plain rotations per step, for the graded digit layout (6 digits of 4 limbs) and the literal dnum = 4 layout
    (4 digits of 6 limbs): rotations/s, evaluation-key GB/s, limb transforms/s."""
    import torch
    import fesc_synth as S
    import paper_2608_17442_b200 as fesc

    torch.cuda.set_device(0)
    hbm_peak, _ = peaks()
    res = {}
    amounts = list(range(1, 9)) + [8 * g for g in range(1, 9)]
    for name in ("full", "full_literal"):
        p = S.params(name)
        ctx = fesc.Context(p["log_n"], p["primes"], p["n_q"], p["n_p"], p["dnum"], p["seed"])
        N = ctx.N
        for k, r in enumerate(amounts):
            ctx.add_galois_key(r, 300 + k)
        q = p["primes"][:LEVEL]
        r = S.hashed_residues(S.config_seed(3), 1, q, 32 * 2 * N, device="cuda")
        ct = r.view(LEVEL, 32, 2, N).permute(1, 2, 0, 3).contiguous()
        out = torch.empty_like(ct)
        del r

        def step():
            for k in range(16):
                ctx.rotate(ct, out, 32, LEVEL, 300 + k)

        for _ in range(max(3, args.warmup)):
            step()
        ctx.profile_enable(fesc.Context.PROFILE_FAMILIES, 60000)
        step()
        fam = ctx.profile_read()
        ctx.profile_enable([])
        c0 = ctx.counters()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for _ in range(args.steps):
            step()
        e1.record()
        ctx.sync()
        c1 = ctx.counters()
        ms = e0.elapsed_time(e1) / args.steps
        beta, rows = ctx.num_digits, LEVEL + ctx.n_p
        launches = fam["inner"][1]
        evk_bytes = launches * beta * 2 * rows * N * 8                      # key words streamed by the inner products
        inner_bytes = 512 * (beta + 2) * rows * N * 8 + evk_bytes
        res[name] = {"digits": beta, "ms_per_step": ms, "rotations_per_s": 512 / (ms * 1e-3),
                     "limb_transforms_per_s": (c1[0] - c0[0]) / args.steps / (ms * 1e-3),
                     "evk_gbs_in_inner_product": evk_bytes / (fam["inner"][0] * 1e-3) / 1e9,
                     "inner_product_gbs": inner_bytes / (fam["inner"][0] * 1e-3) / 1e9,
                     "inner_product_frac_of_hbm_peak": inner_bytes / (fam["inner"][0] * 1e-3) / 1e9 / hbm_peak,
                     "family_ms": {k: round(v[0], 2) for k, v in fam.items() if v[1]}}
        del ctx, ct, out
        torch.cuda.empty_cache()
    g = res["full"]
    print(json.dumps({"metric": "plain rotations (automorphism + hybrid key switch) per second", "value": g["rotations_per_s"],
                      "unit": "key-switches/s", "n_gpus": 1, "steps": args.steps, "warmup": max(3, args.warmup),
                      "ms_per_step": g["ms_per_step"], "higher_is_better": True, "dtype": "u64", "data": "synthetic",
                      "config": {"workload": "rotations: 32 ciphertexts x 16 keys = 512 rotations, N=2^16, 24 limbs + 4 special"},
                      "layouts": res}), flush=True)


def run_conv(args, ctx=None, quiet=False):
    """Times fesc_conv on synthetic residues of the Mamba-2-base shape: the xBC channels (1536 + 2*128 = 1792 = 7
    channel blocks of 256) x 2048 tokens (16 token blocks of 128), d_conv = 4, 24 limbs."""
    import torch
    import fesc_synth as S
    import paper_2608_17442_b200 as fesc

    p = S.params("full")
    if ctx is None:
        torch.cuda.set_device(0)
        ctx = fesc.Context(p["log_n"], p["primes"], p["n_q"], p["n_p"], p["dnum"], p["seed"])
    N = ctx.N
    d_conv, T, blocks, tbs, level, base = 4, T_SEG, 7, 16, LEVEL, 3000
    for r in range(1, d_conv):
        ctx.add_galois_key(-r, base + r)
        ctx.add_galois_key(T - r, base + d_conv + r)
    seed = S.config_seed(5)
    q = p["primes"][:level]
    r = S.hashed_residues(seed, 21, q, tbs * blocks * 2 * N, device="cuda")
    ct = r.view(level, tbs, blocks, 2, N).permute(1, 2, 3, 0, 4).contiguous()
    r = S.hashed_residues(seed, 22, q, blocks * (2 * d_conv - 1) * N, device="cuda")
    masks = r.view(level, blocks, 2 * d_conv - 1, N).permute(1, 2, 0, 3).contiguous()
    r = S.hashed_residues(seed, 23, q, blocks * N, device="cuda")
    bias = r.view(level, blocks, N).permute(1, 0, 2).contiguous()
    del r
    out = torch.empty((tbs, blocks, 2, level - 1, N), dtype=torch.int64, device="cuda")
    desc = fesc.ConvDesc(d_conv, T, blocks, tbs, level, base)
    for _ in range(max(3, args.warmup)):
        ctx.conv(ct, masks, bias, desc, out)
    ctx.profile_enable(fesc.Context.PROFILE_FAMILIES, 60000)
    ctx.conv(ct, masks, bias, desc, out)
    fam = ctx.profile_read()
    ctx.profile_enable([])
    c0 = ctx.counters()
    sampler = ClockSampler(torch.cuda.current_device())
    sampler.start()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(args.steps):
        ctx.conv(ct, masks, bias, desc, out)
    e1.record()
    ctx.sync()
    clocks = sampler.stop()
    c1 = ctx.counters()
    ms = e0.elapsed_time(e1) / args.steps
    ks = (c1[1] - c0[1]) // args.steps
    res = ({"metric": "causal depthwise convolution latency; key-switches/s", "value": ks / (ms * 1e-3),
                      "unit": "key-switches/s", "n_gpus": 1, "steps": args.steps, "warmup": max(3, args.warmup),
                      "ms_per_step": ms, "higher_is_better": True, "dtype": "u64", "data": "synthetic",
                      "config": {"workload": "conv: 1792 channels x 2048 tokens, d_conv=4, T=128, 7 channel blocks x 16 "
                                             "token blocks, N=2^16, 24 limbs, hoisted rotations"},
                      "key_switches_per_step": ks, "gpu_launches": (c1[4] - c0[4]) // args.steps, "clocks": clocks,
                      "kernel_breakdown": {k: {"ms": round(v[0], 2), "records": v[1]} for k, v in fam.items() if v[1]}})
    if not quiet:
        print(json.dumps(res), flush=True)
    return res


def run_norm(args, ctx=None, quiet=False):
    """Times the CKKS steps around the NeRMS protocol on synthetic residues of the Mamba-2-base shape: 1536 channels
    (6 channel blocks of 256) x 2048 tokens (16 token blocks of 128), 24 limbs: fesc_norm_square on the 96
    ciphertexts, then fesc_norm_scale (8 rotate-and-add steps per token block, 96 ciphertext products, 96 plaintext
    products, two rescales)."""
    import torch
    import fesc_synth as S
    import paper_2608_17442_b200 as fesc

    p = S.params("full")
    if ctx is None:
        torch.cuda.set_device(0)
        ctx = fesc.Context(p["log_n"], p["primes"], p["n_q"], p["n_p"], p["dnum"], p["seed"])
    N = ctx.N
    T, blocks, tbs, level, base = T_SEG, 6, 16, LEVEL, 3500
    steps_fill = (N // 2 // T).bit_length() - 1
    for b in range(steps_fill):
        ctx.add_galois_key(-(T << b), base + b)
    seed = S.config_seed(5)
    q = p["primes"][:level]
    r = S.hashed_residues(seed, 31, q, tbs * blocks * 2 * N, device="cuda")
    y = r.view(level, tbs, blocks, 2, N).permute(1, 2, 3, 0, 4).contiguous()
    r = S.hashed_residues(seed, 32, q, tbs * 2 * N, device="cuda")
    sfac = r.view(level, tbs, 2, N).permute(1, 2, 0, 3).contiguous()
    r = S.hashed_residues(seed, 33, q[:level - 1], blocks * N, device="cuda")
    gamma = r.view(level - 1, blocks, N).permute(1, 0, 2).contiguous()
    del r
    u = torch.empty((tbs * blocks, 2, level - 1, N), dtype=torch.int64, device="cuda")
    out = torch.empty((tbs, blocks, 2, level - 2, N), dtype=torch.int64, device="cuda")
    desc = fesc.NormDesc(T, blocks, tbs, level, base)

    def step():
        ctx.norm_square(y, u, tbs * blocks, level)
        ctx.norm_scale(y, sfac, gamma, desc, out)

    for _ in range(max(3, args.warmup)):
        step()
    ctx.profile_enable(fesc.Context.PROFILE_FAMILIES, 60000)
    step()
    fam = ctx.profile_read()
    ctx.profile_enable([])
    c0 = ctx.counters()
    sampler = ClockSampler(torch.cuda.current_device())
    sampler.start()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(args.steps):
        step()
    e1.record()
    ctx.sync()
    clocks = sampler.stop()
    c1 = ctx.counters()
    ms = e0.elapsed_time(e1) / args.steps
    ks = (c1[1] - c0[1]) // args.steps
    res = ({"metric": "NeRMS-side CKKS steps latency; key-switches/s", "value": ks / (ms * 1e-3),
                      "unit": "key-switches/s", "n_gpus": 1, "steps": args.steps, "warmup": max(3, args.warmup),
                      "ms_per_step": ms, "higher_is_better": True, "dtype": "u64", "data": "synthetic",
                      "config": {"workload": "norm: squares and gamma (.) (y (.) br(s)) for 1536 channels x 2048 tokens, "
                                             "T=128, 6 channel blocks x 16 token blocks, N=2^16, 24 limbs"},
                      "key_switches_per_step": ks, "gpu_launches": (c1[4] - c0[4]) // args.steps, "clocks": clocks,
                      "kernel_breakdown": {k: {"ms": round(v[0], 2), "records": v[1]} for k, v in fam.items() if v[1]}})
    if not quiet:
        print(json.dumps(res), flush=True)
    return res


def run_stages(args, ctx, dev):
    """The other CKKS stages of one Mamba-2-base layer at L = 2048 (workload 5), timed one after the other on the same
    context after the headline's buffers have been released: out_proj 1536 -> 768 (its own packed diagonals), the causal
    depthwise convolution, the products around the normalisation, and a slice of the scan-contract (4 heads x 512
    tokens of the deployed geometry; the whole layer takes about a minute and runs with --workload scan_layer or
    --scan-layer 1).  Each stage: CUDA-event time, key switches, clocks sampled during its timed region, family times."""
    import argparse as _ap
    import torch

    global D_IN, D_OUT, PROJ, N1, N2
    stages = {}
    sub = _ap.Namespace(**vars(args))
    sub.steps, sub.warmup = 3, 3

    def keep(res, extra=None):
        out = {"ms": res["ms_per_step"], "key_switches": res.get("key_switches_per_step", res.get("key_switches")),
               "key_switches_per_s": res["value"], "gpu_launches": res.get("gpu_launches"), "clocks": res.get("clocks"),
               "kernel_breakdown": res.get("kernel_breakdown"), "workload": res["config"]["workload"]}
        out.update(extra or {})
        return out

    # out_proj: 6 input blocks x 3 output blocks, 16 x 16 baby / giant split
    saved = (D_IN, D_OUT, PROJ, N1, N2)
    D_IN, D_OUT, PROJ, N1, N2 = 1536, 768, "out_proj", 16, 16
    try:
        stages["out_proj"] = measure_projection(sub, ctx, dev, rank=0, world=1, key_base=(BABY_BASE + 2000, GIANT_BASE + 2000))
    finally:
        D_IN, D_OUT, PROJ, N1, N2 = saved
    torch.cuda.empty_cache()
    ctx.trim()
    # in_proj once more in the token-major packing (slot r*C + c): feature shifts are intra-segment shifts (two
    # rotations each: 63 baby and 15 giant amounts), the diagonals are periodic and their packed image is 128 times
    # smaller per diagonal, so that the weights of a whole model fit beside the activations
    global DIAG_SHIFT, KEY_AMOUNTS
    saved = (D_IN, D_OUT, PROJ, N1, N2)
    n1t, n2t = 32, 8
    KEY_AMOUNTS = ([0] + [a for q in range(1, n1t) for a in (q, q - C_SEG)],
                   [0] + [a for pp in range(1, n2t) for a in (pp * n1t, pp * n1t - C_SEG)])
    PROJ, N1, N2, DIAG_SHIFT = "in_proj (token-major packing, periodic diagonals)", 2 * n1t - 1, 2 * n2t - 1, 7
    os.environ["FESC_BSGS_GROUP_GIB"] = "64"      # 189 terms x 210 accumulators per token block: groups of 4 need 55 GiB of scratch
    try:
        stages["in_proj_token_major"] = measure_projection(sub, ctx, dev, rank=0, world=1,
                                                           key_base=(BABY_BASE + 4000, GIANT_BASE + 4000))
        stages["in_proj_token_major"]["note"] = ("same 768 -> 3352 job; packed diagonals %.2f GiB instead of 110.25 GiB"
                                                 % stages["in_proj_token_major"]["diagonals_gib"])
    finally:
        D_IN, D_OUT, PROJ, N1, N2 = saved
        DIAG_SHIFT, KEY_AMOUNTS = 0, None
        os.environ.pop("FESC_BSGS_GROUP_GIB", None)
    torch.cuda.empty_cache()
    ctx.trim()
    stages["conv"] = keep(run_conv(sub, ctx, quiet=True))
    torch.cuda.empty_cache()
    stages["norm"] = keep(run_norm(sub, ctx, quiet=True))
    torch.cuda.empty_cache()
    ctx.trim()
    sub.workload = "scan_layer" if args.scan_layer else "scan_slice"
    r = run_scan(sub, ctx, quiet=True)
    stages[sub.workload] = keep(r, {"scratch_gib": r["scratch_gib"], "limb_transforms": r["limb_transforms"]})
    return stages


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=3)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--scale-down", dest="scale_down", type=int, default=1, help=argparse.SUPPRESS)
    ap.add_argument("--no-cpu", dest="no_cpu", action="store_true", help="skip the CPU baseline leg")
    ap.add_argument("--profile-case", dest="profile_case", action="store_true",
                    help="run ONE step of a small case (96 terms, 32 (b,p) outputs, 4 token blocks, 4 limbs) and exit; for ncu")
    ap.add_argument("--profile-step", dest="profile_step", action="store_true",
                    help="run ONE step of the full workload without warm-up and exit; for the ncu launch list")
    ap.add_argument("--defer", type=int, default=1, choices=[0, 1],
                    help="1: one division by P per output for the whole giant-step sum")
    ap.add_argument("--packed", type=int, default=1, choices=[0, 1],
                    help="1: the diagonals are packed once into byte-plane operand tiles (fesc_linear_pack_diags) and the "
                         "accumulate runs on the tensor cores; 0: residues as encoded")
    ap.add_argument("--stages", type=int, default=1, choices=[0, 1],
                    help="1: after the headline, time the other CKKS stages of a layer (out_proj, conv, norm, scan slice) "
                         "and report them under `stages`")
    ap.add_argument("--scan-layer", dest="scan_layer", type=int, default=0, choices=[0, 1],
                    help="1: the scan stage of `stages` is the whole layer (24 heads x 2048 tokens, about a minute) instead of the slice")
    ap.add_argument("--hoist", type=int, default=1, choices=[0, 1],
                    help="1: baby rotations share one decomposition per input ciphertext (fesc_rotate_hoisted)")
    ap.add_argument("--group", type=int, default=4, choices=[0, 2, 4, 8, 16],
                    help="scan workloads: tokens per group of the grouped leaf build (0: token by token)")
    ap.add_argument("--scan-limbs", dest="scan_limbs", type=int, default=24,
                    help="scan workloads: limbs of the input ciphertexts (24 = fresh; the grouped Brent-Kung schedule needs 22)")
    ap.add_argument("--stride", type=int, default=256, choices=[128, 256],
                    help="scan workloads: slots per channel of a state ciphertext; 256 (the paper's deployed shape: half of "
                         "the slots idle, 12 chunks) or 128 (every slot used, 6 chunks, two token segments per block)")
    ap.add_argument("--plain", type=int, default=0, choices=[0, 1],
                    help="scan workloads: 1 = the invariant-family mode (plaintext decay, input and output factors; S4D / S5 / LRU)")
    ap.add_argument("--network", default="bk", choices=["bk", "ks", "sk"],
                    help="scan workloads: prefix network (Brent-Kung, Kogge-Stone, Sklansky)")
    ap.add_argument("--workload", default="in_proj", choices=["in_proj", "out_proj", "rotations", "scan_slice", "scan_layer", "conv", "norm"],
                    help="in_proj (default, the benchmark metric), out_proj (1536 -> 768), a scan-contract run, the "
                         "depthwise convolution or the CKKS steps around the normalisation")
    args = ap.parse_args()
    if args.workload == "out_proj":
        global D_IN, D_OUT, PROJ, METRIC, N1, N2
        D_IN, D_OUT, PROJ = 1536, 768, "out_proj"
        N1, N2 = 16, 16      # 6 input blocks, 3 output blocks: fewer, cheaper rotations than 32 x 8
        METRIC = "encrypted 1536->768 projection latency at L=2048; key-switches/s"
        args.workload = "in_proj"
    if args.workload == "conv":
        return run_conv(args)
    if args.workload == "norm":
        return run_norm(args)
    if args.workload == "rotations":
        return run_rotations(args)
    if args.workload != "in_proj":
        return run_scan(args)
    if args.impl == "reference":
        run_reference(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
