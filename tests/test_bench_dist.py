"""The N > 1 path of bench.py on CPU: two gloo ranks run the barrier / max-over-ranks plumbing the GPU
benchmark uses (ranks are independent replicas; there is no data-path collective), and the reference arm
prints only on rank 0."""
import json
import os
import socket
import subprocess
import sys

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

WORKER = r"""
import os, sys, json
sys.path.insert(0, %r)
import bench
rank, world = bench.dist_setup("gloo")
bench.barrier()
local_ms = 10.0 + 5.0 * rank
agg = bench.max_over_ranks(local_ms)
gin, nout, tbs = bench.workload_dims()
ks = bench.key_switches_per_step(gin, nout, tbs)
value = world * ks / (agg * 1e-3)
bench.barrier()
print(json.dumps({"rank": rank, "world": world, "agg": agg, "value": value, "ks": ks}))
"""


def _free_port():
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    p = s.getsockname()[1]
    s.close()
    return p


def test_two_gloo_ranks_take_max_time_and_sum_work():
    port = _free_port()
    procs = []
    for r in range(2):
        env = dict(os.environ, RANK=str(r), LOCAL_RANK=str(r), WORLD_SIZE="2", MASTER_ADDR="127.0.0.1",
                   MASTER_PORT=str(port))
        procs.append(subprocess.Popen([sys.executable, "-c", WORKER % ROOT], env=env, stdout=subprocess.PIPE,
                                      stderr=subprocess.PIPE, text=True))
    outs = []
    for p in procs:
        o, e = p.communicate(timeout=120)
        assert p.returncode == 0, e
        outs.append(json.loads(o.strip().splitlines()[-1]))
    assert {o["rank"] for o in outs} == {0, 1}
    for o in outs:
        assert o["world"] == 2 and o["agg"] == 15.0          # max over ranks of (10, 15) ms
        assert o["ks"] == 3056                                 # 16 * (3*31 + 14*7) key switches per projection
        assert abs(o["value"] - 2 * 3056 / 0.015) < 1e-6      # whole-job rate = work of both ranks / max time


def test_workload_counts():
    sys.path.insert(0, ROOT)
    import bench

    gin, nout, tbs = bench.workload_dims()
    assert (gin, nout, tbs) == (3, 14, 16)
    assert tbs * gin == 48 and nout * bench.N2 * gin * bench.N1 == 10752 and tbs * nout == 224
    assert tbs * nout * bench.N2 * gin * bench.N1 == 172032
    assert tbs * gin * (bench.N1 - 1) == 1488 and tbs * nout * (bench.N2 - 1) == 1568


def test_scan_partition_keeps_chunk_pairs_together():
    sys.path.insert(0, ROOT)
    import bench

    for K_s in (12, 11, 2, 1):
        for world in (1, 2, 3, 4, 6, 8):
            parts = bench.scan_partition(K_s, world)
            assert len(parts) == world
            covered = []
            for first, count in parts:
                assert first % 2 == 0                              # a rank starts on a pair boundary
                covered += list(range(first, first + count))
            assert covered == list(range(K_s))                     # every chunk exactly once, in order
            sizes = [-(-c // 2) for _, c in parts]
            assert max(sizes) - min(sizes) <= 1                    # pairs are balanced to within one
    assert [c for _, c in bench.scan_partition(12, 4)] == [2, 4, 2, 4]
    assert [c for _, c in bench.scan_partition(12, 3)] == [4, 4, 4]


GATHER_WORKER = r"""
import os, sys, json
sys.path.insert(0, %r)
import torch, bench
rank, world = bench.dist_setup("gloo")
K_blk, K_s = 2, 5
parts = bench.scan_partition(K_s, world)
first, mine = parts[rank]
local = torch.empty((K_blk, mine, 3), dtype=torch.int64)
for j in range(K_blk):
    for c in range(mine):
        local[j, c] = 100 * j + (first + c)
full = bench.gather_chunk_outputs(local, parts, rank, world, K_blk, K_s)
want = torch.tensor([[[100 * j + c] * 3 for c in range(K_s)] for j in range(K_blk)])
print(json.dumps({"rank": rank, "ok": bool((full == want).all()), "parts": parts}))
"""


def test_two_gloo_ranks_gather_their_chunk_outputs_once():
    port = _free_port()
    procs = []
    for r in range(2):
        env = dict(os.environ, RANK=str(r), LOCAL_RANK=str(r), WORLD_SIZE="2", MASTER_ADDR="127.0.0.1",
                   MASTER_PORT=str(port))
        procs.append(subprocess.Popen([sys.executable, "-c", GATHER_WORKER % ROOT], env=env, stdout=subprocess.PIPE,
                                      stderr=subprocess.PIPE, text=True))
    for p in procs:
        o, e = p.communicate(timeout=120)
        assert p.returncode == 0, e
        res = json.loads(o.strip().splitlines()[-1])
        assert res["ok"] and res["parts"] == [[0, 2], [2, 3]]      # 5 chunks: pair (0,1) | pair (2,3) and the odd chunk 4


def test_bench_scan_rotation_amounts_match_the_dataflow():
    """bench.py registers Galois keys from its own list of rotation amounts (the product path does not import the
    oracle); the list equals the one the scan dataflow uses, in every mode."""
    import bench
    from oracle.scan import ScanShape

    for n, kw in ((128, dict(L=40, H=8, P=4, d_s=8, B_blk=16)), (32768, dict(L=2048, H=24, P=64, d_s=128, B_blk=256)),
                  (128, dict(L=40, H=8, P=4, d_s=8, B_blk=16, stride=8)),
                  (32768, dict(L=2048, H=24, P=64, d_s=128, B_blk=256, stride=128))):
        sh = ScanShape(n, **kw)
        for hoist in (False, True):
            for group in (0, 2, 4, 8):
                want = sh.rotation_amounts(hoist, group)
                assert bench.scan_rotation_amounts(n, sh.P, sh.d_s, sh.B, sh.stride, hoist, group) == want
