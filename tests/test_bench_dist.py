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
