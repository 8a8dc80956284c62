"""The N > 1 path of the benchmark on CPU: two `gloo` ranks.  Problems are independent, so the
multi-GPU job is N shards with no collective on the data path; what is shared is the timing
protocol (barrier, max over ranks) and the aggregate formula."""
import os
import socket
import subprocess
import sys
import textwrap

import numpy as np

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

WORKER = textwrap.dedent("""
    import os, sys, json
    sys.path.insert(0, %r)
    import numpy as np
    import torch.distributed as dist
    import bench
    from paper_2609_07306_b200 import workload as W
    rank, world = int(os.environ["RANK"]), int(os.environ["WORLD_SIZE"])
    dist.init_process_group("gloo")
    w = bench.shard_workload(W.tiny(), rank)
    q, k = W.generate(w, layers=1)
    dist.barrier()
    ms = bench.max_over_ranks(10.0 * (rank + 1), world)          # rank 1 is the slow one
    agg = bench.aggregate_rows_per_s(w.rows, w.layers, world, ms)
    print(json.dumps({"rank": rank, "seed": w.seed, "ms": ms, "agg": agg,
                      "digest": float(np.abs(q).sum())}))
    dist.barrier()
    dist.destroy_process_group()
""") % ROOT


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def test_two_gloo_ranks_shard_and_time():
    port = _free_port()
    procs = []
    for rank in range(2):
        env = dict(os.environ, RANK=str(rank), WORLD_SIZE="2", LOCAL_RANK=str(rank),
                   MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
        procs.append(subprocess.Popen([sys.executable, "-c", WORKER], env=env,
                                      stdout=subprocess.PIPE, stderr=subprocess.PIPE, text=True))
    outs = []
    for p in procs:
        out, err = p.communicate(timeout=120)
        assert p.returncode == 0, err[-2000:]
        outs.append(__import__("json").loads(out.strip().splitlines()[-1]))
    a, b = sorted(outs, key=lambda o: o["rank"])
    assert a["seed"] != b["seed"] and a["digest"] != b["digest"]      # different problems
    assert a["ms"] == b["ms"] == 20.0                                 # max over ranks
    rows, layers = 128, 4
    assert np.isclose(a["agg"], rows * layers * 2 / 20e-3) and a["agg"] == b["agg"]


def test_reference_arm_only_rank0_prints():
    env = dict(os.environ, RANK="1", WORLD_SIZE="2")
    out = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference",
                          "--steps", "1", "--warmup", "0", "--workload", "tiny"],
                         env=env, capture_output=True, text=True, timeout=120)
    assert out.returncode == 0 and out.stdout.strip() == ""
    env["RANK"] = "0"
    out = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference",
                          "--steps", "1", "--warmup", "0", "--workload", "tiny"],
                         env=env, capture_output=True, text=True, timeout=120)
    line = __import__("json").loads(out.stdout.strip().splitlines()[-1])
    assert line["impl"] == "reference" and line["cpu_baseline"]["kind"] == "oracle"
    assert line["e2e"]["h2d_bytes_per_step"] == 0 and line["value"] > 0
