"""The multi-process path of the benchmark on CPU: two ranks over gloo.  The path does not shard, so
what is tested is the host plumbing ranks share: distinct seeds, the max-over-ranks time, the
aggregate throughput, and that rank 0 alone reports."""
import os
import socket
import subprocess
import sys
import textwrap

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

WORKER = textwrap.dedent("""
    import json, os, sys
    sys.path.insert(0, %r)
    import torch.distributed as dist
    from paper_2505_19115_b200 import replicas, synth
    rank, world, local = replicas.env_rank_world()
    dist.init_process_group("gloo")
    seed = replicas.replica_seed(4000, rank)
    x = synth.normal((4, 16), 1.0, seed)
    my_ms = 10.0 + 5.0 * rank                      # rank 1 is the slow one
    dist.barrier()
    ms = replicas.max_over_ranks(my_ms, dist)
    value = replicas.aggregate_throughput(1000.0, world, ms * 1e-3)
    out = {"rank": rank, "world": world, "seed": seed, "ms": ms, "value": value, "x0": float(x[0, 0])}
    if rank == 0:
        print("LINE " + json.dumps(out))
    else:
        print("OTHER " + json.dumps(out))
    dist.destroy_process_group()
""") % ROOT


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def test_two_replicas_over_gloo(tmp_path):
    import json
    script = tmp_path / "worker.py"
    script.write_text(WORKER)
    port = _free_port()
    procs = []
    for rank in range(2):
        env = dict(os.environ, RANK=str(rank), WORLD_SIZE="2", LOCAL_RANK=str(rank), MASTER_ADDR="127.0.0.1",
                   MASTER_PORT=str(port))
        procs.append(subprocess.Popen([sys.executable, str(script)], env=env, stdout=subprocess.PIPE,
                                      stderr=subprocess.PIPE, text=True))
    outs = [p.communicate(timeout=120) for p in procs]
    assert all(p.returncode == 0 for p in procs), outs
    r0 = json.loads(next(l for l in outs[0][0].splitlines() if l.startswith("LINE "))[5:])
    r1 = json.loads(next(l for l in outs[1][0].splitlines() if l.startswith("OTHER "))[6:])
    assert not any(l.startswith("LINE ") for l in outs[1][0].splitlines())       # rank 0 alone reports
    assert r0["world"] == r1["world"] == 2
    assert r0["seed"] != r1["seed"] and r0["x0"] != r1["x0"]                      # every replica has its own inputs
    assert r0["ms"] == r1["ms"] == 15.0                                           # the slowest rank's time, on both
    assert abs(r0["value"] - 1000.0 * 2 / 15e-3) < 1e-6                           # whole-job aggregate


def test_single_process_needs_no_process_group():
    from paper_2505_19115_b200 import replicas
    assert replicas.max_over_ranks(3.5) == 3.5
    assert replicas.aggregate_throughput(10.0, 1, 2.0) == 5.0
