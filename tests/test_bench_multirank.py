"""The N > 1 plumbing of bench.py on CPU: two gloo ranks.

The path shards by replication only (no collective carries data of the method), so what has to be
right is the barrier, the maximum over ranks of the timed duration, rank-dependent input seeds, and
that only rank 0 prints a line -- for the reference arm too, whose other ranks exit without work.
"""
import json
import os
import subprocess
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

WORKER = r"""
import os, sys, json
sys.path.insert(0, %(root)r)
import bench
env = bench.make_env("gloo")
env["barrier"]()
ms = 10.0 + 5.0 * env["rank"]                 # rank 1 is the slow one
got = env["max_over_ranks"](ms)
env["barrier"]()
print(json.dumps({"rank": env["rank"], "world": env["world"], "max_ms": got}), flush=True)
env["close"]()
"""


def _launch(code_or_args, port, n=2):
    procs = []
    for rank in range(n):
        e = dict(os.environ, RANK=str(rank), LOCAL_RANK=str(rank), WORLD_SIZE=str(n), MASTER_ADDR="127.0.0.1",
                 MASTER_PORT=str(port), OMP_NUM_THREADS="2")
        procs.append(subprocess.Popen([sys.executable] + code_or_args, env=e, stdout=subprocess.PIPE,
                                      stderr=subprocess.PIPE, text=True, cwd=ROOT))
    outs = [p.communicate(timeout=240) for p in procs]
    return [(p.returncode, o, err) for p, (o, err) in zip(procs, outs)]


def test_two_gloo_ranks_take_the_maximum_duration():
    res = _launch(["-c", WORKER % {"root": ROOT}], 29611)
    for rc, out, err in res:
        assert rc == 0, err
    lines = [json.loads(out.strip().splitlines()[-1]) for _, out, _ in res]
    assert sorted(l["rank"] for l in lines) == [0, 1]
    assert all(l["world"] == 2 and l["max_ms"] == 15.0 for l in lines)


def test_reference_arm_prints_on_rank_zero_only():
    args = [os.path.join(ROOT, "bench.py"), "--impl", "reference", "--gpus", "2", "--steps", "1", "--warmup", "0",
            "--workload", "linear_4k", "--ref-tokens", "256"]
    res = _launch(args, 29612)
    for rc, out, err in res:
        assert rc == 0, err
    assert res[1][1].strip() == ""                       # rank 1: no work, no output
    line = json.loads(res[0][1].strip().splitlines()[-1])
    assert line["impl"] == "reference" and line["n_gpus"] == 2 and line["cpu_baseline"]["kind"] == "oracle"
    assert line["e2e"]["h2d_bytes_per_step"] == 0 and line["value"] > 0
