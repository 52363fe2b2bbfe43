"""The path on several GPUs is independent replicas (no exchange inside a step of
Algorithm 1); what the ranks share is the timing reduction.  Two `gloo` ranks on
CPU check that reduction, the per-rank input sets and the reference arm's rule
that rank 0 alone works."""
import json
import os
import socket
import subprocess
import sys

import numpy as np

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

WORKER = r"""
import json, os, sys
sys.path.insert(0, {root!r})
import numpy as np
from paper_2402_11809_b200 import replicas, workloads
rank, world, local = replicas.rank_env()
assert replicas.init("gloo") == world == 2
replicas.barrier()
# rank r pretends that its 100 steps took (r + 1) * 0.5 s
value, t = replicas.job_throughput(100, 0.5 * (rank + 1))
cfg = workloads.resolve("tiny")
x = workloads.make_step_inputs(cfg, set_index=replicas.set_index(rank, 0))
import zlib
out = dict(rank=rank, world=world, value=value, t=t, slowest=replicas.slowest(3.0 - rank),
           q_crc=zlib.crc32(x["q"].tobytes()), kv_len=[int(v) for v in x["kv_len"]])
replicas.barrier()
replicas.shutdown()
print("RESULT " + json.dumps(out), flush=True)
"""


def free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def spawn(code_or_argv, world, extra_env=None):
    port = free_port()
    procs = []
    for r in range(world):
        env = dict(os.environ, RANK=str(r), LOCAL_RANK=str(r), WORLD_SIZE=str(world),
                   MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), **(extra_env or {}))
        argv = [sys.executable, "-c", code_or_argv] if isinstance(code_or_argv, str) else code_or_argv
        procs.append(subprocess.Popen(argv, env=env, cwd=ROOT, stdout=subprocess.PIPE, stderr=subprocess.PIPE,
                                      text=True))
    outs = []
    for p in procs:
        o, e = p.communicate(timeout=240)
        outs.append((p.returncode, o, e))
    return outs


def test_two_gloo_ranks_take_the_slowest_time():
    outs = spawn(WORKER.format(root=ROOT), 2)
    res = []
    for rc, o, e in outs:
        assert rc == 0, e[-2000:]
        line = [l for l in o.splitlines() if l.startswith("RESULT ")][-1]
        res.append(json.loads(line[7:]))
    res.sort(key=lambda r: r["rank"])
    for r in res:
        # the job took the slower rank's 1.0 s; both ranks' 100 steps count
        assert r["t"] == 1.0 and r["value"] == 200.0
        assert r["slowest"] == 3.0
    # replicas work on different seeded inputs of the same shape
    assert res[0]["q_crc"] != res[1]["q_crc"]
    assert len(res[0]["kv_len"]) == len(res[1]["kv_len"])


def test_single_process_needs_no_group():
    sys.path.insert(0, ROOT)
    from paper_2402_11809_b200 import replicas
    env = {k: os.environ.pop(k) for k in ("RANK", "WORLD_SIZE", "LOCAL_RANK") if k in os.environ}
    try:
        assert replicas.rank_env() == (0, 1, 0)
        assert replicas.init("gloo") == 1
        assert replicas.job_throughput(50, 0.25) == (200.0, 0.25)
        assert replicas.set_index(3, 7) == 3007
        try:
            replicas.set_index(0, replicas.SETS_PER_RANK)
            raise AssertionError("set index past a rank's range must be refused")
        except ValueError:
            pass
    finally:
        os.environ.update(env)


def test_input_sets_differ_across_ranks_and_repeat_per_seed():
    sys.path.insert(0, ROOT)
    from paper_2402_11809_b200 import replicas, workloads
    cfg = workloads.resolve("tiny")
    a = workloads.make_step_inputs(cfg, set_index=replicas.set_index(0, 1))
    b = workloads.make_step_inputs(cfg, set_index=replicas.set_index(1, 1))
    a2 = workloads.make_step_inputs(cfg, set_index=replicas.set_index(0, 1))
    assert not np.array_equal(a["logits"], b["logits"])
    assert np.array_equal(a["logits"], a2["logits"]) and np.array_equal(a["q"], a2["q"])


def test_reference_arm_runs_on_rank_zero_only():
    argv = [sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--config", "tiny",
            "--gpus", "2", "--steps", "2", "--warmup", "1"]
    outs = spawn(argv, 2)
    (rc0, o0, e0), (rc1, o1, e1) = outs
    assert rc0 == 0, e0[-2000:]
    assert rc1 == 0, e1[-2000:]
    assert o1.strip() == ""                                # the other rank exits without work or output
    line = json.loads(o0.strip().splitlines()[-1])
    assert line["impl"] == "reference" and line["n_gpus"] == 2
    assert line["cpu_baseline"]["kind"] == "oracle" and line["value"] > 0
    assert line["e2e"]["h2d_bytes_per_step"] == 0 and line["e2e"]["d2h_bytes_per_step"] == 0


def test_projection_reference_arm_runs_on_rank_zero_only():
    argv = [sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--config", "lmhead_tiny",
            "--gpus", "2", "--steps", "2", "--warmup", "1"]
    (rc0, o0, e0), (rc1, o1, e1) = spawn(argv, 2)
    assert rc0 == 0, e0[-2000:]
    assert rc1 == 0, e1[-2000:]
    assert o1.strip() == ""
    line = json.loads(o0.strip().splitlines()[-1])
    assert line["impl"] == "reference" and line["n_gpus"] == 2 and line["config"]["workload"] == "lmhead_tiny"
    assert line["cpu_baseline"]["kind"] == "oracle" and line["value"] > 0
