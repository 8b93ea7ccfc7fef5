"""The multi-GPU benchmark runs independent replicas (the path does not shard): what the ranks share is the timing
protocol.  Two `gloo` ranks on CPU check it: barrier, maximum of the per-rank times, whole-job rate, and that the
reference arm works on rank 0 only."""
import json
import os
import socket
import subprocess
import sys

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

WORKER = r"""
import json, os, sys
sys.path.insert(0, sys.argv[1])
from paper_2605_17842_b200 import replicas
rk = replicas.ranks_from_env()
replicas.init(rk, "gloo")
replicas.barrier(rk)
ms = replicas.max_over_ranks(rk, 10.0 + 5.0 * rk.rank)          # rank 1 is the slow one
rate = replicas.whole_job_rate(rk, 4, ms)                        # 4 units per replica and step
replicas.barrier(rk)
print(json.dumps({"rank": rk.rank, "root": rk.is_root, "ms": ms, "rate": rate}), flush=True)
replicas.finish(rk)
"""


def free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def test_two_gloo_ranks_agree_on_the_slowest_time_and_the_whole_job_rate(tmp_path):
    script = tmp_path / "worker.py"
    script.write_text(WORKER)
    port = free_port()
    procs = []
    for r in range(2):
        env = dict(os.environ, RANK=str(r), WORLD_SIZE="2", LOCAL_RANK=str(r), MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
        procs.append(subprocess.Popen([sys.executable, str(script), ROOT], env=env, stdout=subprocess.PIPE, stderr=subprocess.PIPE, text=True))
    outs = []
    for p in procs:
        out, err = p.communicate(timeout=120)
        assert p.returncode == 0, err
        outs.append(json.loads(out.strip().splitlines()[-1]))
    outs.sort(key=lambda o: o["rank"])
    assert [o["root"] for o in outs] == [True, False]
    for o in outs:
        assert o["ms"] == 15.0                       # the maximum over the ranks, on every rank
        assert abs(o["rate"] - 2 * 4 * 1e3 / 15.0) < 1e-9


def test_single_process_needs_no_group():
    sys.path.insert(0, ROOT)
    from paper_2605_17842_b200 import replicas
    rk = replicas.ranks_from_env({})
    assert (rk.rank, rk.world, rk.local, rk.is_root) == (0, 1, 0, True)
    replicas.init(rk, "gloo")
    replicas.barrier(rk)
    assert replicas.max_over_ranks(rk, 3.5) == 3.5
    assert replicas.whole_job_rate(rk, 8, 2.0) == 4000.0
    replicas.finish(rk)


def test_reference_arm_does_nothing_on_other_ranks():
    env = dict(os.environ, RANK="1", WORLD_SIZE="2", LOCAL_RANK="1")
    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--gpus", "2", "--steps", "1", "--warmup", "1"],
                       env=env, capture_output=True, text=True, timeout=120)
    assert r.returncode == 0, r.stderr
    assert r.stdout.strip() == ""
