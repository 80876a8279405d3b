"""Multi-GPU plumbing on CPU: two gloo ranks run the replica helpers the bench uses (barrier,
MAX over ranks of the elapsed time; the whole-job value is world size x units / that time) and the
reference arm's rule that only rank 0 works."""
import json
import os
import subprocess
import sys

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

WORKER = r"""
import json, os, sys
sys.path.insert(0, %r)
from paper_2608_20961_b200 import replicas
rank, size, local = replicas.init("gloo")
replicas.barrier()
ms = replicas.max_over_ranks(10.0 * (rank + 1))          # rank 1 is the slow one
units = size * 1000.0                                    # what bench.py does: replicas of one workload
replicas.barrier()
print(json.dumps({"rank": rank, "size": size, "ms": ms, "units": units}))
replicas.shutdown()
"""


def test_two_gloo_ranks_agree_on_max_time(tmp_path):
    script = tmp_path / "worker.py"
    script.write_text(WORKER % ROOT)
    env = dict(os.environ, MASTER_ADDR="127.0.0.1", MASTER_PORT="29533", WORLD_SIZE="2")
    procs = []
    for rank in range(2):
        e = dict(env, RANK=str(rank), LOCAL_RANK=str(rank))
        procs.append(subprocess.Popen([sys.executable, str(script)], env=e, stdout=subprocess.PIPE,
                                      stderr=subprocess.PIPE, text=True))
    outs = []
    for p in procs:
        out, err = p.communicate(timeout=120)
        assert p.returncode == 0, err
        outs.append(json.loads(out.strip().splitlines()[-1]))
    for o in outs:
        assert o["size"] == 2 and o["ms"] == 20.0 and o["units"] == 2000.0
    assert sorted(o["rank"] for o in outs) == [0, 1]


def test_reference_arm_runs_on_rank_zero_only():
    env = dict(os.environ, RANK="1", WORLD_SIZE="2", LOCAL_RANK="1")
    res = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference",
                          "--steps", "1", "--warmup", "0", "--ref-seqs", "1"], env=env,
                         capture_output=True, text=True, timeout=300)
    assert res.returncode == 0 and res.stdout.strip() == ""
    env = dict(os.environ, RANK="0", WORLD_SIZE="2", LOCAL_RANK="0")
    res = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference",
                          "--gpus", "2", "--steps", "1", "--warmup", "0", "--ref-seqs", "1"], env=env,
                         capture_output=True, text=True, timeout=300)
    line = json.loads(res.stdout.strip().splitlines()[-1])
    assert line["impl"] == "reference" and line["cpu_baseline"]["kind"] == "oracle"
    assert line["e2e"]["h2d_bytes_per_step"] == 0 and line["value"] > 0
