"""The multi-rank host logic of bench.py, run as two gloo ranks on the CPU: the path has no
exchange step, so ranks are independent replicas and only the barrier and the max over ranks of
the device time use torch.distributed."""
import json
import os
import subprocess
import sys

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

RANK_SCRIPT = r"""
import json, os, sys
sys.path.insert(0, {root!r})
import bench
from paper_2405_18832_b200 import synthetic as S
dist, rank, world, local = bench.dist_setup("gloo")
w = bench.replica_workload(S.config("C0"), rank, world)
dist.barrier()
slowest = bench.max_over_ranks(dist, 1.0 + rank)          # rank 1 is the slow one
value = bench.aggregate_tokens_per_s(w.problem.T, world, slowest)
g = S.generate(w, with_weights=False)
print(json.dumps(dict(rank=rank, world=world, seed=w.seed, slowest=slowest, value=value,
                      x0=float(g["x"][0, 0]))))
dist.barrier()
dist.destroy_process_group()
"""


def test_two_gloo_ranks_are_independent_replicas_timed_by_the_slowest(tmp_path):
    script = tmp_path / "rank.py"
    script.write_text(RANK_SCRIPT.format(root=ROOT))
    procs = []
    for rank in range(2):
        env = dict(os.environ, RANK=str(rank), LOCAL_RANK=str(rank), WORLD_SIZE="2",
                   MASTER_ADDR="127.0.0.1", MASTER_PORT="29541")
        procs.append(subprocess.Popen([sys.executable, str(script)], env=env, stdout=subprocess.PIPE, text=True))
    outs = [json.loads(p.communicate(timeout=120)[0].strip().splitlines()[-1]) for p in procs]
    assert all(p.returncode == 0 for p in procs)
    a, b = sorted(outs, key=lambda o: o["rank"])
    assert a["world"] == b["world"] == 2
    assert a["slowest"] == b["slowest"] == 2.0                      # max over ranks, on every rank
    assert a["value"] == b["value"] == 2 * 64 / 2.0e-3               # whole-job tokens/s
    assert a["seed"] != b["seed"] and a["x0"] != b["x0"]           # each replica has its own batch


def test_reference_arm_runs_on_rank_zero_only():
    env = dict(os.environ, RANK="1", LOCAL_RANK="1", WORLD_SIZE="2")
    out = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--gpus", "2",
                          "--steps", "1", "--warmup", "0"], env=env, capture_output=True, text=True, timeout=120)
    assert out.returncode == 0 and out.stdout.strip() == ""
