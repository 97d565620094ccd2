"""The multi-replica plumbing of bench.py on CPU (gloo, world size 2): the path shards as independent replicas, so
what needs covering is the rank environment, the max-over-ranks timing, the whole-job value, distinct prompts per
replica and the reference arm running on rank 0 alone."""
import json
import os
import subprocess
import sys

import numpy as np

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

WORKER = r"""
import os, sys, json
sys.path.insert(0, %r)
import torch, torch.distributed as dist
import bench
dist.init_process_group("gloo")
world, rank, local = bench.rank_env()
ms = bench.max_over_ranks(10.0 + 5.0 * rank, world, "cpu")      # rank 1 is the slow replica
prompt = bench.replica_prompt(1000, 16, rank)
with open(os.path.join(sys.argv[1], "rank" + str(rank) + ".json"), "w") as fh:
    json.dump({"rank": rank, "world": world, "local": local, "ms": ms,
               "value": bench.whole_job_value(world, 2, 64, ms), "prompt": prompt.tolist()}, fh)
dist.barrier()
dist.destroy_process_group()
""" % ROOT


def _torchrun(args, port):
    env = dict(os.environ, OMP_NUM_THREADS="1")
    return subprocess.run([sys.executable, "-m", "torch.distributed.run", "--nnodes=1", "--nproc-per-node", "2",
                           "--master-addr", "127.0.0.1", "--master-port", str(port)] + args,
                          capture_output=True, text=True, timeout=240, env=env, cwd=ROOT)


def test_two_replicas_take_the_slowest_time_and_add_their_tokens(tmp_path):
    script = tmp_path / "worker.py"
    script.write_text(WORKER)
    r = _torchrun([str(script), str(tmp_path)], 29611)
    assert r.returncode == 0, r.stderr[-2000:]
    lines = [json.load(open(tmp_path / ("rank%d.json" % k))) for k in (0, 1)]
    assert sorted(l["rank"] for l in lines) == [0, 1]
    for l in lines:
        assert l["world"] == 2 and l["local"] == l["rank"]
        assert l["ms"] == 15.0                                   # the max over ranks, on every rank
        assert abs(l["value"] - 2 * 2 * 64 / 15e-3) < 1e-6       # tokens of both replicas over the slowest time
    assert lines[0]["prompt"] != lines[1]["prompt"]              # every replica decodes its own sequence


def test_single_process_needs_no_process_group():
    sys.path.insert(0, ROOT)
    import bench
    assert bench.max_over_ranks(3.5, 1, "cpu") == 3.5
    assert bench.whole_job_value(1, 3, 256, 1000.0) == 768.0
    assert np.array_equal(bench.replica_prompt(50, 8, 0), bench.replica_prompt(50, 8, 0))


def test_reference_arm_runs_on_rank_0_alone():
    r = _torchrun(["bench.py", "--impl", "reference", "--workload", "tiny", "--gpus", "2", "--steps", "1", "--warmup", "0"], 29612)
    assert r.returncode == 0, r.stderr[-2000:]
    lines = [json.loads(l) for l in r.stdout.splitlines() if l.startswith("{")]
    assert len(lines) == 1
    line = lines[0]
    assert line["impl"] == "reference" and line["n_gpus"] == 2 and line["cpu_baseline"]["kind"] == "oracle"
    assert line["e2e"]["h2d_bytes_per_step"] == 0 and line["value"] > 0
