"""The benchmark's multi-rank protocol on CPU: two gloo ranks, max-over-ranks timing, whole-job value,
and the reference arm's rule that only rank 0 prints."""
import json
import os
import subprocess
import sys

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

WORKER = r"""
import os, sys, json
sys.path.insert(0, os.environ["HEART_ROOT"])
import torch.distributed as dist
from paper_2605_14513_b200 import replicas
rank, local, world = replicas.env_rank_world()
dist.init_process_group("gloo")
replicas.barrier()
mine = 10.0 + 5.0 * rank            # rank 1 is the slow replica
slowest = replicas.max_over_ranks(mine)
replicas.barrier()
print(json.dumps({"rank": rank, "world": world, "slowest": slowest,
                  "job": replicas.job_ms_per_layer_step(slowest, world)}), flush=True)
dist.destroy_process_group()
"""


def _torchrun(args, env_extra=None):
    env = dict(os.environ, HEART_ROOT=ROOT, MASTER_ADDR="127.0.0.1")
    env.update(env_extra or {})
    return subprocess.run([sys.executable, "-m", "torch.distributed.run", "--nnodes=1", "--nproc-per-node=2",
                           "--master-addr", "127.0.0.1", "--master-port", "29731"] + args,
                          capture_output=True, text=True, env=env, cwd=ROOT, timeout=300)


def test_max_over_ranks_and_job_value(tmp_path):
    script = tmp_path / "worker.py"
    script.write_text(WORKER)
    out = _torchrun([str(script)])
    assert out.returncode == 0, out.stderr[-2000:]
    import re

    lines = [json.loads(m) for m in re.findall(r"\{[^{}]*\}", out.stdout)]  # ranks may share a line
    assert sorted(l["rank"] for l in lines) == [0, 1]
    for l in lines:
        assert l["world"] == 2 and l["slowest"] == 15.0 and l["job"] == 7.5


def test_single_process_needs_no_process_group():
    sys.path.insert(0, ROOT)
    from paper_2605_14513_b200 import replicas

    assert replicas.max_over_ranks(3.25) == 3.25
    assert replicas.job_ms_per_layer_step(8.0, 1) == 8.0
    replicas.barrier()


def test_reference_arm_prints_on_rank0_only():
    out = _torchrun(["bench.py", "--impl", "reference", "--gpus", "2", "--steps", "1", "--warmup", "1",
                     "--workload", "tiny", "--cpu-sample-rows", "4"])
    assert out.returncode == 0, out.stderr[-2000:]
    lines = [json.loads(l) for l in out.stdout.splitlines() if l.startswith("{")]
    assert len(lines) == 1 and lines[0]["impl"] == "reference" and lines[0]["n_gpus"] == 2
    assert lines[0]["cpu_baseline"]["kind"] == "oracle" and lines[0]["e2e"]["h2d_bytes_per_step"] == 0


def test_gpu_count_must_match_the_ranks_that_were_started():
    """`--gpus N` inside a launch of another size is an error, not a silent single-replica run."""
    env = dict(os.environ, WORLD_SIZE="1", RANK="0", LOCAL_RANK="0")
    out = subprocess.run([sys.executable, "bench.py", "--gpus", "2", "--workload", "tiny"], capture_output=True,
                         text=True, env=env, cwd=ROOT, timeout=120)
    assert out.returncode == 2 and "WORLD_SIZE" in out.stderr
