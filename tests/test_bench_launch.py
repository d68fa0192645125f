"""`bench.py --gpus N` starts its own ranks when it is not already running under a launcher (CPU, gloo, world size 2):
the rank plumbing of the benchmark -- process group, batch shards, barrier, max over ranks -- without any GPU work,
and the reference arm, where rank 0 alone works and prints."""
import json
import os
import subprocess
import sys

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _run(*flags):
    env = {k: v for k, v in os.environ.items() if k not in ("RANK", "WORLD_SIZE", "LOCAL_RANK", "MASTER_ADDR", "MASTER_PORT")}
    env["CUDA_VISIBLE_DEVICES"] = ""              # the plumbing is the same on CPU: gloo instead of NCCL
    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), *flags], capture_output=True, text=True, timeout=300, env=env)
    assert r.returncode == 0, r.stderr[-2000:]
    lines = [ln for ln in r.stdout.splitlines() if ln.startswith("{")]
    assert len(lines) == 1, r.stdout                # rank 0 prints, the others stay silent
    return json.loads(lines[0])


def test_gpus_flag_starts_that_many_ranks():
    j = _run("--gpus", "2", "--impl", "launch-check")
    assert j["n_gpus"] == 2 and j["requested"] == 2 and j["max_over_ranks"] == 2.0
    (a0, b0), (a1, b1) = j["shards"]
    assert a0 == 0 and b0 == a1 and b1 == 128       # contiguous shards that cover the job's batch
    t0, t1 = j["shard_tokens"]
    assert abs(t0 - t1) <= 0.05 * (t0 + t1)         # balanced by cached tokens, not by sequence count


def test_single_rank_needs_no_launcher():
    j = _run("--gpus", "1", "--impl", "launch-check")
    assert j["n_gpus"] == 1 and j["shards"] == [[0, 64]]


def test_reference_arm_under_two_ranks_prints_once():
    j = _run("--gpus", "2", "--impl", "reference", "--steps", "1", "--warmup", "0", "--cpu-seqs", "1", "--cpu-decode-steps", "1")
    assert j["impl"] == "reference" and j["n_gpus"] == 2 and j["gpu_launches"] == 0
    assert j["value"] > 0 and j["e2e"]["h2d_bytes_per_step"] == 0
