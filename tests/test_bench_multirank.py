"""The benchmark's N > 1 path on CPU: two gloo ranks, barrier, max-over-ranks time and summed tokens.

The decode path does not shard (replicas only), so the only multi-rank logic is the timing reduction.
"""
import json
import os
import subprocess
import sys
import textwrap

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

WORKER = textwrap.dedent("""
    import os, sys, json
    sys.path.insert(0, %r)
    import torch
    import bench
    rank, world, local = bench.dist_setup(2)
    assert world == 2 and rank == int(os.environ["RANK"])
    bench.barrier(world)
    # rank 0 took 3.0 ms and committed 10 tokens, rank 1 took 5.0 ms and committed 12
    t, tok = bench.reduce_max_sum(world, 3.0 + 2.0 * rank, 10 + 2 * rank, torch.device("cpu"))
    bench.barrier(world)
    if rank == 0:
        print(json.dumps({"t": t, "tok": tok}))
    import torch.distributed as dist
    dist.destroy_process_group()
""") % ROOT


def test_two_gloo_ranks_reduce_max_time_and_sum_tokens(tmp_path):
    script = tmp_path / "worker.py"
    script.write_text(WORKER)
    env = dict(os.environ, CUDA_VISIBLE_DEVICES="", MASTER_ADDR="127.0.0.1")
    out = subprocess.run([sys.executable, "-m", "torch.distributed.run", "--nnodes=1", "--nproc-per-node", "2",
                          "--master-addr", "127.0.0.1", "--master-port", "29533", str(script)],
                         capture_output=True, text=True, env=env, timeout=240)
    assert out.returncode == 0, out.stderr[-2000:]
    line = [l for l in out.stdout.splitlines() if l.startswith("{")][-1]
    res = json.loads(line)
    assert res["t"] == 5.0 and res["tok"] == 22.0


def test_reference_arm_runs_on_rank0_only(tmp_path):
    """Under torchrun the reference arm prints one line from rank 0; the other rank exits 0 without work."""
    env = dict(os.environ, CUDA_VISIBLE_DEVICES="", MASTER_ADDR="127.0.0.1")
    out = subprocess.run([sys.executable, "-m", "torch.distributed.run", "--nnodes=1", "--nproc-per-node", "2",
                          "--master-addr", "127.0.0.1", "--master-port", "29534", os.path.join(ROOT, "bench.py"),
                          "--impl", "reference", "--workload", "tiny", "--gpus", "2", "--steps", "3", "--warmup", "3"],
                         capture_output=True, text=True, env=env, timeout=300)
    assert out.returncode == 0, out.stderr[-2000:]
    lines = [l for l in out.stdout.splitlines() if l.startswith("{")]
    assert len(lines) == 1
    d = json.loads(lines[0])
    assert d["impl"] == "reference" and d["cpu_baseline"]["kind"] == "oracle" and d["value"] > 0
