"""The multi-rank plumbing of bench.py on CPU (gloo, world size 2): ranks are independent
replicas, the reported time is the maximum over ranks, and only rank 0 of the reference arm
prints a line."""
import json
import os
import subprocess
import sys
import textwrap

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

WORKER = textwrap.dedent("""
    import os, sys
    sys.path.insert(0, %r)
    import bench
    rank, world, local, dist = bench.init_distributed(2)
    assert world == 2 and dist is not None
    dist.barrier()
    slowest = bench.max_over_ranks(dist, 10.0 + 5.0 * rank, "cpu")
    assert slowest == 15.0, slowest
    dist.barrier()
    dist.destroy_process_group()
    print("rank %%d ok" %% rank)
""") % ROOT


def test_max_over_ranks_with_gloo(tmp_path):
    script = tmp_path / "worker.py"
    script.write_text(WORKER)
    env = dict(os.environ, CUDA_VISIBLE_DEVICES="", MASTER_ADDR="127.0.0.1")
    out = subprocess.run([sys.executable, "-m", "torch.distributed.run", "--nnodes=1", "--nproc-per-node=2",
                          "--master-addr", "127.0.0.1", "--master-port", "29531", str(script)],
                         capture_output=True, text=True, env=env, timeout=240)
    assert out.returncode == 0, out.stderr[-2000:]
    assert "rank 0 ok" in out.stdout and "rank 1 ok" in out.stdout


def test_reference_arm_prints_on_rank_zero_only():
    base = [sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--gpus", "2", "--steps", "1",
            "--warmup", "1", "--workload", "cfg1"]
    out0 = subprocess.run(base, capture_output=True, text=True, env=dict(os.environ, RANK="0", WORLD_SIZE="2"), timeout=240)
    out1 = subprocess.run(base, capture_output=True, text=True, env=dict(os.environ, RANK="1", WORLD_SIZE="2"), timeout=240)
    assert out0.returncode == 0 and out1.returncode == 0, out0.stderr + out1.stderr
    line = json.loads(out0.stdout.strip().splitlines()[-1])
    assert line["impl"] == "reference" and line["unit"] == "GB/s" and line["vs_baseline"] is None
    assert line["cpu_baseline"]["kind"] == "oracle" and line["e2e"]["h2d_bytes_per_step"] == 0
    assert out1.stdout.strip() == ""
