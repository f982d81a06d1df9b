"""The N > 1 launch path on CPU: world_size-2 gloo processes exercise the rank plumbing the benchmark
uses (rank / world from the environment, barrier, max over ranks) and the reference arm's rule that
only rank 0 prints."""
import json
import os
import socket
import subprocess
import sys

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def run_two_ranks(script_args, timeout=300):
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", "--nproc-per-node", "2",
           "--master-addr", "127.0.0.1", "--master-port", str(free_port())] + script_args
    env = dict(os.environ, CUDA_VISIBLE_DEVICES="", OMP_NUM_THREADS="2")
    return subprocess.run(cmd, cwd=ROOT, env=env, capture_output=True, text=True, timeout=timeout)


def test_max_over_ranks_and_barrier_with_gloo(tmp_path):
    script = tmp_path / "ranks.py"
    script.write_text(
        "import sys, torch, torch.distributed as dist\n"
        f"sys.path.insert(0, {ROOT!r})\n"
        "import bench\n"
        "rank, world, local = bench.dist_env()\n"
        "dist.init_process_group('gloo')\n"
        "bench.barrier(world)\n"
        "m = bench.max_over_ranks(10.0 + rank, world, 'cpu')\n"
        "assert world == 2 and m == 11.0, (world, m)\n"
        "bench.barrier(world)\n"
        "print(f'rank {rank} ok {m}')\n"
        "dist.destroy_process_group()\n")
    r = run_two_ranks([str(script)])
    assert r.returncode == 0, r.stderr[-2000:]
    assert "rank 0 ok 11.0" in r.stdout and "rank 1 ok 11.0" in r.stdout


def test_reference_arm_prints_once_under_two_ranks():
    r = run_two_ranks(["bench.py", "--impl", "reference", "--gpus", "2", "--steps", "1", "--warmup", "0",
                       "--cpu-seconds", "1"])
    assert r.returncode == 0, r.stderr[-2000:]
    lines = [l for l in r.stdout.splitlines() if l.startswith("{")]
    assert len(lines) == 1
    j = json.loads(lines[0])
    assert j["impl"] == "reference" and j["n_gpus"] == 2 and j["value"] > 0 and j["cpu_baseline"]["kind"] == "oracle"
    assert j["e2e"]["h2d_bytes_per_step"] == 0 and j["gpu_launches"] == 0
