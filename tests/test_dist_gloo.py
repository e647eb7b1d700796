"""World-size-2 gloo runs on CPU: the replicas path of the benchmark (rendezvous, barrier, max-over-ranks timing,
one sequence per rank) and the reference arm under torchrun (rank 0 prints the line, the other rank exits 0)."""
import json
import os
import subprocess
import sys

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _torchrun(args, port, timeout=600):
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", "--nproc-per-node", "2", "--master-addr", "127.0.0.1",
           "--master-port", str(port)] + args
    env = dict(os.environ, CUDA_VISIBLE_DEVICES="", OMP_NUM_THREADS="2")
    return subprocess.run(cmd, cwd=ROOT, env=env, capture_output=True, text=True, timeout=timeout)


def test_two_rank_host_logic(tmp_path):
    r = _torchrun([os.path.join(ROOT, "tests", "dist_worker.py"), str(tmp_path)], 29517)
    assert r.returncode == 0, r.stderr[-2000:]
    assert (tmp_path / "ok.0").exists() and (tmp_path / "ok.1").exists()


def test_reference_arm_under_torchrun_prints_one_line():
    r = _torchrun([os.path.join(ROOT, "bench.py"), "--impl", "reference", "--workload", "tiny", "--gpus", "2", "--steps", "3",
                   "--warmup", "3"], 29519)
    assert r.returncode == 0, r.stderr[-2000:]
    lines = [l for l in r.stdout.splitlines() if l.startswith("{")]
    assert len(lines) == 1
    d = json.loads(lines[0])
    assert d["impl"] == "reference" and d["cpu_baseline"]["kind"] == "oracle" and d["value"] > 0
    assert d["e2e"]["h2d_bytes_per_step"] == 0
