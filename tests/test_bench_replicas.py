"""The path has no exchange step, so `bench.py --gpus N` runs N independent replicas.  These CPU
tests cover the multi-process host logic with two gloo ranks: rendezvous, barrier, max over ranks,
and the reference arm, where rank 0 alone works and prints."""
import json
import os
import socket
import subprocess
import sys

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _torchrun(script_args, timeout=300):
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", "--nproc-per-node", "2",
           "--master-addr", "127.0.0.1", "--master-port", str(_free_port())] + script_args
    env = dict(os.environ, OMP_NUM_THREADS="2")
    return subprocess.run(cmd, cwd=ROOT, env=env, capture_output=True, text=True, timeout=timeout)


def test_two_gloo_ranks_barrier_and_max_over_ranks():
    r = _torchrun([os.path.join(ROOT, "tests", "replica_worker.py")])
    assert r.returncode == 0, r.stderr[-2000:]
    lines = [l for l in r.stdout.splitlines() if l.startswith("{")]
    assert len(lines) == 1                       # rank 0 only
    out = json.loads(lines[0])
    assert out["world"] == 2 and out["worst_ms"] == 15.0      # the slower replica's time
    assert abs(out["value"] - 2 * 3.0 / 15.0e-3) < 1e-9        # both replicas' work / that time


def test_reference_arm_under_torchrun_prints_once():
    r = _torchrun([os.path.join(ROOT, "bench.py"), "--impl", "reference", "--gpus", "2",
                   "--workload", "tiny", "--batch", "1", "--steps", "1", "--warmup", "0"])
    assert r.returncode == 0, r.stderr[-2000:]
    lines = [l for l in r.stdout.splitlines() if l.startswith("{")]
    assert len(lines) == 1
    out = json.loads(lines[0])
    assert out["impl"] == "reference" and out["cpu_baseline"]["kind"] == "oracle"
    assert out["e2e"]["h2d_bytes_per_step"] == 0 and out["n_gpus"] == 2
