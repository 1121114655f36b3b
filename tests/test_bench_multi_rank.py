"""The benchmark's multi-rank logic on CPU: two gloo ranks for the replica aggregation
(max of the per-rank times, sum of the replicas' work), and the reference arm under a
two-rank launch (rank 0 alone runs and prints, the other rank exits 0 silently)."""
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


def _json_lines(text):
    return [json.loads(l) for l in text.splitlines() if l.startswith("{")]


def test_replica_aggregation_two_gloo_ranks():
    r = _torchrun([os.path.join("tests", "dist_worker.py")])
    assert r.returncode == 0, r.stderr[-2000:]
    (out,) = _json_lines(r.stdout)
    assert out["world"] == 2
    assert out["worst_ms"] == 15.0                       # the slower rank decides
    # two replicas of 2e12 operations each in 15 ms
    assert abs(out["value"] - 2 * 2.0e12 / 15e-3 / 1e12) < 1e-9


def test_reference_arm_under_two_ranks_prints_once():
    r = _torchrun(["bench.py", "--impl", "reference", "--gpus", "2", "--steps", "1", "--warmup", "0",
                   "--config", "1"])
    assert r.returncode == 0, r.stderr[-2000:]
    lines = _json_lines(r.stdout)
    assert len(lines) == 1
    line = lines[0]
    assert line["impl"] == "reference" and line["n_gpus"] == 2
    assert line["value"] > 0 and line["cpu_baseline"]["kind"] == "oracle"
    assert line["e2e"]["h2d_bytes_per_step"] == 0
