"""The multi-GPU plumbing, exercised with two gloo ranks on CPU (no collective is on the data path: ranks only
agree on the slowest rank's time)."""
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


def _torchrun(script_args, nproc=2, timeout=240):
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", f"--nproc-per-node={nproc}",
           "--master-addr", "127.0.0.1", "--master-port", str(_free_port())] + script_args
    env = dict(os.environ, PYTHONPATH=ROOT, OMP_NUM_THREADS="2")
    return subprocess.run(cmd, cwd=ROOT, env=env, capture_output=True, text=True, timeout=timeout)


def test_two_ranks_agree_on_slowest_time_and_draw_different_batches():
    r = _torchrun([os.path.join("tests", "dist_worker.py")])
    assert r.returncode == 0, r.stderr[-2000:]
    line = [l for l in r.stdout.splitlines() if l.startswith("[{")][-1]
    got = sorted(json.loads(line), key=lambda d: d["rank"])
    assert [d["rank"] for d in got] == [0, 1]
    assert all(d["slowest"] == 5.0 for d in got)                  # max(2.0, 5.0) on every rank
    assert all(abs(d["rate"] - 2 * 1000.0 / 5e-3) < 1e-6 for d in got)
    assert got[0]["cfg"] == 4 and got[1]["cfg"] == 104 and got[0]["first"] != got[1]["first"]


def test_reference_arm_prints_one_line_from_rank_0_only():
    r = _torchrun(["bench.py", "--impl", "reference", "--gpus", "2", "--steps", "1", "--warmup", "0",
                   "--reference-rows", "16"])
    assert r.returncode == 0, r.stderr[-2000:]
    lines = [l for l in r.stdout.splitlines() if l.startswith("{")]
    assert len(lines) == 1
    d = json.loads(lines[0])
    assert d["impl"] == "reference" and d["n_gpus"] == 2 and d["cpu_baseline"]["kind"] == "oracle"
    assert d["e2e"]["h2d_bytes_per_step"] == 0 and d["value"] > 0
