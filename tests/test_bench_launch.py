"""The benchmark's multi-process launch path, on CPU: `--gpus N` alone must start N replicas itself, and under an
external launcher (RANK / WORLD_SIZE already set) it must not start them twice.  The ranks run the stub step (a
sleep) over gloo; the bracketing barriers, the max-over-ranks time and the whole-job rate are the real code."""
import json
import os
import socket
import subprocess
import sys

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _clean_env():
    env = {k: v for k, v in os.environ.items()
           if k not in ("RANK", "WORLD_SIZE", "LOCAL_RANK", "MASTER_ADDR", "MASTER_PORT", "LOCAL_WORLD_SIZE", "GROUP_RANK")}
    env["CUDA_VISIBLE_DEVICES"] = ""
    return env


def _json_lines(text):
    return [json.loads(ln) for ln in text.splitlines() if ln.startswith("{")]


def test_gpus_flag_starts_the_replicas_itself():
    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--gpus", "2", "--stub-step-ms", "2", "--steps", "4",
                        "--warmup", "1"], capture_output=True, text=True, timeout=180, env=_clean_env(), cwd=ROOT)
    assert r.returncode == 0, r.stderr[-2000:]
    lines = _json_lines(r.stdout)
    assert len(lines) == 1                                   # rank 0 alone prints
    line = lines[0]
    assert line["n_gpus"] == 2 and line["stub"] and line["steps"] == 4
    assert line["ms_per_step"] >= 2.0                        # the slowest replica's time, per step
    # whole-job rate: the units of both replicas over that time
    assert abs(line["value"] - 2.0 / (line["ms_per_step"] * 1e-3)) < 1e-6 * line["value"]


def test_under_an_external_launcher_nothing_is_started_twice():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        port = s.getsockname()[1]
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", "--nproc-per-node", "2", "--master-addr",
           "127.0.0.1", "--master-port", str(port), os.path.join(ROOT, "bench.py"), "--gpus", "2", "--stub-step-ms", "1",
           "--steps", "3", "--warmup", "1"]
    r = subprocess.run(cmd, capture_output=True, text=True, timeout=180, env=_clean_env(), cwd=ROOT)
    assert r.returncode == 0, r.stderr[-2000:]
    lines = _json_lines(r.stdout)
    assert len(lines) == 1 and lines[0]["n_gpus"] == 2
