"""The launch path of bench.py on CPU: `--gpus 2` must start two ranks by itself (and must also run under a launcher
that already set WORLD_SIZE), reduce over them the way the GPU run does, and print one JSON line from rank 0.  The
`--dry` mode replaces the CUDA calls by a sleep (rank r sleeps r + 1 ms per step) over gloo."""
import json
import os
import socket
import subprocess
import sys

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
BENCH = os.path.join(ROOT, "bench.py")


def _json_line(stdout: str) -> dict:
    lines = [l for l in stdout.splitlines() if l.startswith("{")]
    assert len(lines) == 1, stdout
    return json.loads(lines[0])


def _env():
    env = dict(os.environ)
    for k in ("RANK", "LOCAL_RANK", "WORLD_SIZE", "MASTER_ADDR", "MASTER_PORT"):
        env.pop(k, None)
    return env


def _check_two_ranks(line):
    assert line["n_gpus"] == 2 and line["dry"] and line["steps"] == 3
    assert line["config"]["parallelism"] == "replicas x2"
    # the slow rank (2 ms per step) decides the step time; the value is the tokens of both ranks over it
    assert 1.9 < line["ms_per_step"] < 4.0
    assert abs(line["value"] - 2 * line["config"]["tokens_per_step_per_gpu"] / (line["ms_per_step"] * 1e-3)) < 1e-6
    b = line["blocks"]
    assert b["n"] >= 2 and b["steps_per_block"] == 3 and b["min_ms"] <= b["median_ms"] <= b["max_ms"]


def test_gpus_2_starts_its_own_ranks():
    res = subprocess.run([sys.executable, BENCH, "--dry", "--gpus", "2", "--steps", "3"], capture_output=True, text=True,
                         env=_env(), timeout=300)
    assert res.returncode == 0, res.stderr[-2000:]
    _check_two_ranks(_json_line(res.stdout))


def test_runs_under_an_external_launcher():
    s = socket.socket(); s.bind(("127.0.0.1", 0)); port = s.getsockname()[1]; s.close()
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", "--nproc-per-node", "2", "--master-addr",
           "127.0.0.1", "--master-port", str(port), BENCH, "--dry", "--gpus", "2", "--steps", "3"]
    res = subprocess.run(cmd, capture_output=True, text=True, env=_env(), timeout=300)
    assert res.returncode == 0, res.stderr[-2000:]
    _check_two_ranks(_json_line(res.stdout))


def test_single_rank_dry_line():
    res = subprocess.run([sys.executable, BENCH, "--dry", "--steps", "4"], capture_output=True, text=True, env=_env(),
                         timeout=300)
    assert res.returncode == 0, res.stderr[-2000:]
    line = _json_line(res.stdout)
    assert line["n_gpus"] == 1 and 0.9 < line["ms_per_step"] < 3.0
