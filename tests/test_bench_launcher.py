"""`python bench.py --gpus N` started by hand must itself produce N replicas (one process per GPU, the rendezvous
variables torchrun would set) and print ONE line with n_gpus = N; under torchrun it must use the ranks it is given.
Checked on CPU with the benchmark's stub step (gloo, no GPU work): the launcher, the rendezvous, the barrier, the
MAX-over-ranks timing and the line's base keys are the real ones."""
import json
import os
import socket
import subprocess
import sys

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
BENCH = os.path.join(ROOT, "bench.py")


def _lines(out):
    return [json.loads(l) for l in out.stdout.splitlines() if l.startswith("{")]


def test_gpus_flag_spawns_replicas_by_itself():
    env = {k: v for k, v in os.environ.items() if k not in ("RANK", "LOCAL_RANK", "WORLD_SIZE", "MASTER_ADDR", "MASTER_PORT")}
    out = subprocess.run([sys.executable, BENCH, "--stub", "--gpus", "2", "--steps", "5", "--warmup", "3"], env=env,
                         capture_output=True, text=True, timeout=300, cwd=ROOT)
    assert out.returncode == 0, out.stderr[-2000:]
    lines = _lines(out)
    assert len(lines) == 1
    d = lines[0]
    assert d["n_gpus"] == 2 and d["steps"] == 5 and d["unit"] == "rounds/s" and d["scaling"] == "weak"
    assert d["config"]["parallelism"] == "replicas x2" and "workload" in d["config"]
    # both ranks' steps count, over the slower rank's time (rank 1 sleeps 4 ms per step)
    assert d["ms_per_step"] >= 4.0 and abs(d["value"] - 2 * 1000.0 / d["ms_per_step"]) < 1e-2 * d["value"]


def test_ranks_given_by_the_environment_are_used():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        port = s.getsockname()[1]
    procs = []
    for r in range(2):
        env = dict(os.environ, RANK=str(r), LOCAL_RANK=str(r), WORLD_SIZE="2", MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
        procs.append(subprocess.Popen([sys.executable, BENCH, "--stub", "--gpus", "2", "--steps", "3", "--warmup", "3"], env=env,
                                      stdout=subprocess.PIPE, stderr=subprocess.PIPE, text=True, cwd=ROOT))
    outs = [p.communicate(timeout=300) for p in procs]
    assert [p.returncode for p in procs] == [0, 0], outs[0][1][-1000:] + outs[1][1][-1000:]
    first = [json.loads(l) for l in outs[0][0].splitlines() if l.startswith("{")]
    assert len(first) == 1 and first[0]["n_gpus"] == 2
    assert not [l for l in outs[1][0].splitlines() if l.startswith("{")]          # only rank 0 prints


def test_single_gpu_default_does_not_spawn():
    out = subprocess.run([sys.executable, BENCH, "--stub", "--steps", "3"], capture_output=True, text=True, timeout=300, cwd=ROOT)
    assert out.returncode == 0, out.stderr[-2000:]
    d = _lines(out)
    assert len(d) == 1 and d[0]["n_gpus"] == 1 and "config 5" in d[0]["config"]["workload"]
