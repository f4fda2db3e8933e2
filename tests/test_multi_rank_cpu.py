"""The N > 1 path of the benchmark on CPU: two gloo ranks launched the way the driver launches
bench.py (torch.distributed.run, 127.0.0.1).  The path has no data-path collective (heads and
batches are independent, every rank runs a replica), so what there is to cover is the
rendezvous, the barrier, the max-over-ranks step time, the whole-job aggregate, and that the
reference arm prints from rank 0 only."""
import json
import os
import subprocess
import sys

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def torchrun(script_args, port):
    env = dict(os.environ, OMP_NUM_THREADS="2")
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", "--nproc-per-node", "2",
           "--master-addr", "127.0.0.1", "--master-port", str(port)] + script_args
    return subprocess.run(cmd, cwd=ROOT, env=env, capture_output=True, text=True, timeout=280)


def json_lines(text):
    out = []
    for line in text.splitlines():
        line = line.strip()
        if line.startswith("{") and line.endswith("}"):
            out.append(json.loads(line))
    return out


def test_two_gloo_ranks_max_time_and_aggregate():
    r = torchrun([os.path.join("tests", "rank_worker.py")], 29611)
    assert r.returncode == 0, r.stderr[-2000:]
    lines = json_lines(r.stdout)
    assert len(lines) == 1                     # rank 0 only
    d = lines[0]
    assert d["world"] == 2
    assert d["ms"] == 20.0                     # the slower rank's time
    assert d["value"] == 1000 * 2 * 4 / 20e-3  # all ranks' tokens over that time


def test_reference_arm_under_torchrun_prints_once():
    r = torchrun(["bench.py", "--impl", "reference", "--gpus", "2", "--steps", "1", "--warmup", "0",
                  "--config", "1"], 29612)
    assert r.returncode == 0, r.stderr[-2000:]
    lines = json_lines(r.stdout)
    assert len(lines) == 1
    d = lines[0]
    assert d["impl"] == "reference" and d["n_gpus"] == 2 and d["value"] > 0
    assert d["cpu_baseline"]["kind"] == "oracle" and d["e2e"]["h2d_bytes_per_step"] == 0
