"""The multi-rank plumbing of the benchmark on CPU: two gloo ranks run as independent replicas,
meet at the barrier and reduce their timings (max) and units (sum). Also the reference arm of
bench.py (the CPU checker timed alone), which needs no GPU."""
import json
import os
import socket
import subprocess
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

WORKER = r"""
import os, sys, json
sys.path.insert(0, {root!r})
from paper_2306_08289_b200.distutil import Ranks, aggregate_throughput
r = Ranks(backend="gloo")
assert r.world == 2
r.barrier()
units = 100.0 * (r.rank + 1)          # rank 0: 100 units, rank 1: 200 units
secs = 2.0 if r.rank == 0 else 4.0    # the slower rank sets the time
thr, slow = aggregate_throughput(r, units, secs)
mx = r.max_over_ranks(float(r.rank))
r.barrier()
print(json.dumps({{"rank": r.rank, "thr": thr, "slow": slow, "mx": mx}}), flush=True)
r.close()
"""


def _free_port():
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    p = s.getsockname()[1]
    s.close()
    return p


def test_two_gloo_ranks_aggregate_like_the_benchmark(tmp_path):
    script = tmp_path / "worker.py"
    script.write_text(WORKER.format(root=ROOT))
    port = _free_port()
    procs = []
    for rank in range(2):
        env = dict(os.environ, RANK=str(rank), LOCAL_RANK=str(rank), WORLD_SIZE="2", MASTER_ADDR="127.0.0.1",
                   MASTER_PORT=str(port))
        procs.append(subprocess.Popen([sys.executable, str(script)], env=env, stdout=subprocess.PIPE, text=True))
    outs = []
    for p in procs:
        out, _ = p.communicate(timeout=120)
        assert p.returncode == 0
        outs.append(json.loads(out.strip().splitlines()[-1]))
    for o in outs:
        assert o["slow"] == 4.0 and abs(o["thr"] - 300.0 / 4.0) < 1e-12 and o["mx"] == 1.0


def test_single_process_needs_no_process_group():
    from paper_2306_08289_b200.distutil import Ranks, aggregate_throughput

    env = {k: os.environ.pop(k) for k in ("WORLD_SIZE", "RANK", "LOCAL_RANK") if k in os.environ}
    try:
        r = Ranks()
        assert r.world == 1 and r.dist is None
        r.barrier()
        assert aggregate_throughput(r, 50.0, 2.0) == (25.0, 2.0)
    finally:
        os.environ.update(env)


def test_reference_arm_runs_on_cpu_and_prints_the_contract_line():
    cmd = [sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--config", "cfg1", "--steps", "2",
           "--warmup", "1", "--events-per-step", "100"]
    env = {k: v for k, v in os.environ.items() if k not in ("WORLD_SIZE", "RANK", "LOCAL_RANK")}
    out = subprocess.run(cmd, capture_output=True, text=True, timeout=300, env=env)
    assert out.returncode == 0, out.stderr
    line = json.loads(out.stdout.strip().splitlines()[-1])
    assert line["impl"] == "reference" and line["unit"] == "events/s" and line["value"] > 0
    assert line["cpu_baseline"]["kind"] == "oracle" and line["cpu_baseline"]["cores"] >= 1
    assert line["e2e"]["h2d_bytes_per_step"] == 0 and line["steps"] == 2 and line["warmup"] == 1


def test_benchmark_refuses_to_run_its_own_arm_without_a_gpu():
    import torch

    if torch.cuda.is_available():
        pytest.skip("a CUDA device is present")
    out = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--config", "cfg1", "--steps", "1", "--warmup", "1"],
                         capture_output=True, text=True, timeout=300)
    assert out.returncode != 0 and "no CPU path" in (out.stderr + out.stdout)
