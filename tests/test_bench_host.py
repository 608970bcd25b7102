"""Host-side logic of bench.py, on CPU: the reference arm (the oracle timed as it stands) alone and
under a two-rank launch, and the multi-rank reduction of the step time over a gloo process group."""
import json
import os
import socket
import subprocess
import sys

import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
sys.path.insert(0, ROOT)

import bench  # noqa: E402


def free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def json_lines(text):
    return [json.loads(l) for l in text.splitlines() if l.startswith("{")]


REF_KEYS = {"impl", "metric", "value", "unit", "n_gpus", "steps", "warmup", "ms_per_step", "higher_is_better", "scaling",
            "vs_baseline", "dtype", "data", "config", "cpu_baseline", "e2e"}


def test_reference_arm_prints_one_contract_line():
    out = subprocess.run([sys.executable, "bench.py", "--impl", "reference", "--shape", "tiny", "--ctx", "64", "--steps", "2",
                          "--warmup", "1"], cwd=ROOT, capture_output=True, text=True, timeout=600)
    assert out.returncode == 0, out.stderr[-2000:]
    lines = json_lines(out.stdout)
    assert len(lines) == 1
    line = lines[0]
    assert REF_KEYS <= set(line)
    assert line["impl"] == "reference" and line["higher_is_better"] is False and line["vs_baseline"] is None
    assert line["value"] > 0 and line["unit"] == "us/token/layer" and line["dtype"] == "f64"
    assert line["cpu_baseline"]["kind"] == "oracle" and line["cpu_baseline"]["cores"] >= 1
    assert line["e2e"] == {"value": line["value"], "unit": line["unit"], "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}
    assert "workload" in line["config"] and "model" not in line["config"]


def test_reference_arm_under_a_two_rank_launch():
    # launched the way the N > 1 runs are: rank 0 alone works and prints, the other rank leaves with 0
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", "--nproc-per-node", "2", "--master-addr", "127.0.0.1",
           "--master-port", str(free_port()), "bench.py", "--impl", "reference", "--gpus", "2", "--shape", "tiny", "--ctx", "64",
           "--steps", "1", "--warmup", "1"]
    out = subprocess.run(cmd, cwd=ROOT, capture_output=True, text=True, timeout=900)
    assert out.returncode == 0, out.stderr[-2000:]
    lines = json_lines(out.stdout)
    assert len(lines) == 1 and lines[0]["impl"] == "reference" and lines[0]["n_gpus"] == 2


def _rank_main(rank, world, port, q):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    mine = 10.0 + 5.0 * rank                      # rank 1 is the slower replica
    worst = bench.max_over_ranks(mine, world, torch.device("cpu"))
    dist.barrier()
    dist.destroy_process_group()
    q.put((rank, worst))


def test_step_time_is_the_slowest_rank_and_value_counts_every_replica():
    world, port = 2, free_port()
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    procs = [ctx.Process(target=_rank_main, args=(r, world, port, q)) for r in range(world)]
    for p in procs:
        p.start()
    got = dict(q.get(timeout=300) for _ in range(world))
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    assert got == {0: 15.0, 1: 15.0}
    # replicas: the same wall time yields half the time per token with twice the replicas (weak scaling)
    one = bench.us_per_token_per_layer(15.0, steps=3, n_layers=26, batch=1, world=1)
    two = bench.us_per_token_per_layer(15.0, steps=3, n_layers=26, batch=1, world=2)
    assert one == pytest.approx(15.0 / 3 * 1e3 / 26) and two == pytest.approx(one / 2)
    assert bench.max_over_ranks(7.5, 1, torch.device("cpu")) == 7.5
