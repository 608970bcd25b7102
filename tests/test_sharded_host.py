"""Host logic of the sharded statistical top-k (paper_2506_06644_b200.sharded) on two CPU ranks over gloo:
the all-gather of the parts' moments, their order, the length check, and that every rank ends with the
threshold of the whole row.  The arithmetic of the three steps comes from the oracle here; on a GPU the
same function runs on the library's kernels (tests/test_gpu_stat_shard.py)."""
import os
import socket

import numpy as np
import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from oracle import spark_oracle as O
from paper_2506_06644_b200 import sharded

ROWS, N, K = 3, 8192, 410
CUT = 3000                                   # rank 0 holds [0, CUT), rank 1 the rest: unequal parts


def free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def rows_of_x():
    rng = np.random.default_rng(123)
    x = rng.normal(size=(ROWS, N))
    x[:, CUT:] += 0.5                        # parts with different means: merging must use the distances of the means
    return x


def oracle_steps():
    def moments(x):
        return torch.tensor([O.shard_moments(r.numpy()) for r in x], dtype=torch.float64)

    def merge(parts, k, n_total):
        out = []
        for row in range(parts.shape[1]):
            n, mean, m2 = O.combine_moments([tuple(parts[s, row].tolist()) for s in range(parts.shape[0])])
            assert n == n_total
            out.append(mean + np.sqrt(m2 / (n - 1)) * O.gaussian_upper_quantile(k / n))
        return torch.tensor(out, dtype=torch.float64)

    def select(x, theta):
        return [np.nonzero(x[r].numpy() > float(theta[r]))[0] for r in range(x.shape[0])]

    return sharded.Steps(moments, merge, select)


def _rank_main(rank, world, port, q):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    x = rows_of_x()
    mine = torch.from_numpy(x[:, :CUT] if rank == 0 else x[:, CUT:]).contiguous()
    theta, picked = sharded.global_stat_topk(mine, K, N, oracle_steps())
    parts = sharded.gather_parts(oracle_steps().moments(mine))
    bad = None
    try:
        sharded.global_stat_topk(mine, K, N + 1, oracle_steps())
    except ValueError as e:
        bad = str(e)
    dist.barrier()
    dist.destroy_process_group()
    q.put((rank, theta.numpy(), [p + (0 if rank == 0 else CUT) for p in picked], parts.numpy(), bad))


def test_two_ranks_agree_on_the_threshold_of_the_whole_row():
    world, port = 2, free_port()
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    procs = [ctx.Process(target=_rank_main, args=(r, world, port, q)) for r in range(world)]
    for p in procs:
        p.start()
    got = {}
    for _ in range(world):
        rank, theta, picked, parts, bad = q.get(timeout=120)
        got[rank] = (theta, picked, parts, bad)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    x = rows_of_x()
    for row in range(ROWS):
        ref_theta, ref_mask, _ = O.stat_topk(x[row], K)
        for rank in range(world):
            assert got[rank][0][row] == pytest.approx(ref_theta, rel=1e-12)
        both = np.concatenate([got[0][1][row], got[1][1][row]])
        assert np.array_equal(np.sort(both), np.nonzero(ref_mask)[0])
    # part r of the gathered moments is rank r's, on every rank
    for rank in range(world):
        parts = got[rank][2]
        assert parts.shape == (2, ROWS, 3)
        assert np.all(parts[0, :, 0] == CUT) and np.all(parts[1, :, 0] == N - CUT)
        assert np.array_equal(parts, got[0][2])
        assert got[rank][3] is not None and "n_total" in got[rank][3]


def test_local_k():
    assert sharded.local_k(410, 2) == 205 and sharded.local_k(3, 8) == 1 and sharded.local_k(7, 2) == 3
