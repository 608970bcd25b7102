"""GPU parity of the sharded statistical top-k entry points (spark_stat_moments, spark_stat_merge,
spark_stat_select) against the oracle: the parts of each row live on one GPU here, one call per part,
which is what every rank of a sharded job runs on its own part."""
import numpy as np
import pytest
import torch

from oracle import spark_oracle as O
from paper_2506_06644_b200 import binding as S
from paper_2506_06644_b200 import sharded
from tests import parity

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def ctx():
    c = S.SparkContext(0)
    yield c
    assert c.device_status() == S.SPARK_OK
    c.close()


def make_rows(rows, lens, seed):
    rng = np.random.default_rng(seed)
    parts = [rng.normal(0.3 * i, 1.0 + 0.1 * i, size=(rows, n)).astype(np.float32) for i, n in enumerate(lens)]
    return parts


@pytest.mark.parametrize("lens,k,fill", [((1000, 3096), 205, "zero"), ((100, 20000, 70000), 2000, "neginf"),
                                         ((4096, 4096, 4096, 4096), 1311, "zero"), ((260000, 40), 5000, "zero")])
def test_global_form_equals_the_oracle_on_the_whole_row(ctx, lens, k, fill):
    rows = 5
    parts = make_rows(rows, lens, seed=len(lens))
    n_total = sum(lens)
    fillc = S.SPARK_FILL_ZERO if fill == "zero" else S.SPARK_FILL_NEGINF
    dev = [torch.from_numpy(p).cuda() for p in parts]
    steps = sharded.gpu_steps(ctx, fillc, idx_cap=max(lens))
    moms = torch.stack([steps.moments(x) for x in dev])             # [m][rows][3], what the all-gather leaves on every rank
    for i, x in enumerate(parts):
        for r in range(rows):
            n, mean, m2 = O.shard_moments(x[r])
            got = moms[i, r].cpu().numpy()
            assert got[0] == n and got[1] == pytest.approx(mean, rel=1e-6, abs=1e-7) and got[2] == pytest.approx(m2, rel=1e-6)
    theta = steps.merge(moms, k, n_total)
    merged = torch.empty(rows, 3, dtype=torch.float64, device="cuda")
    S.spark_stat_merge(ctx, moms, len(lens), rows, k, n_total, theta, merged)
    torch.cuda.synchronize()
    picked = [steps.select(x, theta) for x in dev]
    dense = []
    for x in dev:
        y = torch.empty_like(x)
        S.spark_stat_select(ctx, x, rows, x.shape[1], x.stride(0), theta, fillc, None, None, None, 0, y)
        dense.append(y.cpu().numpy())
    torch.cuda.synchronize()
    th = theta.cpu().numpy()
    for r in range(rows):
        whole = np.concatenate([p[r] for p in parts])
        ref_theta, masks, outs = O.stat_topk_sharded_global([p[r] for p in parts], k, fill)
        _, std = O.mean_std(whole)
        parity.check_theta(th[r], ref_theta, std, f"row {r}")
        assert merged[r, 0].item() == n_total and merged[r, 1].item() == pytest.approx(float(np.mean(whole.astype(np.float64))), rel=1e-6, abs=1e-7)
        for i, x in enumerate(parts):
            count, idx, val = (t.cpu().numpy() for t in picked[i])
            got = idx[r, : count[r]]
            assert np.all(np.diff(got) > 0)                                  # ascending within the part
            parity.check_set(got, masks[i], x[r].astype(np.float64), ref_theta, std, f"row {r} part {i}")
            np.testing.assert_allclose(val[r, : count[r]], x[r][got] - th[r], rtol=0, atol=1e-6 * max(1.0, std))
            near = np.abs(x[r] - ref_theta) <= 1e-4 * std                    # entries whose side of theta may differ
            ok = ~near
            np.testing.assert_allclose(dense[i][r][ok], outs[i][ok], rtol=0, atol=2e-5 * max(1.0, std))


def test_k_at_least_the_total_length_keeps_everything_unshifted(ctx):
    parts = make_rows(2, (300, 724), seed=9)
    dev = [torch.from_numpy(p).cuda() for p in parts]
    steps = sharded.gpu_steps(ctx, S.SPARK_FILL_ZERO, idx_cap=724)
    moms = torch.stack([steps.moments(x) for x in dev])
    theta = steps.merge(moms, 1024, 1024)
    torch.cuda.synchronize()
    assert torch.isneginf(theta).all()
    # the selection with that threshold keeps every entry as it is (no shift by -inf), lists and dense form alike
    for fill, fillc in (("zero", S.SPARK_FILL_ZERO), ("neginf", S.SPARK_FILL_NEGINF)):
        steps = sharded.gpu_steps(ctx, fillc, idx_cap=724)
        for r in range(2):
            _, masks, outs = O.stat_topk_sharded_global([p[r] for p in parts], 1024, fill)
            for i, x in enumerate(dev):
                count, idx, val = (t.cpu().numpy() for t in steps.select(x, theta))
                y = torch.full_like(x, float("nan"))
                S.spark_stat_select(ctx, x, 2, x.shape[1], x.stride(0), theta, fillc, None, None, None, 0, y)
                torch.cuda.synchronize()
                n = parts[i].shape[1]
                assert count[r] == n == int(masks[i].sum())
                assert np.array_equal(idx[r, :n], np.arange(n))
                assert np.array_equal(val[r, :n], parts[i][r])
                assert np.array_equal(y.cpu().numpy()[r], outs[i].astype(np.float32))


def test_argument_errors(ctx):
    x = torch.zeros(2, 64, device="cuda")
    with pytest.raises(S.SparkError):
        S.spark_stat_moments(ctx, x, 2, 64, 64, None)
    with pytest.raises(S.SparkError):
        S.spark_stat_select(ctx, x, 2, 64, 64, None, S.SPARK_FILL_ZERO, None, None, None, 0, None)
    with pytest.raises(S.SparkError):
        S.spark_stat_merge(ctx, torch.zeros(1, 2, 3, dtype=torch.float64, device="cuda"), 0, 2, 5, 64, torch.zeros(2, device="cuda"), None)
