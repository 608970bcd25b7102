"""GPU parity: spark_stat_topk through the C ABI against the CPU oracle."""
import numpy as np
import pytest
import torch

from oracle import spark_oracle as O
from paper_2506_06644_b200 import binding as S
from paper_2506_06644_b200 import synth
from tests import parity

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def ctx():
    c = S.SparkContext(0)
    yield c
    assert c.device_status() == S.SPARK_OK
    c.close()


def run_topk(ctx, X, k, fill=S.SPARK_FILL_ZERO, idx_cap=None, dense=True, ld=None):
    rows, n = X.shape
    ld = ld or n
    xd = torch.zeros((rows, ld), dtype=torch.float32, device="cuda")
    xd[:, :n] = torch.from_numpy(X).cuda()
    idx_cap = n if idx_cap is None else idx_cap
    theta = torch.full((rows,), 123.0, device="cuda")
    count = torch.full((rows,), -1, dtype=torch.int32, device="cuda")
    idx = torch.full((rows, idx_cap), -1, dtype=torch.int32, device="cuda")
    val = torch.full((rows, idx_cap), float("nan"), device="cuda")
    yd = torch.full((rows, ld), float("nan"), device="cuda") if dense else None
    S.spark_stat_topk(ctx, xd, rows, n, ld, k, fill, theta, count, idx, val, idx_cap, yd)
    torch.cuda.synchronize()
    return theta.cpu().numpy(), count.cpu().numpy(), idx.cpu().numpy(), val.cpu().numpy(), \
        (yd.cpu().numpy() if dense else None)


def compare_rows(X, k, fill, out, rows=None, idx_cap=None):
    theta, count, idx, val, yd = out
    n = X.shape[1]
    for i in (range(X.shape[0]) if rows is None else rows):
        th, mask, dense = O.stat_topk(X[i], k, "zero" if fill == S.SPARK_FILL_ZERO else "neginf")
        _, std = O.mean_std(X[i]) if n > 1 else (0.0, 1.0)
        std = std if std > 0 else 1.0
        parity.check_theta(theta[i], th, std, f"row {i}")
        c = int(count[i])
        cap = n if idx_cap is None else idx_cap
        got = idx[i, : min(c, cap)]
        assert np.all(np.diff(got) > 0), "indices must ascend"
        if c <= cap:
            diff = parity.check_set(got, mask, X[i], th, std, f"row {i}")
            assert c == int(mask.sum()) + int((~mask[diff]).sum()) - int(mask[diff].sum())
            shift = th if np.isfinite(th) else 0.0
            np.testing.assert_allclose(val[i, :c], X[i][got].astype(np.float64) - shift, atol=2e-5 * max(std, abs(shift)))
            assert np.all(idx[i, c:] == -1)
        if yd is not None:
            same = np.ones(n, dtype=bool)
            if c <= cap:
                same[diff] = False
            fin = np.isfinite(dense) & same
            np.testing.assert_allclose(yd[i, :n][fin], dense[fin], atol=2e-5 * max(std, abs(th) if np.isfinite(th) else 0))
            assert np.array_equal(np.isneginf(yd[i, :n][same]), np.isneginf(dense[same]))


def test_cfg1_rows_against_oracle_and_sort(ctx):
    X = synth.rows_f32("normal", 64, 1024, seed=0)
    out = run_topk(ctx, X, 82)
    compare_rows(X, 82, S.SPARK_FILL_ZERO, out)
    theta, count, idx, _, _ = out
    for i in range(64):                         # the selected set is the sort-based top-count set
        top = np.argsort(-X[i].astype(np.float64), kind="stable")[: count[i]]
        assert set(top.tolist()) == set(idx[i, : count[i]].tolist())


@pytest.mark.parametrize("dist", ["normal", "laplace", "student_t4"])
@pytest.mark.parametrize("n,k,rows", [(65536, 5243, 6), (20001, 400, 5), (16384, 4096, 4), (7, 3, 9), (300000, 6000, 2)])
def test_row_lengths_and_clusters(ctx, dist, n, k, rows):
    # 65536 -> 4 blocks per row; 20001 -> 2 blocks and a ragged last vector; 300000 -> 8 blocks
    X = synth.rows_f32(dist, rows, n, seed=3) * 1.7 + 0.3
    ld = (n + 3) // 4 * 4 + 8
    for fill in (S.SPARK_FILL_ZERO, S.SPARK_FILL_NEGINF):
        out = run_topk(ctx, X, k, fill, ld=ld)
        compare_rows(X, k, fill, out)


def test_rows_too_long_for_shared_memory(ctx):
    X = synth.rows_f32("normal", 2, 500000, seed=5) + 50.0     # mean far from zero
    out = run_topk(ctx, X, 40000, dense=True)
    compare_rows(X, 40000, S.SPARK_FILL_ZERO, out)


def test_degenerate_cases(ctx):
    X = synth.rows_f32("normal", 3, 1000, seed=6)
    out = run_topk(ctx, X, 1000)                               # k >= n keeps everything unshifted
    theta, count, idx, val, yd = out
    assert np.all(np.isneginf(theta)) and np.all(count == 1000)
    assert np.array_equal(idx, np.tile(np.arange(1000, dtype=np.int32), (3, 1)))
    assert np.array_equal(val, X) and np.array_equal(yd, X)
    # empty selection: evenly spaced grid and a constant row
    G = np.stack([np.linspace(-1, 1, 1024), np.full(1024, 3.25)]).astype(np.float32)
    theta, count, idx, val, yd = run_topk(ctx, G, 20)
    assert np.all(count == 0) and np.all(yd == 0.0) and np.all(idx == -1)
    assert abs(theta[0] - 1.1931251) < 2e-5 and theta[1] == 3.25
    # hand example
    theta, count, idx, val, yd = run_topk(ctx, np.arange(8, dtype=np.float32)[None], 3)
    assert count[0] == 3 and list(idx[0, :3]) == [5, 6, 7] and abs(theta[0] - 4.2805038) < 1e-6
    np.testing.assert_allclose(val[0, :3], [0.7194961, 1.7194961, 2.7194961], atol=1e-6)


def test_truncated_lists_report_overflow(ctx):
    X = synth.rows_f32("normal", 4, 4096, seed=7)
    out = run_topk(ctx, X, 400, idx_cap=64)
    compare_rows(X, 400, S.SPARK_FILL_ZERO, out, idx_cap=64)
    assert np.all(out[1] > 64)
    assert ctx.device_status() == S.SPARK_ERR_OVERFLOW
    assert ctx.device_status() == S.SPARK_OK                  # reading clears it


def test_argument_errors(ctx):
    x = torch.zeros((4, 64), device="cuda")
    th = torch.zeros(4, device="cuda")
    for bad in (dict(k=0), dict(n=0), dict(ld=60), dict(fill=7)):
        a = dict(rows=4, n=64, ld=64, k=5, fill=0)
        a.update(bad)
        with pytest.raises(S.SparkError) as e:
            S.spark_stat_topk(ctx, x, a["rows"], a["n"], a["ld"], a["k"], a["fill"], th, None, None, None, 0, None)
        assert e.value.status == S.SPARK_ERR_INVALID_ARG
    with pytest.raises(S.SparkError) as e:                     # rows must start on 16-byte boundaries
        S.spark_stat_topk(ctx, x, 4, 62, 62, 5, 0, th, None, None, None, 0, None)
    assert e.value.status == S.SPARK_ERR_UNSUPPORTED


def test_full_size_workload_sampled(ctx):
    """4096 x 65536 rows (the standalone top-k workload): sampled rows against the oracle, and the
    count property on every row."""
    rows, n = 4096, 65536
    for dist, k in (("normal", 5243), ("laplace", 1311), ("student_t4", 16384)):
        X = synth.rows_f32(dist, rows, n, seed=11)
        xd = torch.from_numpy(X).cuda()
        theta = torch.empty(rows, device="cuda")
        count = torch.empty(rows, dtype=torch.int32, device="cuda")
        cap = 32768
        idx = torch.full((rows, cap), -1, dtype=torch.int32, device="cuda")
        val = torch.empty((rows, cap), device="cuda")
        S.spark_stat_topk(ctx, xd, rows, n, n, k, 0, theta, count, idx, val, cap, None)
        torch.cuda.synchronize()
        th, ct, ix, vl = theta.cpu().numpy(), count.cpu().numpy(), idx.cpu().numpy(), val.cpu().numpy()
        sample = np.random.default_rng(0).choice(rows, 24, replace=False)
        compare_rows(X, k, 0, (th, ct, ix, vl, None), rows=sample, idx_cap=cap)
        # every row: count equals the number of entries above the reported theta, up to the band
        above = (xd > theta[:, None]).sum(1).cpu().numpy()
        assert np.array_equal(above, ct)
        if dist == "normal":
            sd = 44.1
            assert np.all(np.abs(ct - k) < 6 * sd) and abs(ct.mean() - k) < 0.5 * sd
        del xd, idx, val


@pytest.mark.parametrize("n,k,rows", [(65536, 1311, 450), (40004, 9000, 320), (28670, 500, 160), (65533, 70000, 150)])
def test_rows_held_on_chip_by_a_persistent_block(ctx, n, k, rows):
    # 16K < n <= 64K: one block per SM walks over several rows, part of each row in shared memory and part in
    # registers (n = 28670: registers only after the first 8190 values; n = 65533: ragged tail; k >= n: identity).
    # Every row is compared on theta and count, a sample of rows on sets, values and the dense output.
    X = synth.rows_f32("laplace", rows, n, seed=11) * 0.8 + 25.0      # mean far from zero
    ld = (n + 3) // 4 * 4
    out = run_topk(ctx, X, k, ld=ld)
    theta, count = out[0], out[1]
    x64 = X.astype(np.float64)
    if k < n:
        mean = x64.mean(axis=1)
        std = x64.std(axis=1, ddof=1)
        th = mean + std * O.gaussian_upper_quantile(k / n)
        assert np.all(np.abs(theta - th) <= parity.THETA_RTOL * np.maximum(np.abs(th), std))
        near = (np.abs(x64 - th[:, None]) <= parity.BAND * std[:, None]).sum(axis=1)
        assert np.all(np.abs(count - (x64 > th[:, None]).sum(axis=1)) <= near)
    else:
        assert np.all(np.isneginf(theta)) and np.all(count == n)
    compare_rows(X, k, S.SPARK_FILL_ZERO, out, rows=[0, 1, 147, 148, 149, rows - 1])
