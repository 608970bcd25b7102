"""Pins for the CPU oracle: every check compares it with something other than itself --
hand-worked fixtures, closed forms, the paper's theorem, library routines on special
cases, brute force on tiny inputs.  No GPU needed."""
import math

import numpy as np
import pytest
import scipy.special
import scipy.stats
import torch

from oracle import spark_oracle as O
from paper_2506_06644_b200 import synth
from tests.conftest import read_golden


# ----------------------------------------------------------------------------- quantile
def test_quantile_matches_table_and_library():
    rows = read_golden("gaussian_quantiles.txt")
    assert len(rows) == 14
    for p_str, (val,) in ((k, v[0]) for k, v in rows.items()):
        p = float(p_str)
        z = O.gaussian_upper_quantile(1.0 - p)
        assert abs(z - val) < 2e-12, (p, z, val)
        assert abs(z - scipy.special.ndtri(p)) < 1e-12


def test_quantile_tails_and_symmetry():
    for p in (1e-12, 1e-6, 0.003, 0.3, 0.5, 0.7, 0.999):
        z = O.gaussian_upper_quantile(p)
        assert abs(z + scipy.special.ndtri(p)) < 1e-10 * max(1.0, abs(z))
        assert abs(z + O.gaussian_upper_quantile(1.0 - p)) < 1e-9 or p < 1e-9
    with pytest.raises(ValueError):
        O.gaussian_upper_quantile(0.0)


# ----------------------------------------------------------------------------- mean / std
def test_mean_std_is_bessel():
    x = synth.normal_f32((4097,), 3, 0) * 3.0 + 100.0
    m, s = O.mean_std(x)
    assert abs(m - np.mean(x, dtype=np.float64)) < 1e-12 * 100
    assert abs(s - np.std(x.astype(np.float64), ddof=1)) < 1e-12
    assert abs(s - np.std(x.astype(np.float64), ddof=0)) > 1e-5      # not the population form


# ----------------------------------------------------------------------------- hand examples
def test_w1_hand_example():
    g = read_golden("w1_stat_topk.txt")
    x = np.arange(8.0)
    theta, mask, out = O.stat_topk(x, 3)
    m, s = O.mean_std(x)
    assert abs(m - g["mean"][0][0]) < 1e-15
    assert abs(s - g["std"][0][0]) < 1e-14
    assert abs(O.gaussian_upper_quantile(3 / 8) - g["z"][0][0]) < 1e-12
    assert abs(theta - g["theta"][0][0]) < 1e-12
    assert list(np.flatnonzero(mask)) == [int(v) for v in g["active"][0]]
    np.testing.assert_allclose(out[mask], g["values"][0], atol=1e-12)
    assert np.all(out[~mask] == 0.0)
    _, mask2, out2 = O.stat_topk(x, 3, "neginf")
    assert np.array_equal(mask, mask2) and np.all(np.isneginf(out2[~mask]))
    np.testing.assert_array_equal(out2[mask], out[mask])


def test_w2_tie_rule_and_tiny_ffn():
    g = read_golden("w2_tiny_ffn.txt")
    x = np.array([1.0, 2.0, 1.0, -1.0])
    K1 = np.array([[1, 0, -1, 2], [0, 1, 1, -1.0]])
    K2 = np.array([[1, 2, 0, 0], [0, 1, 1, 2.0]])
    V = np.array([[1, 0, 0, 1], [0, 1, 0, -1], [0, 0, 1, 1], [1, 1, 1, 0.0]])
    for form in ("erf", "tanh"):
        res = O.spark_ffn(x, K1, K2, V, k=2, r=2, gelu_form=form)
        np.testing.assert_allclose(res["s"], g["s"][0], atol=0)
        assert res["theta"] == g["theta"][0][0]
        assert list(np.flatnonzero(res["mask"])) == [1]          # entries equal to theta are dropped
        u1 = g["gelu1_" + form][0][0]
        np.testing.assert_allclose(res["y"], [0.0, u1, 0.0, u1], atol=1e-15)


# ----------------------------------------------------------------------------- structure of the selected set
@pytest.mark.parametrize("dist", ["normal", "laplace", "student_t4"])
def test_selected_set_is_the_sorted_top_count(dist):
    X = synth.rows_f32(dist, 64, 1024, seed=0)
    for row in X:
        theta, mask, out = O.stat_topk(row, 82)
        m = int(mask.sum())
        top = np.argsort(-row.astype(np.float64), kind="stable")[:m]
        assert set(top.tolist()) == set(np.flatnonzero(mask).tolist())
        # soft threshold: max(x - theta, 0) written out
        np.testing.assert_array_equal(out, np.maximum(row.astype(np.float64) - theta, 0.0))


def _count_sd(n, k):
    # std of (#{x_i > theta} - k) for i.i.d. Gaussian entries when mean and std are estimated:
    # n * [p(1-p) - phi(z)^2 (1 + z^2/2)]
    p = k / n
    z = scipy.special.ndtri(1 - p)
    phi = math.exp(-0.5 * z * z) / math.sqrt(2 * math.pi)
    return math.sqrt(n * (p * (1 - p) - phi * phi * (1 + 0.5 * z * z)))


@pytest.mark.parametrize("n,k", [(1024, 82), (9216, 737), (65536, 1311), (65536, 16384), (32768, 256)])
def test_count_close_to_k_on_gaussian_rows(n, k):
    rows = 48
    X = synth.normal_f32((rows, n), 1, n + k) * 2.5 - 7.0
    counts = np.array([O.stat_topk(r, k)[1].sum() for r in X])
    # Theorem 1 with delta = 0.01 (always true, loose)
    delta = 0.01
    bound = 4 * math.sqrt(math.log(6 / delta) / n) * (1 + math.sqrt(-2 * math.log(min(k / n, 1 - k / n))))
    assert np.all(np.abs(counts - k) / n <= bound)
    sd = _count_sd(n, k)
    assert np.all(np.abs(counts - k) <= 6 * sd + 1)
    assert abs(counts.mean() - k) <= 0.5 * sd + 1


@pytest.mark.parametrize("frac", [0.02, 0.08, 0.25])
def test_selected_fraction_on_laplace_rows(frac):
    # population std of Laplace(0,1) is sqrt(2): P(x > sqrt(2) z) = exp(-sqrt(2) z) / 2
    n = 65536
    k = round(frac * n)
    z = scipy.special.ndtri(1 - k / n)
    expect = 0.5 * math.exp(-math.sqrt(2) * z)
    X = synth.laplace_f32((16, n), 2, 7)
    got = np.mean([O.stat_topk(r, k)[1].mean() for r in X])
    assert abs(got - expect) < 0.004


def test_empty_selection_is_legitimate():
    x = np.linspace(-1.0, 1.0, 1024)
    theta, mask, out = O.stat_topk(x, 20)
    assert abs(theta - 1.1931251346) < 1e-9 and mask.sum() == 0 and np.all(out == 0)
    theta, mask, out = O.stat_topk(np.full(100, 3.25), 5)
    assert mask.sum() == 0                                # constant row: nothing is strictly above


def test_degenerate_k():
    x = synth.normal_f32((50,), 5, 0)
    theta, mask, out = O.stat_topk(x, 50)
    assert theta == -np.inf and mask.all() and np.array_equal(out, x.astype(np.float64))
    theta, mask, out = O.stat_topk(x, 0, "neginf")
    assert not mask.any() and np.all(np.isneginf(out))


# ----------------------------------------------------------------------------- activations
def test_activations_match_library():
    a = torch.linspace(-9, 9, 2001, dtype=torch.float64)
    np.testing.assert_allclose(O.gelu(a.numpy(), "erf"), torch.nn.functional.gelu(a).numpy(), atol=1e-14)
    np.testing.assert_allclose(O.gelu(a.numpy(), "tanh"),
                               torch.nn.functional.gelu(a, approximate="tanh").numpy(), atol=1e-14)
    b = torch.tensor([-800.0, -40.0, -1.0, 0.0, 1e-9, 2.0, 19.0, 40.0], dtype=torch.float64)
    np.testing.assert_allclose(O.softplus(b.numpy()), torch.nn.functional.softplus(b, threshold=700.0).numpy(),
                               rtol=1e-14, atol=0)
    assert O.softplus(np.array([800.0]))[0] == 800.0          # no overflow
    assert O.softplus(np.array([0.0]))[0] == math.log(2.0)


# ----------------------------------------------------------------------------- Spark FFN
def _tiny_ffn(seed=0, batch=1):
    return synth.ffn_inputs(256, 1024, 128, 82, batch, "f32", seed)


def test_ffn_brute_force_loops():
    p = synth.ffn_inputs(16, 48, 6, 9, 1, "f32", seed=4)
    K1, K2, V, x = p.K1t.T.astype(np.float64), p.K2t.T.astype(np.float64), p.Vt.T.astype(np.float64), p.x[0].astype(np.float64)
    res = O.spark_ffn(x, K1, K2, V, p.k, p.r, "erf")
    # element loops straight from Eq. 2, with the active set taken by sorting the scores
    s = [sum(K1[i][j] * x[i] for i in range(p.r)) for j in range(p.d_ff)]
    mean = sum(s) / len(s)
    std = math.sqrt(sum((v - mean) ** 2 for v in s) / (len(s) - 1))
    theta = mean + std * scipy.special.ndtri(1 - p.k / p.d_ff)
    order = sorted(range(p.d_ff), key=lambda j: -s[j])
    m = int(res["mask"].sum())
    assert 0 < m < p.d_ff and set(order[:m]) == set(np.flatnonzero(res["mask"]).tolist())
    y = [0.0] * p.d
    for j in order[:m]:
        a = s[j] - theta
        g = a * 0.5 * (1 + math.erf(a / math.sqrt(2)))
        t = sum(K2[i][j] * x[p.r + i] for i in range(p.d - p.r))
        for c in range(p.d):
            y[c] += V[c][j] * g * t
    np.testing.assert_allclose(res["y"], y, rtol=1e-11, atol=1e-13)


def test_ffn_zeroing_inactive_rows_changes_nothing():
    p = _tiny_ffn()
    K1, K2, V = p.K1t.T, p.K2t.T.copy(), p.Vt.T.copy()
    a = O.spark_ffn(p.x[0], K1, K2, V, p.k, p.r)
    K2[:, ~a["mask"]] = 0.0
    V[:, ~a["mask"]] = 0.0
    b = O.spark_ffn(p.x[0], K1, K2, V, p.k, p.r)
    assert np.array_equal(a["y"], b["y"]) and 60 < a["mask"].sum() < 105
    # and the inactive rows do matter to a dense evaluation (the test has teeth)
    K2b = p.K2t.T.copy()
    K2b[:, a["mask"]] = 0.0
    assert np.allclose(O.spark_ffn(p.x[0], K1, K2b, p.Vt.T, p.k, p.r)["y"], 0.0)


@pytest.mark.parametrize("form", ["tanh", "erf"])
def test_ffn_k_equal_n_is_dense_gelu_ffn(form):
    p = _tiny_ffn(seed=1)
    res = O.spark_ffn(p.x[0], p.K1t.T, p.K2t.T, p.Vt.T, p.d_ff, p.r, form)
    x = torch.from_numpy(p.x[0]).double()
    K1t, K2t, Vt = (torch.from_numpy(a).double() for a in (p.K1t, p.K2t, p.Vt))
    act = torch.nn.functional.gelu(K1t @ x[: p.r], approximate="tanh" if form == "tanh" else "none")
    y = Vt.T @ (act * (K2t @ x[p.r:]))
    np.testing.assert_allclose(res["y"], y.numpy(), rtol=1e-12, atol=1e-14)
    assert res["mask"].all()


def test_ffn_permutation_and_linearity():
    p = _tiny_ffn(seed=2)
    K1, K2, V = p.K1t.T.astype(np.float64), p.K2t.T.astype(np.float64), p.Vt.T.astype(np.float64)
    base = O.spark_ffn(p.x[0], K1, K2, V, p.k, p.r)
    perm = np.random.default_rng(0).permutation(p.d_ff)
    per = O.spark_ffn(p.x[0], K1[:, perm], K2[:, perm], V[:, perm], p.k, p.r)
    np.testing.assert_allclose(per["y"], base["y"], rtol=1e-10, atol=1e-13)
    assert np.array_equal(per["mask"], base["mask"][perm])
    lin = O.spark_ffn(p.x[0], K1, -2.0 * K2, 3.0 * V, p.k, p.r)
    np.testing.assert_allclose(lin["y"], -6.0 * base["y"], rtol=1e-12, atol=1e-14)


def test_ffn_gelu_sees_the_shifted_score():
    # one active neuron far above the rest: y = V[:,j] * GELU(s_j - theta) * t_j, not GELU(s_j)
    d, d_ff, r = 8, 64, 4
    rng = np.random.default_rng(3)
    K1 = rng.normal(size=(r, d_ff)) * 0.01
    K1[:, 5] = 2.0
    K2, V = rng.normal(size=(d - r, d_ff)), rng.normal(size=(d, d_ff))
    x = np.ones(d)
    res = O.spark_ffn(x, K1, K2, V, 1, r, "erf")
    assert list(np.flatnonzero(res["mask"])) == [5]
    a = res["s"][5] - res["theta"]
    expect = V[:, 5] * (a * 0.5 * (1 + math.erf(a / math.sqrt(2)))) * (K2[:, 5] @ x[r:])
    np.testing.assert_allclose(res["y"], expect, rtol=1e-12)


# ----------------------------------------------------------------------------- Spark attention
def _attn_case(n, seed=0, hd=64, r=32):
    rng = np.random.default_rng(seed)
    return rng.normal(size=hd) / 4, rng.normal(size=(hd, n)), rng.normal(size=(hd, n)), r


def test_attention_short_context_is_dense_spark_attention():
    q, K, V, r = _attn_case(40)
    res = O.spark_attention_head(q, K, V, k_attn=64, r=r)
    tq, tK, tV = (torch.from_numpy(a) for a in (q, K, V))
    w = torch.softmax(tK[:r].T @ tq[:r], dim=0) * torch.nn.functional.softplus(tK[r:].T @ tq[r:])
    np.testing.assert_allclose(res["o"], (tV @ w).numpy(), rtol=1e-12, atol=1e-14)
    assert res["mask"].all() and res["theta"] == -np.inf


def test_attention_reduces_to_library_sdpa():
    # with q[r:] = 0 the gate is softplus(0) = ln 2 for every token
    q, K, V, r = _attn_case(300, seed=1)
    q[r:] = 0.0
    for k_attn in (512, 32):
        res = O.spark_attention_head(q, K, V, k_attn, r)
        tq = torch.from_numpy(q[:r])[None, None, None, :]
        tk = torch.from_numpy(K[:r].T.copy())[None, None]
        tv = torch.from_numpy(V.T.copy())[None, None]
        am = torch.from_numpy(res["mask"])[None, None, None, :]
        ref = torch.nn.functional.scaled_dot_product_attention(tq, tk, tv, attn_mask=am, scale=1.0)
        np.testing.assert_allclose(res["o"], math.log(2.0) * ref[0, 0, 0].numpy(), rtol=1e-11, atol=1e-13)
        if k_attn == 32:
            assert 15 < res["mask"].sum() < 55
            s = K[:r].T @ q[:r]
            top = np.argsort(-s)[: res["mask"].sum()]
            assert set(top.tolist()) == set(np.flatnonzero(res["mask"]).tolist())


def test_attention_general_against_masked_library_ops():
    q, K, V, r = _attn_case(500, seed=2)
    res = O.spark_attention_head(q, K, V, 48, r)
    tq, tK, tV = (torch.from_numpy(a) for a in (q, K, V))
    logits = (tK[:r].T @ tq[:r]).masked_fill(~torch.from_numpy(res["mask"]), float("-inf"))
    w = torch.softmax(logits, 0) * torch.nn.functional.softplus(tK[r:].T @ tq[r:])
    np.testing.assert_allclose(res["o"], (tV @ w).numpy(), rtol=1e-11, atol=1e-13)
    # unselected tokens' K2 and V rows are never needed
    K2z, Vz = K.copy(), V.copy()
    K2z[r:, ~res["mask"]] = 0.0
    Vz[:, ~res["mask"]] = 0.0
    assert np.array_equal(O.spark_attention_head(q, K2z, Vz, 48, r)["o"], res["o"])


def test_attention_empty_selection_and_standard_form():
    hd, n, r = 8, 1024, 4
    K = np.zeros((hd, n))
    K[0] = np.linspace(-1, 1, n)
    q = np.zeros(hd)
    q[0] = 1.0
    res = O.spark_attention_head(q, K, np.ones((hd, n)), 20, r)
    assert not res["mask"].any() and np.all(res["o"] == 0.0)
    q, K, V, _ = _attn_case(77, seed=5)
    ref = torch.nn.functional.scaled_dot_product_attention(
        torch.from_numpy(q)[None, None, None], torch.from_numpy(K.T.copy())[None, None],
        torch.from_numpy(V.T.copy())[None, None], scale=1.0)[0, 0, 0].numpy()
    np.testing.assert_allclose(O.standard_attention_head(q, K, V), ref, rtol=1e-12, atol=1e-14)


def test_attention_grouped_heads_and_window():
    a = synth.attn_inputs(1, 4, 2, 64, 32, 256, [200], "f32", seed=3)
    kc = np.concatenate([a.k1c[0], a.k2c[0]], axis=-1)
    full = O.spark_attention(a.q[0], kc, a.vc[0], 200, 16, 32, window=0)
    same = O.spark_attention(a.q[0], kc, a.vc[0], 200, 16, 32, window=200)
    assert np.array_equal(full["o"], same["o"])
    for h in range(4):
        g = h // 2
        one = O.spark_attention_head(a.q[0, h], kc[g, :200].T, a.vc[0][g, :200].T, 16, 32)
        assert np.array_equal(one["o"], full["o"][h])
    loc = O.spark_attention(a.q[0], kc, a.vc[0], 200, 16, 32, window=50)
    assert not loc["mask"][:, :150].any()
    one = O.spark_attention_head(a.q[0, 3], kc[1, 150:200].T, a.vc[0][1, 150:200].T, 16, 32)
    assert np.array_equal(one["o"], loc["o"][3])


def test_attention_mask_override_branch():
    # the parity harness hands the oracle a selected set of its own when an entry sits within rounding distance of
    # theta: (i) its own set changes nothing; (ii) any other set gives softmax over that set x gate, by library ops
    q, K, V, r = _attn_case(400, seed=7)
    base = O.spark_attention_head(q, K, V, 40, r)
    same = O.spark_attention_head(q, K, V, 40, r, mask_override=base["mask"].copy())
    assert np.array_equal(same["o"], base["o"]) and same["theta"] == base["theta"]
    hand = np.zeros(400, dtype=bool)
    hand[[3, 17, 250, 399]] = True                      # a hand-made set, unrelated to the scores
    got = O.spark_attention_head(q, K, V, 40, r, mask_override=hand)
    tq, tK, tV = (torch.from_numpy(a) for a in (q, K, V))
    logits = (tK[:r].T @ tq[:r]).masked_fill(~torch.from_numpy(hand), float("-inf"))
    w = torch.softmax(logits, 0) * torch.nn.functional.softplus(tK[r:].T @ tq[r:])
    np.testing.assert_allclose(got["o"], (tV @ w).numpy(), rtol=1e-11, atol=1e-13)
    assert np.array_equal(got["mask"], hand) and got["theta"] == base["theta"]
    # one flipped entry moves the output (the override is really used), an empty override attends to nothing
    flip = base["mask"].copy()
    flip[np.flatnonzero(~flip)[0]] = True
    assert not np.array_equal(O.spark_attention_head(q, K, V, 40, r, mask_override=flip)["o"], base["o"])
    assert np.all(O.spark_attention_head(q, K, V, 40, r, mask_override=np.zeros(400, dtype=bool))["o"] == 0.0)
    # short context (k >= n, theta = -inf): the override still restricts the softmax
    q2, K2, V2, _ = _attn_case(30, seed=8)
    m = np.arange(30) % 2 == 0
    got = O.spark_attention_head(q2, K2, V2, 64, r, mask_override=m)
    tq, tK, tV = (torch.from_numpy(a) for a in (q2, K2, V2))
    logits = (tK[:r].T @ tq[:r]).masked_fill(~torch.from_numpy(m), float("-inf"))
    w = torch.softmax(logits, 0) * torch.nn.functional.softplus(tK[r:].T @ tq[r:])
    np.testing.assert_allclose(got["o"], (tV @ w).numpy(), rtol=1e-11, atol=1e-13)
    # through the grouped-head wrapper: per-head overrides over the whole context, cut to the window inside
    a = synth.attn_inputs(1, 4, 2, 64, 32, 256, [200], "f32", seed=3)
    kc = np.concatenate([a.k1c[0], a.k2c[0]], axis=-1)
    loc = O.spark_attention(a.q[0], kc, a.vc[0], 200, 16, 32, window=50)
    again = O.spark_attention(a.q[0], kc, a.vc[0], 200, 16, 32, window=50, mask_override=loc["mask"])
    assert np.array_equal(again["o"], loc["o"])


# ----------------------------------------------------------------------------- FLOP counts the paper prints
def test_flop_counts_match_the_papers_closed_forms():
    d, d_ff, r, k = 2304, 13824, 1024, 1106
    assert O.ffn_flops_dense(d, d_ff) == 2 * r * d_ff + 2 * (d - r) * d_ff + 2 * d * d_ff      # Eq. 3
    assert O.ffn_flops_spark(d, d_ff, r, k) == 2 * (d_ff - k) * r + 4 * d * k                  # Eq. 4
    ratio = O.ffn_flops_spark(d, d_ff, r, k) / O.ffn_flops_dense(d, d_ff)
    assert abs(ratio - 0.2844) < 5e-4                     # "-72 %" in the related-work table
    # r = d/2: d*d_ff + 3*d*k, i.e. 4 / (1 + 3*0.08) = 3.2x
    d2, dff2 = 2048, 16384
    k2 = round(0.08 * dff2)
    assert O.ffn_flops_spark(d2, dff2, d2 // 2, k2) == d2 * dff2 + 3 * d2 * k2
    assert abs(O.ffn_flops_dense(d2, dff2) / O.ffn_flops_spark(d2, dff2, d2 // 2, k2) - 3.2) < 0.03
    # Eq. 8 at r = d_attn/2, and "nearly 4x" at long context
    da, n = 256, 8192
    assert O.attn_flops_spark(da, n, 256, 128) == da * n + 3 * da * 256
    assert O.attn_flops_spark(da, 100, 256, 128) == da * 100 + 3 * da * 100
    assert 3.5 < O.attn_flops_dense(da, n) / O.attn_flops_spark(da, n, 256, 128) < 4.0


# ----------------------------------------------------------------------------- layer pieces
def test_rmsnorm_matches_library():
    h = torch.from_numpy(synth.normal_f32((300,), 1, 1)).double() * 3
    w = torch.from_numpy(synth.normal_f32((300,), 1, 2)).double()
    ref = torch.nn.functional.rms_norm(h, (300,), w, eps=1e-6)
    np.testing.assert_allclose(O.rmsnorm(h.numpy(), w.numpy()), ref.numpy(), rtol=1e-13)


def test_rope_identities():
    rng = np.random.default_rng(0)
    a, b = rng.normal(size=128), rng.normal(size=128)
    assert np.array_equal(O.rope_part(a, 0), a)                           # position 0 is the identity
    assert abs(np.linalg.norm(O.rope_part(a, 1234)) - np.linalg.norm(a)) < 1e-12
    d1 = O.rope_part(a, 907) @ O.rope_part(b, 900)                        # depends on the offset only
    d2 = O.rope_part(a, 12) @ O.rope_part(b, 5)
    assert abs(d1 - d2) < 1e-10
    # pair (i, i + m/2) turns by pos * base^(-2i/m): check one pair as a complex rotation
    i, m, pos = 5, 128, 77
    zc = complex(a[i], a[i + m // 2]) * complex(math.cos(pos * 10000 ** (-2 * i / m)), math.sin(pos * 10000 ** (-2 * i / m)))
    out = O.rope_part(a, pos)
    assert abs(out[i] - zc.real) < 1e-12 and abs(out[i + m // 2] - zc.imag) < 1e-12
    v = rng.normal(size=256)
    sp = O.rope_split(v, 33, 128)
    assert np.array_equal(sp[:128], O.rope_part(v[:128], 33)) and np.array_equal(sp[128:], O.rope_part(v[128:], 33))


def test_round_to_bf16_matches_torch():
    a = synth.normal_f32((5000,), 9, 9)
    ref = torch.from_numpy(a).to(torch.bfloat16).double().numpy()
    assert np.array_equal(O.round_to_bf16(a.astype(np.float64)), ref)


def test_decoder_layer_composition_against_library_ops():
    """With k_ff >= d_ff and ctx_len <= k_attn nothing is thresholded, and the layer is a
    composition of library routines."""
    sh = synth.TINY
    lw = synth.layer_weights(sh, seed=0, layer=0)
    W = {"norm1": lw.norm1, "norm2": lw.norm2,
         "Wqkv": synth.bf16_bits_to_f32(lw.Wqkv_bits), "Wo": synth.bf16_bits_to_f32(lw.Wo_bits),
         "K1t": synth.bf16_bits_to_f32(lw.K1t_bits), "K2t": synth.bf16_bits_to_f32(lw.K2t_bits),
         "Vt": synth.bf16_bits_to_f32(lw.Vt_bits)}
    ctx, cap = 9, 16
    kc = synth.normal_f32((sh.n_kv, cap, sh.hd), 0, 50).astype(np.float64)
    vc = synth.normal_f32((sh.n_kv, cap, sh.hd), 0, 51).astype(np.float64)
    h0 = synth.normal_f32((sh.d,), 0, 52).astype(np.float64)
    kc0, vc0 = kc.copy(), vc.copy()
    out = O.decoder_layer(h0, W, kc, vc, ctx, n_q=sh.n_q, n_kv=sh.n_kv, hd=sh.hd, r_attn=sh.r_attn,
                          k_attn=64, r_ff=sh.r_ff, k_ff=sh.d_ff, cache_bf16=False, gelu_form="erf")
    # the same with torch
    T = lambda a: torch.from_numpy(np.asarray(a, dtype=np.float64))
    h = T(h0)
    a = torch.nn.functional.rms_norm(h, (sh.d,), T(W["norm1"]), eps=1e-6)
    qkv = T(W["Wqkv"]) @ a
    nq, nkv, hd, r = sh.n_q, sh.n_kv, sh.hd, sh.r_attn
    q = qkv[: nq * hd].reshape(nq, hd).numpy()
    kn = qkv[nq * hd:(nq + nkv) * hd].reshape(nkv, hd).numpy()
    vn = qkv[(nq + nkv) * hd:].reshape(nkv, hd)
    q = T(O.rope_split(q, ctx - 1, r)) / math.sqrt(hd)
    kc0[:, ctx - 1] = O.rope_split(kn, ctx - 1, r)
    vc0[:, ctx - 1] = vn.numpy()
    np.testing.assert_allclose(kc0, kc, rtol=1e-12, atol=1e-14)
    np.testing.assert_allclose(vc0, vc, rtol=1e-12, atol=1e-14)
    outs = []
    for hh in range(nq):
        Kh, Vh = T(kc0[hh // (nq // nkv), :ctx]), T(vc0[hh // (nq // nkv), :ctx])
        w = torch.softmax(Kh[:, :r] @ q[hh, :r], 0) * torch.nn.functional.softplus(Kh[:, r:] @ q[hh, r:])
        outs.append(Vh.T @ w)
    h = h + T(W["Wo"]) @ torch.cat(outs)
    b = torch.nn.functional.rms_norm(h, (sh.d,), T(W["norm2"]), eps=1e-6)
    act = torch.nn.functional.gelu(T(W["K1t"]) @ b[: sh.r_ff])
    h = h + T(W["Vt"]).T @ (act * (T(W["K2t"]) @ b[sh.r_ff:]))
    np.testing.assert_allclose(out["h"], h.numpy(), rtol=1e-11, atol=1e-13)


# ---- storage rounding to FP8 E4M3 (used by the quantised-weight FFN; a library routine is the pin) ----------------
def test_decoder_layer_hands_a_mask_override_to_the_attention():
    sh = synth.TINY
    lw = synth.layer_weights(sh, 3, 0)
    W = {"norm1": lw.norm1, "norm2": lw.norm2, "Wqkv": synth.bf16_bits_to_f32(lw.Wqkv_bits), "Wo": synth.bf16_bits_to_f32(lw.Wo_bits),
         "K1t": synth.bf16_bits_to_f32(lw.K1t_bits), "K2t": synth.bf16_bits_to_f32(lw.K2t_bits), "Vt": synth.bf16_bits_to_f32(lw.Vt_bits)}
    kv = synth.attn_inputs(1, sh.n_q, sh.n_kv, sh.hd, sh.r_attn, 128, [100], "bf16", seed=4)
    kc = np.concatenate([kv.k1c[0], kv.k2c[0]], axis=-1).astype(np.float64)
    vc = kv.vc[0].astype(np.float64)
    h = synth.normal_f32((sh.d,), 3, 60)
    kw = dict(n_q=sh.n_q, n_kv=sh.n_kv, hd=sh.hd, r_attn=sh.r_attn, k_attn=sh.k_attn, r_ff=sh.r_ff, k_ff=sh.k_ff)
    base = O.decoder_layer(h, W, kc.copy(), vc.copy(), 100, **kw)
    same = O.decoder_layer(h, W, kc.copy(), vc.copy(), 100, attn_mask_override=base["attn"]["mask"], **kw)
    assert np.array_equal(same["h"], base["h"])
    # the override reaches the attention: it gives what spark_attention gives with it, and a toggled token moves the layer output
    flip = base["attn"]["mask"].copy()
    flip[0, np.flatnonzero(~flip[0])[0]] = True
    other = O.decoder_layer(h, W, kc.copy(), vc.copy(), 100, attn_mask_override=flip, **kw)
    kc2, vc2 = kc.copy(), vc.copy()
    O.decoder_layer(h, W, kc2, vc2, 100, **kw)                      # leaves the appended row in kc2 / vc2
    att = O.spark_attention(base["q"], kc2, vc2, 100, sh.k_attn, sh.r_attn, 0, flip)
    assert np.array_equal(other["attn"]["o"], att["o"])
    assert not np.array_equal(other["h"], base["h"])
    # the storage-rounding hook of the appended key rows: bf16 rounding through it is the default; another rule is what gets stored
    same2 = O.decoder_layer(h, W, kc.copy(), vc.copy(), 100, k_round=O.round_to_bf16, **kw)
    assert np.array_equal(same2["h"], base["h"])
    kc3 = kc.copy()
    O.decoder_layer(h, W, kc3, vc.copy(), 100, k_round=lambda rows: np.round(rows * 4.0) / 4.0, **kw)
    assert np.all(kc3[:, 99] * 4.0 == np.round(kc3[:, 99] * 4.0)) and not np.array_equal(kc3[:, 99], kc2[:, 99])


def test_e4m3_rounding_matches_the_library_cast_and_known_codes():
    import torch
    from paper_2506_06644_b200 import synth
    rng = np.random.default_rng(5)
    x = np.concatenate([rng.standard_normal(50000).astype(np.float32) * s for s in (1e-3, 2e-2, 1.0, 40.0, 200.0)])
    x = np.clip(x, -448.0, 448.0)                      # the library cast does not saturate; the generator does
    ref = torch.from_numpy(x).to(torch.float8_e4m3fn).view(torch.uint8).numpy()
    assert np.array_equal(synth.f32_to_e4m3_bits(x), ref)
    # known codes: 1 = 0x38, largest finite 448 = 0x7e, smallest subnormal 2^-9 = 0x01, smallest normal 2^-6 = 0x08
    known = {1.0: 0x38, 448.0: 0x7E, 2.0 ** -9: 0x01, 2.0 ** -6: 0x08, -2.0: 0xC0, 0.0: 0x00, 1.5: 0x3C}
    got = synth.f32_to_e4m3_bits(np.array(list(known), dtype=np.float32))
    assert got.tolist() == list(known.values())
    # ties go to the even mantissa; beyond the range the value saturates
    ties = synth.f32_to_e4m3_bits(np.array([1.0625, 1.1875, 2.0 ** -10, 3 * 2.0 ** -10, 1000.0, -1e9], dtype=np.float32))
    assert ties.tolist() == [0x38, 0x3A, 0x00, 0x02, 0x7E, 0xFE]
    # decoding all 254 finite codes agrees with the library, and encode(decode(code)) is the identity
    codes = np.arange(256, dtype=np.uint8)
    val = synth.e4m3_bits_to_f32(codes)
    lib = torch.from_numpy(codes).view(torch.float8_e4m3fn).float().numpy()
    fin = ~np.isnan(lib)
    assert fin.sum() == 254 and np.array_equal(val[fin], lib[fin]) and np.all(np.isnan(val[~fin]))
    back = synth.f32_to_e4m3_bits(val[fin])
    assert np.array_equal(back & 0x7F, codes[fin] & 0x7F) and np.array_equal(back[val[fin] != 0], codes[fin][val[fin] != 0])


def test_row_scaled_e4m3_quantisation_error_bound():
    from paper_2506_06644_b200 import synth
    W = synth.normal_f32((64, 512), 9, 1, 0.02)
    W[3] = 0.0
    bits, scale = synth.quantize_rows_e4m3(W)
    deq = synth.e4m3_bits_to_f32(bits) * scale[:, None]
    assert scale[3] == 1.0 and np.all(deq[3] == 0)
    amax = np.abs(W).max(axis=1, keepdims=True)
    # three mantissa bits: relative error <= 2^-4 for normal values; absolute error <= half a subnormal step (scaled) below
    err = np.abs(deq - W)
    bound = np.maximum(np.abs(W) * 2.0 ** -4, (amax / 448.0) * 2.0 ** -10)
    assert np.all(err <= bound * (1 + 1e-6))
    assert np.all(np.abs(deq).max(axis=1) <= amax[:, 0] * (1 + 1e-6))


# ---- sharded statistical top-k (appendix on distributed training) ----------------------------------------
def test_combined_moments_hand_example_and_library():
    # parts [1, 2, 3] and [4 .. 8]: eight values, mean 4.5, sum of squared deviations 42 (by hand)
    parts = [O.shard_moments(np.array([1.0, 2.0, 3.0])), O.shard_moments(np.array([4.0, 5.0, 6.0, 7.0, 8.0]))]
    assert parts[0] == (3.0, 2.0, 2.0) and parts[1] == (5.0, 6.0, 10.0)
    assert O.combine_moments(parts) == (8.0, 4.5, 42.0)
    rng = np.random.default_rng(11)
    x = rng.normal(3.0, 2.0, size=5000)
    cuts = [0, 17, 1200, 1201, 4000, 5000]
    n, mean, m2 = O.combine_moments([O.shard_moments(x[a:b]) for a, b in zip(cuts[:-1], cuts[1:])])
    assert n == 5000 and mean == pytest.approx(np.mean(x), rel=1e-13)
    assert m2 / (n - 1) == pytest.approx(np.var(x, ddof=1), rel=1e-12)


@pytest.mark.parametrize("m", [2, 3, 8])
def test_global_sharded_topk_equals_the_unsharded_operator(m):
    # the appendix's claim: the output is exactly that of statistical top-k without sharding
    rng = np.random.default_rng(m)
    x = rng.normal(size=4096) + np.repeat(rng.normal(size=m), -(-4096 // m))[:4096]      # parts with different means
    cuts = np.concatenate([[0], np.sort(rng.choice(np.arange(1, 4096), size=m - 1, replace=False)), [4096]])
    shards = [x[a:b] for a, b in zip(cuts[:-1], cuts[1:])]
    for fill in ("zero", "neginf"):
        theta, masks, outs = O.stat_topk_sharded_global(shards, 300, fill)
        ref_theta, ref_mask, ref_out = O.stat_topk(x, 300, fill)
        assert theta == pytest.approx(ref_theta, rel=1e-12)
        assert np.array_equal(np.concatenate(masks), ref_mask)
        np.testing.assert_allclose(np.concatenate(outs), ref_out, rtol=0, atol=1e-12)
    theta, masks, _ = O.stat_topk_sharded_global(shards, 4096)
    assert theta == -np.inf and all(mk.all() for mk in masks)


def test_local_sharded_topk_is_the_operator_per_part_and_differs_from_global():
    rng = np.random.default_rng(5)
    lo, hi = rng.normal(0.0, 1.0, size=2048), rng.normal(6.0, 1.0, size=2048)       # the second part holds the largest values
    local = O.stat_topk_sharded_local([lo, hi], 200)
    for part, (theta, mask, out) in zip((lo, hi), local):
        ref = O.stat_topk(part, 100)
        assert theta == ref[0] and np.array_equal(mask, ref[1])
    # each part keeps about k / m; the global form takes nothing from the part with the smaller values (how many it
    # takes from the other is no longer about k: the mixture is far from Gaussian)
    assert abs(int(local[0][1].sum()) - 100) < 40 and abs(int(local[1][1].sum()) - 100) < 40
    _, gmasks, _ = O.stat_topk_sharded_global([lo, hi], 200)
    assert gmasks[0].sum() == 0 and gmasks[1].sum() > 0 and local[0][1].sum() > 0
    # k not divisible by m: k' = floor(k / m), never below one
    assert O.stat_topk_sharded_local([lo, hi], 201)[0][0] == local[0][0]
    assert O.stat_topk_sharded_local([lo, hi, lo, hi], 3)[0][0] == O.stat_topk(lo, 1)[0]
