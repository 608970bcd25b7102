"""GPU parity: spark_ffn_decode through the C ABI against the CPU oracle."""
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


def upload(p: synth.FfnInputs):
    if p.wdtype == "bf16":
        f = lambda bits: torch.from_numpy(bits.view(np.int16)).cuda().view(torch.bfloat16)
        return f(p.K1t_bits), f(p.K2t_bits), f(p.Vt_bits)
    return tuple(torch.from_numpy(a).cuda() for a in (p.K1t, p.K2t, p.Vt))


def run_ffn(ctx, p: synth.FfnInputs, k=None, flags=0, want_idx=True, weights=None):
    k = p.k if k is None else k
    B = p.x.shape[0]
    K1t, K2t, Vt = weights if weights is not None else upload(p)
    x = torch.from_numpy(p.x).cuda()
    y = torch.full((B, p.d), float("nan"), device="cuda")
    theta = torch.full((B,), 77.0, device="cuda")
    count = torch.full((B,), -5, dtype=torch.int32, device="cuda") if want_idx else None
    idx = torch.full((B, p.d_ff), -1, dtype=torch.int32, device="cuda") if want_idx else None
    S.spark_ffn_decode(ctx, x, B, K1t, K2t, Vt, S.SPARK_BF16 if p.wdtype == "bf16" else S.SPARK_F32,
                       p.d, p.d_ff, p.r, k, flags, y, theta, count, idx)
    torch.cuda.synchronize()
    return (y.cpu().numpy(), theta.cpu().numpy(),
            count.cpu().numpy() if want_idx else None, idx.cpu().numpy() if want_idx else None)


def oracle_ffn(p, b, k=None, form="tanh"):
    return O.spark_ffn(p.x[b], p.K1t.T, p.K2t.T, p.Vt.T, p.k if k is None else k, p.r, form)


def compare(p, out, k=None, form="tanh"):
    y, theta, count, idx = out
    worst = 0.0
    for b in range(p.x.shape[0]):
        ref = oracle_ffn(p, b, k, form)
        _, std = O.mean_std(ref["s"])
        parity.check_theta(theta[b], ref["theta"], std, f"token {b}")
        if idx is not None:
            got = idx[b, : count[b]]
            diff = parity.check_set(got, ref["mask"], ref["s"], ref["theta"], std, f"token {b}")
            assert np.all(idx[b, count[b]:] == -1)
            assert diff.size <= 2
        worst = max(worst, parity.check_output(y[b], ref["y"], p.wdtype, f"token {b}"))
    return worst


def test_tiny_fp32_layer(ctx):
    # d=256, d_ff=1024, r=128, k=82, one token, fp32 weights
    p = synth.ffn_inputs(256, 1024, 128, 82, 1, "f32", seed=0)
    for flags, form in ((S.SPARK_GELU_TANH, "tanh"), (S.SPARK_GELU_ERF, "erf")):
        compare(p, run_ffn(ctx, p, flags=flags), form=form)


@pytest.mark.parametrize("B", [1, 2, 3, 4, 8, 16])     # 1: one-token kernel; 2-4: few-token kernel; 8, 16: tcgen05 chunk kernels
def test_gemma2_2b_shape_bf16(ctx, B):
    p = synth.ffn_inputs(2304, 9216, 1024, 737, B, "bf16", seed=0)
    w = upload(p)
    out = run_ffn(ctx, p, weights=w)
    err = compare(p, out)
    assert err < 5e-3                              # well inside the 2e-2 bar
    assert np.all(np.abs(out[2] - 737) < 6 * 16.5 + 1)
    dense = run_ffn(ctx, p, flags=S.SPARK_DENSE_LOADS, weights=w)
    np.testing.assert_allclose(dense[0], out[0], rtol=0, atol=1e-5 * parity.rms(out[0]))
    assert np.array_equal(dense[1], out[1]) and np.array_equal(dense[2], out[2])
    again = run_ffn(ctx, p, weights=w, want_idx=False)          # optional outputs may be absent
    np.testing.assert_allclose(again[0], out[0], rtol=0, atol=1e-5 * parity.rms(out[0]))


@pytest.mark.parametrize("d,d_ff,r,k,B,form", [(2304, 9216, 1024, 737, 17, "tanh"), (2304, 9216, 1152, 737, 40, "tanh"),
                                              (2304, 9216, 1024, 737, 64, "erf"), (3584, 14336, 1792, 1147, 24, "tanh"),
                                              (256, 1024, 128, 82, 33, "tanh"), (512, 2048, 64, 164, 20, "tanh")])
def test_token_chunks_on_the_tensor_cores(ctx, d, d_ff, r, k, B, form):
    # TMA-fed tcgen05 kernels that read every weight row (the union of the active sets covers most); shapes with one and
    # two partial K2 products, 9B shape, token counts that fill 2, 3 and 4 sixteen-token groups
    p = synth.ffn_inputs(d, d_ff, r, k, B, "bf16", seed=B)
    w = upload(p)
    out = run_ffn(ctx, p, weights=w, flags=S.SPARK_GELU_ERF if form == "erf" else S.SPARK_GELU_TANH)
    assert compare(p, out, form=form) < 5e-3
    again = run_ffn(ctx, p, weights=w, want_idx=False, flags=S.SPARK_GELU_ERF if form == "erf" else S.SPARK_GELU_TANH)
    np.testing.assert_allclose(again[0], out[0], rtol=0, atol=1e-5 * parity.rms(out[0]))
    assert np.array_equal(again[1], out[1])


def test_gemma2_9b_shape_bf16(ctx):
    p = synth.ffn_inputs(3584, 14336, 1792, 1147, 2, "bf16", seed=1)
    compare(p, run_ffn(ctx, p))


@pytest.mark.parametrize("wdtype", ["f32", "bf16"])
@pytest.mark.parametrize("d,d_ff,r,k,B", [(64, 100, 8, 9, 1), (264, 1000, 136, 80, 3), (512, 3001, 256, 240, 7),
                                           (128, 150, 64, 20, 20), (1024, 40000, 512, 1000, 2)])
def test_ragged_shapes(ctx, wdtype, d, d_ff, r, k, B):
    # fewer neurons than thread blocks, neuron counts that do not divide, batches that do not
    # fill a token group, and more tokens than one group holds
    p = synth.ffn_inputs(d, d_ff, r, k, B, wdtype, seed=d_ff)
    compare(p, run_ffn(ctx, p))


def test_k_ge_dff_is_the_dense_gelu_ffn(ctx):
    p = synth.ffn_inputs(256, 1024, 128, 82, 2, "f32", seed=2)
    y, theta, count, idx = run_ffn(ctx, p, k=1024)
    assert np.all(np.isneginf(theta)) and np.all(count == 1024)
    x = torch.from_numpy(p.x).double()
    K1t, K2t, Vt = (torch.from_numpy(a).double() for a in (p.K1t, p.K2t, p.Vt))
    for b in range(2):
        act = torch.nn.functional.gelu(K1t @ x[b, :128], approximate="tanh")
        ref = Vt.T @ (act * (K2t @ x[b, 128:]))
        parity.check_output(y[b], ref.numpy(), "f32")
        assert sorted(idx[b].tolist()) == list(range(1024))


def test_zeroing_inactive_rows_changes_nothing(ctx):
    p = synth.ffn_inputs(512, 2048, 256, 164, 2, "bf16", seed=3)
    base = run_ffn(ctx, p)
    keep = np.zeros(p.d_ff, dtype=bool)
    for b in range(2):
        keep[base[3][b, : base[2][b]]] = True
    p.K2t_bits[~keep] = 0
    p.Vt_bits[~keep] = 0
    zeroed = run_ffn(ctx, p)
    np.testing.assert_allclose(zeroed[0], base[0], rtol=0, atol=1e-5 * parity.rms(base[0]))
    # garbage (NaN bit patterns) in the inactive rows must not be read into the result either
    p.K2t_bits[~keep] = 0x7FC0
    p.Vt_bits[~keep] = 0x7FC0
    poisoned = run_ffn(ctx, p)
    np.testing.assert_allclose(poisoned[0], base[0], rtol=0, atol=1e-5 * parity.rms(base[0]))


def test_tie_example_and_empty_selection(ctx):
    # scores with evenly spaced values: theta lies above the maximum, nothing is selected, y = 0
    d, d_ff, r = 16, 1024, 8
    K1t = np.zeros((d_ff, r), dtype=np.float32)
    K1t[:, 0] = np.linspace(-1, 1, d_ff)
    p = synth.ffn_inputs(d, d_ff, r, 20, 1, "f32", seed=0)
    p.K1t = K1t
    p.x[0, :r] = 0
    p.x[0, 0] = 1.0
    y, theta, count, idx = run_ffn(ctx, p)
    assert count[0] == 0 and np.all(y == 0.0) and abs(theta[0] - 1.1931251) < 2e-5


def test_argument_errors(ctx):
    p = synth.ffn_inputs(64, 128, 32, 10, 1, "f32", seed=0)
    K1t, K2t, Vt = upload(p)
    x = torch.from_numpy(p.x).cuda()
    y = torch.empty((1, 64), device="cuda")

    def call(**kw):
        a = dict(B=1, d=64, d_ff=128, r=32, k=10, wd=S.SPARK_F32)
        a.update(kw)
        S.spark_ffn_decode(ctx, x, a["B"], K1t, K2t, Vt, a["wd"], a["d"], a["d_ff"], a["r"], a["k"], 0, y, None, None, None)

    for bad, code in ((dict(k=0), 1), (dict(r=0), 1), (dict(r=64), 1), (dict(B=0), 1), (dict(B=65), 1),
                      (dict(r=36), 2), (dict(wd=9), 2)):
        with pytest.raises(S.SparkError) as e:
            call(**bad)
        assert e.value.status == code, bad
    call()
    torch.cuda.synchronize()


@pytest.mark.parametrize("seed", range(6))
def test_seeded_random_shapes_of_the_chunk_path(ctx, seed):
    # widths, predictor splits (r close to 0 and close to d), neuron counts, token counts and k from a seeded generator
    rng = np.random.default_rng(500 + seed)
    d = 256 * int(rng.integers(1, 4)); r = 64 * int(rng.integers(1, d // 64)); d_ff = 128 * int(rng.integers(2, 24)); B = int(rng.integers(5, 65))
    k = max(1, int(d_ff * float(rng.choice([0.02, 0.08, 0.3]))))
    p = synth.ffn_inputs(d, d_ff, r, k, B, "bf16", seed=600 + seed)
    out = run_ffn(ctx, p, weights=upload(p))
    assert compare(p, out) < 5e-3
