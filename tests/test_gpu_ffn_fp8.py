"""GPU parity: spark_ffn_decode_fp8 (FP8 E4M3 weights, one scale per neuron, one to four tokens) against the CPU oracle
run on the dequantised weights (both sides read the same stored bits and scales)."""
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


def quantised(d, d_ff, r, k, seed):
    p = synth.ffn_inputs(d, d_ff, r, k, 1, "f32", seed=seed)
    q = {}
    for name in ("K1t", "K2t", "Vt"):
        bits, scale = synth.quantize_rows_e4m3(getattr(p, name))
        q[name] = (bits, scale, synth.e4m3_bits_to_f32(bits).astype(np.float64) * scale[:, None].astype(np.float64))
    return p, q


def run(ctx, p, q, k, flags=0):
    dev = {n: (torch.from_numpy(b).cuda(), torch.from_numpy(s).cuda()) for n, (b, s, _) in q.items()}
    x = torch.from_numpy(p.x).cuda()
    y = torch.full((1, p.d), float("nan"), device="cuda")
    theta = torch.full((1,), 77.0, device="cuda")
    count = torch.full((1,), -5, dtype=torch.int32, device="cuda")
    idx = torch.full((1, p.d_ff), -1, dtype=torch.int32, device="cuda")
    S.spark_ffn_decode_fp8(ctx, x, 1, dev["K1t"][0], dev["K1t"][1], dev["K2t"][0], dev["K2t"][1], dev["Vt"][0], dev["Vt"][1],
                           p.d, p.d_ff, p.r, k, flags, y, theta, count, idx)
    torch.cuda.synchronize()
    return y.cpu().numpy()[0], float(theta[0]), int(count[0]), idx.cpu().numpy()[0]


@pytest.mark.parametrize("d,d_ff,r,k", [(2304, 9216, 1024, 737), (256, 1024, 128, 82), (264, 1000, 136, 80), (3584, 14336, 1792, 1147)])
def test_fp8_weights_against_oracle(ctx, d, d_ff, r, k):
    p, q = quantised(d, d_ff, r, k, seed=31)
    y, theta, count, idx = run(ctx, p, q, k)
    ref = O.spark_ffn(p.x[0], q["K1t"][2].T, q["K2t"][2].T, q["Vt"][2].T, k, r, "tanh")
    _, std = O.mean_std(ref["s"])
    parity.check_theta(theta, ref["theta"], std, "theta")
    diff = parity.check_set(idx[:count], ref["mask"], ref["s"], ref["theta"], std, "set")
    assert diff.size <= 2 and np.all(idx[count:] == -1)
    # the stored values are exact on both sides (fp8 times an fp32 scale): the fp32 bar applies
    parity.check_output(y, ref["y"], "f32", "y")
    # quantisation itself moves the result by a few percent of its RMS: say how much (not a parity statement)
    full = O.spark_ffn(p.x[0], p.K1t.T, p.K2t.T, p.Vt.T, k, r, "tanh")
    assert parity.rms(ref["y"] - full["y"]) < 0.2 * parity.rms(full["y"])
    dense = run(ctx, p, q, k, flags=S.SPARK_DENSE_LOADS)
    np.testing.assert_allclose(dense[0], y, rtol=0, atol=1e-5 * parity.rms(y))
    assert dense[1] == theta and dense[2] == count


@pytest.mark.parametrize("B", [2, 3, 4])
@pytest.mark.parametrize("d,d_ff,r,k", [(2304, 9216, 1024, 737), (256, 1024, 128, 82), (264, 1000, 136, 80)])
def test_fp8_weights_two_to_four_tokens(ctx, B, d, d_ff, r, k):
    p = synth.ffn_inputs(d, d_ff, r, k, B, "f32", seed=40 + B)
    q = {}
    for name in ("K1t", "K2t", "Vt"):
        bits, scale = synth.quantize_rows_e4m3(getattr(p, name))
        q[name] = (bits, scale, synth.e4m3_bits_to_f32(bits).astype(np.float64) * scale[:, None].astype(np.float64))
    dev = {n: (torch.from_numpy(b).cuda(), torch.from_numpy(s).cuda()) for n, (b, s, _) in q.items()}
    x = torch.from_numpy(p.x).cuda()
    for flags in (0, S.SPARK_DENSE_LOADS):
        y = torch.full((B, d), float("nan"), device="cuda")
        theta = torch.full((B,), 77.0, device="cuda")
        count = torch.full((B,), -5, dtype=torch.int32, device="cuda")
        idx = torch.full((B, d_ff), -1, dtype=torch.int32, device="cuda")
        S.spark_ffn_decode_fp8(ctx, x, B, dev["K1t"][0], dev["K1t"][1], dev["K2t"][0], dev["K2t"][1], dev["Vt"][0], dev["Vt"][1],
                               d, d_ff, r, k, flags, y, theta, count, idx)
        torch.cuda.synchronize()
        for b in range(B):
            ref = O.spark_ffn(p.x[b], q["K1t"][2].T, q["K2t"][2].T, q["Vt"][2].T, k, r, "tanh")
            _, std = O.mean_std(ref["s"])
            parity.check_theta(float(theta[b]), ref["theta"], std, f"token {b}")
            got = idx[b, : int(count[b])].cpu().numpy()
            assert parity.check_set(got, ref["mask"], ref["s"], ref["theta"], std, f"token {b}").size <= 2
            parity.check_output(y[b].cpu().numpy(), ref["y"], "f32", f"token {b}")


def test_fp8_needs_scales_and_at_most_four_tokens(ctx):
    p, q = quantised(256, 1024, 128, 82, seed=1)
    dev = {n: (torch.from_numpy(b).cuda(), torch.from_numpy(s).cuda()) for n, (b, s, _) in q.items()}
    x = torch.zeros(5, 256, device="cuda")
    y = torch.zeros(5, 256, device="cuda")
    with pytest.raises(S.SparkError) as e:
        S.spark_ffn_decode_fp8(ctx, x, 5, dev["K1t"][0], dev["K1t"][1], dev["K2t"][0], dev["K2t"][1], dev["Vt"][0], dev["Vt"][1],
                               256, 1024, 128, 82, 0, y, None, None, None)
    assert e.value.status == S.SPARK_ERR_UNSUPPORTED
    with pytest.raises(S.SparkError) as e:
        S.spark_ffn_decode_fp8(ctx, x, 1, dev["K1t"][0], None, dev["K2t"][0], dev["K2t"][1], dev["Vt"][0], dev["Vt"][1],
                               256, 1024, 128, 82, 0, y, None, None, None)
    assert e.value.status == S.SPARK_ERR_INVALID_ARG
