"""GPU test of spark_ffn_decode_noalloc, the FFN entry point for callers that cannot allocate
device memory (its inter-block state is a fixed array inside the library instead of a workspace
the caller would have to cudaMalloc).  It must give what spark_ffn_decode gives.  The file name
sorts last on purpose: a run that stops at the first failure has then already run everything else.
"""
import numpy as np
import pytest
import torch

from paper_2506_06644_b200 import binding as S
from paper_2506_06644_b200 import synth

pytestmark = pytest.mark.gpu


def _weights(p):
    f = lambda bits: torch.from_numpy(bits.view(np.int16)).cuda().view(torch.bfloat16)
    return f(p.K1t_bits), f(p.K2t_bits), f(p.Vt_bits)


@pytest.mark.parametrize("B", [1, 5])
def test_noalloc_matches_the_workspace_entry_point_twice_in_a_row(B):
    d, d_ff, r, k = 512, 3000, 256, 240
    p = synth.ffn_inputs(d, d_ff, r, k, B, "bf16", seed=21 + B)
    K1t, K2t, Vt = _weights(p)
    x = torch.from_numpy(p.x).cuda()
    ctx = S.SparkContext(0)
    y_ref = torch.empty((B, d), device="cuda")
    th_ref = torch.empty(B, device="cuda")
    S.spark_ffn_decode(ctx, x, B, K1t, K2t, Vt, S.SPARK_BF16, d, d_ff, r, k, 0, y_ref, th_ref, None, None)
    torch.cuda.synchronize()
    assert ctx.device_status() == S.SPARK_OK
    scale = float(y_ref.pow(2).mean().sqrt())
    assert scale > 0
    for call in range(2):                      # the second call runs on the state the first one left
        y = torch.full((B, d), float("nan"), device="cuda")
        th = torch.full((B,), float("nan"), device="cuda")
        S.spark_ffn_decode_noalloc(x, B, K1t, K2t, Vt, S.SPARK_BF16, d, d_ff, r, k, 0, y, th)
        torch.cuda.synchronize()
        # same kernels, same inputs: equal up to the order of the fp32 reductions into y
        assert float((th - th_ref).abs().max()) <= 1e-6 * max(1.0, float(th_ref.abs().max())), f"call {call}"
        err = float((y - y_ref).abs().max())
        assert err <= 1e-5 * scale, f"call {call}: max|diff| {err:.3e} vs RMS {scale:.3e}"
    ctx.close()


def test_noalloc_rejects_more_tokens_than_its_static_state_serves():
    d, d_ff, r = 64, 128, 32
    B = 17
    x = torch.zeros((B, d), device="cuda")
    w1 = torch.zeros((d_ff, r), device="cuda")
    w2 = torch.zeros((d_ff, d - r), device="cuda")
    v = torch.zeros((d_ff, d), device="cuda")
    y = torch.zeros((B, d), device="cuda")
    with pytest.raises(S.SparkError) as e:
        S.spark_ffn_decode_noalloc(x, B, w1, w2, v, S.SPARK_F32, d, d_ff, r, 10, 0, y, None)
    assert e.value.status == S.SPARK_ERR_UNSUPPORTED
