"""GPU tests of the failure path, made without faulting, trapping or hanging anything: a bounded wait between thread blocks is
made to run out by a host-side test hook (the kernel waits for one arrival more than its grid has blocks, with a wait limit of
a fraction of a millisecond), returns by itself, and the host reads SPARK_ERR_TIMEOUT, after which the context works again.
Also the SPARK_CHECK_FINITE debugging flag."""
import numpy as np
import pytest
import torch

from oracle import spark_oracle as O
from paper_2506_06644_b200 import binding as S
from paper_2506_06644_b200 import synth
from tests import parity

pytestmark = pytest.mark.gpu


def _ffn_case(seed):
    d, d_ff, r, k = 512, 3000, 256, 240
    p = synth.ffn_inputs(d, d_ff, r, k, 1, "bf16", seed=seed)
    f = lambda bits: torch.from_numpy(bits.view(np.int16)).cuda().view(torch.bfloat16)
    return p, (d, d_ff, r, k), (f(p.K1t_bits), f(p.K2t_bits), f(p.Vt_bits)), torch.from_numpy(p.x).cuda()


def _check_against_oracle(p, dims, y, th):
    d, d_ff, r, k = dims
    ref = O.spark_ffn(p.x[0], p.K1t.astype(np.float64).T, p.K2t.astype(np.float64).T, p.Vt.astype(np.float64).T, k, r)
    parity.check_theta(float(th[0]), ref["theta"], float(np.std(ref["s"], ddof=1)))
    parity.check_output(y.cpu().numpy()[0], ref["y"], "bf16")


@pytest.mark.parametrize("overlap", [False, True])
def test_a_wait_that_runs_out_is_reported_and_the_context_recovers(overlap):
    p, dims, (K1t, K2t, Vt), x = _ffn_case(31)
    d, d_ff, r, k = dims
    ctx = S.SparkContext(0, max_batch=1, max_dff=d_ff, max_d=d)
    ctx.set_launch_overlap(overlap)
    y = torch.empty((1, d), device="cuda")
    th = torch.empty(1, device="cuda")
    S.spark_ffn_decode(ctx, x, 1, K1t, K2t, Vt, S.SPARK_BF16, d, d_ff, r, k, 0, y, th, None, None)
    assert ctx.device_status() == S.SPARK_OK
    _check_against_oracle(p, dims, y, th)

    ctx.set_wait_limit(200_000)                 # about 0.1 ms of SM cycles instead of two seconds
    ctx.debug_expect_arrivals(1)                # one arrival that no block delivers
    S.spark_ffn_decode(ctx, x, 1, K1t, K2t, Vt, S.SPARK_BF16, d, d_ff, r, k, 0, y, th, None, None)
    torch.cuda.synchronize()                    # the kernel ended by itself
    assert ctx.device_status() == S.SPARK_ERR_TIMEOUT
    assert ctx.device_status() == S.SPARK_OK    # reading the status cleared it and reset the workspace

    ctx.debug_expect_arrivals(0)
    for _ in range(3):                          # ordinary calls work again (the wait limit survived the reset)
        y.fill_(float("nan"))
        S.spark_ffn_decode(ctx, x, 1, K1t, K2t, Vt, S.SPARK_BF16, d, d_ff, r, k, 0, y, th, None, None)
        assert ctx.device_status() == S.SPARK_OK
        _check_against_oracle(p, dims, y, th)
    ctx.set_wait_limit(0)
    S.spark_ffn_decode(ctx, x, 1, K1t, K2t, Vt, S.SPARK_BF16, d, d_ff, r, k, 0, y, th, None, None)
    assert ctx.device_status() == S.SPARK_OK
    _check_against_oracle(p, dims, y, th)
    ctx.close()


def test_wait_limit_argument_errors():
    ctx = S.SparkContext(0, max_batch=1)
    with pytest.raises(S.SparkError):
        ctx.set_wait_limit(-1)
    with pytest.raises(S.SparkError):
        ctx.debug_expect_arrivals(-1)
    ctx.close()


def test_check_finite_flag_reports_a_nan_that_reached_the_predictor():
    p, dims, (K1t, K2t, Vt), x = _ffn_case(32)
    d, d_ff, r, k = dims
    ctx = S.SparkContext(0, max_batch=1, max_dff=d_ff, max_d=d)
    y = torch.empty((1, d), device="cuda")
    th = torch.empty(1, device="cuda")
    S.spark_ffn_decode(ctx, x, 1, K1t, K2t, Vt, S.SPARK_BF16, d, d_ff, r, k, S.SPARK_CHECK_FINITE, y, th, None, None)
    assert ctx.device_status() == S.SPARK_OK
    _check_against_oracle(p, dims, y, th)
    bad = x.clone()
    bad[0, 7] = float("nan")
    S.spark_ffn_decode(ctx, bad, 1, K1t, K2t, Vt, S.SPARK_BF16, d, d_ff, r, k, 0, y, th, None, None)
    assert ctx.device_status() == S.SPARK_OK                      # without the flag nothing is reported
    S.spark_ffn_decode(ctx, bad, 1, K1t, K2t, Vt, S.SPARK_BF16, d, d_ff, r, k, S.SPARK_CHECK_FINITE, y, th, None, None)
    assert ctx.device_status() == S.SPARK_ERR_NONFINITE
    S.spark_ffn_decode(ctx, x, 1, K1t, K2t, Vt, S.SPARK_BF16, d, d_ff, r, k, S.SPARK_CHECK_FINITE, y, th, None, None)
    assert ctx.device_status() == S.SPARK_OK
    _check_against_oracle(p, dims, y, th)
    # attention: an infinite query component
    a = synth.attn_inputs(1, 4, 2, 64, 32, 512, [400], "bf16", seed=6)
    bf = lambda bits: torch.from_numpy(bits.view(np.int16)).cuda().view(torch.bfloat16)
    k1c, k2c, vc = bf(a.k1c_bits), bf(a.k2c_bits), bf(a.vc_bits)
    q = torch.from_numpy(a.q).cuda()
    o = torch.empty(1, 4, 64, device="cuda")
    cl = torch.tensor([400], dtype=torch.int32, device="cuda")
    actx = S.SparkContext(0, max_batch=1, max_cap=512, n_q=4, hd=64)
    S.spark_attn_decode(actx, q, k1c, k2c, vc, S.SPARK_BF16, 1, 4, 2, 64, 32, 512, cl, 0, 16, S.SPARK_CHECK_FINITE, o, None, None, None, 0)
    assert actx.device_status() == S.SPARK_OK
    q[0, 1, 3] = float("inf")
    S.spark_attn_decode(actx, q, k1c, k2c, vc, S.SPARK_BF16, 1, 4, 2, 64, 32, 512, cl, 0, 16, S.SPARK_CHECK_FINITE, o, None, None, None, 0)
    assert actx.device_status() == S.SPARK_ERR_NONFINITE
    actx.close()
    ctx.close()
