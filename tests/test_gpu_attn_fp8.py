"""GPU parity: spark_attn_decode_fp8k (predictor slice of the cache in FP8 E4M3, one scale per cached row; bf16
k2c / vc) against the CPU oracle run on the dequantised slice (both sides read the same stored bits and scales)."""
import dataclasses

import numpy as np
import pytest
import torch

from paper_2506_06644_b200 import binding as S
from paper_2506_06644_b200 import synth
from tests.test_gpu_attn import compare

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def ctx():
    c = S.SparkContext(0, max_batch=8, max_cap=16384, n_q=16, hd=256)
    yield c
    assert c.device_status() == S.SPARK_OK
    c.close()


def run(ctx, a, k_attn, window=0, flags=0):
    B, n_kv, cap, r = a.k1c.shape
    bits, scale = synth.quantize_rows_e4m3(a.k1c.reshape(-1, r))
    deq = (synth.e4m3_bits_to_f32(bits) * scale[:, None]).reshape(a.k1c.shape).astype(np.float32)
    bf = lambda b: torch.from_numpy(b.view(np.int16)).cuda().view(torch.bfloat16)
    k1 = torch.from_numpy(bits.reshape(B, n_kv, cap, r)).cuda()
    k1s = torch.from_numpy(scale.reshape(B, n_kv, cap)).cuda()
    q = torch.from_numpy(a.q).cuda()
    cl = torch.from_numpy(a.ctx_len).cuda()
    idx_cap = int(a.ctx_len.max())
    o = torch.full((B, a.n_q, a.hd), float("nan"), device="cuda")
    theta = torch.full((B, a.n_q), 9.0, device="cuda")
    count = torch.full((B, a.n_q), -3, dtype=torch.int32, device="cuda")
    idx = torch.full((B, a.n_q, idx_cap), -1, dtype=torch.int32, device="cuda")
    S.spark_attn_decode_fp8k(ctx, q, k1, k1s, bf(a.k2c_bits), bf(a.vc_bits), B, a.n_q, a.n_kv, a.hd, a.r, a.cap, cl, window,
                             k_attn, flags, o, theta, count, idx, idx_cap)
    torch.cuda.synchronize()
    return dataclasses.replace(a, k1c=deq), (o.cpu().numpy(), theta.cpu().numpy(), count.cpu().numpy(), idx.cpu().numpy())


@pytest.mark.parametrize("B,n_q,n_kv,hd,r,cap,lens,k_attn,window", [
    (1, 8, 4, 256, 128, 4096, [4096], 256, 0),
    (3, 8, 4, 256, 128, 2048, [2048, 700, 33], 256, 512),
    (8, 16, 8, 256, 128, 1024, [1024, 1000, 900, 512, 300, 100, 17, 1], 64, 0),       # aligned cut
    (2, 4, 4, 64, 32, 300, [300, 150], 16, 0),                                          # r = 32: plain-ALU first pass
    (1, 4, 4, 256, 128, 700, [650], 64, 0),                                             # one query head per KV head
    (2, 16, 4, 256, 128, 500, [500, 77], 32, 128),                                      # four per KV head: plain-ALU first pass
])
def test_fp8_predictor_slice_against_oracle(ctx, B, n_q, n_kv, hd, r, cap, lens, k_attn, window):
    a = synth.attn_inputs(B, n_q, n_kv, hd, r, cap, lens, "bf16", seed=13)
    adeq, out = run(ctx, a, k_attn, window)
    compare(adeq, out, k_attn, window)
    dense = run(ctx, a, k_attn, window, flags=S.SPARK_DENSE_LOADS)[1]
    assert np.array_equal(dense[1], out[1]) and np.array_equal(dense[2], out[2])
    np.testing.assert_allclose(dense[0], out[0], rtol=0, atol=2e-5 * max(1e-30, float(np.abs(out[0]).max())))


def run_kv(ctx, a, k_attn, window=0, flags=0):
    """The whole cache quantised: every tensor's rows as e4m3 with a row scale."""
    B, n_kv, cap, r = a.k1c.shape
    dev, deq = {}, {}
    for name in ("k1c", "k2c", "vc"):
        t = getattr(a, name)
        bits, scale = synth.quantize_rows_e4m3(t.reshape(-1, t.shape[-1]))
        deq[name] = (synth.e4m3_bits_to_f32(bits) * scale[:, None]).reshape(t.shape).astype(np.float32)
        dev[name] = (torch.from_numpy(bits.reshape(t.shape)).cuda(), torch.from_numpy(scale.reshape(t.shape[:-1])).cuda())
    q = torch.from_numpy(a.q).cuda()
    cl = torch.from_numpy(a.ctx_len).cuda()
    idx_cap = int(a.ctx_len.max())
    o = torch.full((B, a.n_q, a.hd), float("nan"), device="cuda")
    theta = torch.full((B, a.n_q), 9.0, device="cuda")
    count = torch.full((B, a.n_q), -3, dtype=torch.int32, device="cuda")
    idx = torch.full((B, a.n_q, idx_cap), -1, dtype=torch.int32, device="cuda")
    S.spark_attn_decode_fp8kv(ctx, q, dev["k1c"][0], dev["k1c"][1], dev["k2c"][0], dev["k2c"][1], dev["vc"][0], dev["vc"][1], B, a.n_q, a.n_kv,
                              a.hd, a.r, a.cap, cl, window, k_attn, flags, o, theta, count, idx, idx_cap)
    torch.cuda.synchronize()
    return dataclasses.replace(a, **deq), (o.cpu().numpy(), theta.cpu().numpy(), count.cpu().numpy(), idx.cpu().numpy())


@pytest.mark.parametrize("B,n_q,n_kv,hd,r,cap,lens,k_attn,window", [
    (1, 8, 4, 256, 128, 4096, [4096], 256, 0),
    (3, 8, 4, 256, 128, 2048, [2048, 700, 33], 256, 512),
    (8, 16, 8, 256, 128, 1024, [1024, 1000, 900, 512, 300, 100, 17, 1], 64, 0),
    (2, 4, 4, 64, 32, 300, [300, 150], 16, 0),
    (2, 16, 4, 256, 128, 500, [500, 77], 32, 128),
])
def test_fp8_whole_cache_against_oracle(ctx, B, n_q, n_kv, hd, r, cap, lens, k_attn, window):
    a = synth.attn_inputs(B, n_q, n_kv, hd, r, cap, lens, "bf16", seed=14)
    adeq, out = run_kv(ctx, a, k_attn, window)
    compare(adeq, out, k_attn, window)
    dense = run_kv(ctx, a, k_attn, window, flags=S.SPARK_DENSE_LOADS)[1]
    assert np.array_equal(dense[1], out[1]) and np.array_equal(dense[2], out[2])
    np.testing.assert_allclose(dense[0], out[0], rtol=0, atol=2e-5 * max(1e-30, float(np.abs(out[0]).max())))
