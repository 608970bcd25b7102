"""GPU parity: spark_dense_gemv and spark_layer_decode through the C ABI against the CPU oracle."""
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
    c = S.SparkContext(0, max_batch=16, max_cap=16384, n_q=16, hd=256)
    yield c
    assert c.device_status() == S.SPARK_OK
    c.close()


def bf16_dev(bits):
    return torch.from_numpy(bits.view(np.int16)).cuda().view(torch.bfloat16)


@pytest.mark.parametrize("wd", ["bf16", "f32"])
@pytest.mark.parametrize("B,n_in,n_out", [(1, 2304, 4096), (1, 2048, 2304), (4, 256, 1000), (16, 3584, 300),
                                          (7, 64, 5), (2, 1024, 20000),
                                          (5, 2304, 4096), (12, 2048, 2304),      # five and more tokens: tensor cores (tcgen05 GEMM)
                                          (20, 2304, 4096), (64, 2048, 2304),     # more than one sixteen-token group
                                          (9, 96, 200), (40, 96, 200),            # shapes the GEMM does not take: mma.sync kernel
                                          (8, 264, 500)])                          # ... unless n_in % 32 != 0
def test_dense_gemv(ctx, wd, B, n_in, n_out):
    W = synth.normal_f32((n_out, n_in), 3, 1, 1 / np.sqrt(n_in))
    x = synth.normal_f32((B, n_in), 3, 2)
    add = synth.normal_f32((B, n_out), 3, 3)
    if wd == "bf16":
        bits = synth.f32_to_bf16_bits(W)
        W = synth.bf16_bits_to_f32(bits)
        Wd = bf16_dev(bits)
    else:
        Wd = torch.from_numpy(W).cuda()
    xd, addd = torch.from_numpy(x).cuda(), torch.from_numpy(add).cuda()
    y = torch.full((B, n_out), float("nan"), device="cuda")
    S.spark_dense_gemv(ctx, xd, B, Wd, S.SPARK_BF16 if wd == "bf16" else S.SPARK_F32, n_in, n_out, None, y)
    ref = x.astype(np.float64) @ W.astype(np.float64).T
    # exact weights either way: fp32 bar, except on the tensor-core path (bf16, five and more tokens, n_in % 32 == 0)
    bar = "split2" if wd == "bf16" and B >= 5 and n_in % 32 == 0 else "f32"
    parity.check_output(y.cpu().numpy(), ref, bar)
    S.spark_dense_gemv(ctx, xd, B, Wd, S.SPARK_BF16 if wd == "bf16" else S.SPARK_F32, n_in, n_out, addd, addd)
    parity.check_output(addd.cpu().numpy(), ref + add, bar)


def make_layer(sh: synth.LayerShape, B, cap, lens, seed, window=0, flags=0):
    lw = synth.layer_weights(sh, seed, 0)
    kv = synth.attn_inputs(B, sh.n_q, sh.n_kv, sh.hd, sh.r_attn, cap, lens, "bf16", seed=seed + 1)
    h0 = synth.normal_f32((B, sh.d), seed, 60)
    dev = dict(norm1=torch.from_numpy(lw.norm1).cuda(), norm2=torch.from_numpy(lw.norm2).cuda(),
               Wqkv=bf16_dev(lw.Wqkv_bits), Wo=bf16_dev(lw.Wo_bits), K1t=bf16_dev(lw.K1t_bits),
               K2t=bf16_dev(lw.K2t_bits), Vt=bf16_dev(lw.Vt_bits))
    cache = dict(k1c=bf16_dev(kv.k1c_bits), k2c=bf16_dev(kv.k2c_bits), vc=bf16_dev(kv.vc_bits))
    cfg = dict(d=sh.d, d_ff=sh.d_ff, r_ff=sh.r_ff, k_ff=sh.k_ff, n_q=sh.n_q, n_kv=sh.n_kv, hd=sh.hd,
               r_attn=sh.r_attn, k_attn=sh.k_attn, window=window, cap=cap, rms_eps=1e-6, rope_base=10000.0, flags=flags)
    return lw, kv, h0, S.make_layer(dev, cfg, cache), cache


def oracle_layer(sh, lw, kv, h0, b, n, window):
    W = {"norm1": lw.norm1, "norm2": lw.norm2, "Wqkv": synth.bf16_bits_to_f32(lw.Wqkv_bits),
         "Wo": synth.bf16_bits_to_f32(lw.Wo_bits), "K1t": synth.bf16_bits_to_f32(lw.K1t_bits),
         "K2t": synth.bf16_bits_to_f32(lw.K2t_bits), "Vt": synth.bf16_bits_to_f32(lw.Vt_bits)}
    kc = np.concatenate([kv.k1c[b], kv.k2c[b]], axis=-1).astype(np.float64)
    vc = kv.vc[b].astype(np.float64)
    out = O.decoder_layer(h0[b], W, kc, vc, n, n_q=sh.n_q, n_kv=sh.n_kv, hd=sh.hd, r_attn=sh.r_attn,
                          k_attn=sh.k_attn, r_ff=sh.r_ff, k_ff=sh.k_ff, window=window)
    return out, kc, vc


def run_layer(ctx, sh, B, cap, lens, seed, window=0, flags=0):
    lw, kv, h0, layer, cache = make_layer(sh, B, cap, lens, seed, window, flags)
    h = torch.from_numpy(h0).cuda()
    cl = torch.tensor(lens, dtype=torch.int32, device="cuda")
    nqkv = (sh.n_q + 2 * sh.n_kv) * sh.hd
    scratch = torch.empty(B * (nqkv + 2 * sh.n_q * sh.hd + sh.d + 2 + sh.n_q), device="cuda")
    S.spark_layer_decode(ctx, layer, cl, h, B, scratch)
    torch.cuda.synchronize()
    return lw, kv, h0, h.cpu().numpy(), cache


@pytest.mark.parametrize("shape,B,cap,lens,window", [
    (synth.TINY, 1, 64, [40], 0),
    (synth.TINY, 3, 128, [128, 1, 17], 0),
    (synth.TINY, 2, 128, [100, 90], 32),
    (synth.GEMMA2_2B, 1, 2048, [2048], 0),
    (synth.GEMMA2_2B, 2, 1024, [700, 1024], 512),
    (synth.TINY, 5, 64, [64, 3, 40, 17, 1], 0),                    # five and more tokens: tensor-core projections
    (synth.GEMMA2_2B, 6, 512, [512, 300, 77, 1, 450, 260], 0),
    (synth.GEMMA2_2B, 20, 256, [256, 200, 77, 1, 150, 60, 3, 90, 256, 17, 100, 101, 102, 33, 64, 65, 128, 129, 250, 5], 128),   # more than sixteen sequences
    (synth.GEMMA2_9B, 1, 1024, [1024], 0),                         # 16 query / 8 KV heads, d_ff 14336
    (synth.GEMMA2_9B, 2, 512, [512, 100], 256),
])
def test_layer_against_oracle(ctx, shape, B, cap, lens, window):
    lw, kv, h0, h, cache = run_layer(ctx, shape, B, cap, lens, seed=4, window=window)
    k1 = cache["k1c"].float().cpu().numpy()
    k2 = cache["k2c"].float().cpu().numpy()
    v = cache["vc"].float().cpu().numpy()
    for b in range(B):
        n = lens[b]
        ref, kc, vc = oracle_layer(shape, lw, kv, h0, b, n, window)
        # the appended cache row: equal up to one bf16 rounding step of an fp32-vs-fp64 difference; with five or
        # more tokens the projection's inputs are a two-term bf16 split (16 mantissa bits), an absolute error of
        # about 1e-5 of the row's scale before the rounding
        got_k = np.concatenate([k1[b, :, n - 1], k2[b, :, n - 1]], axis=-1)
        atol = 1e-6 if B < 5 else 1e-4 * parity.rms(kc[:, n - 1])
        np.testing.assert_allclose(got_k, kc[:, n - 1], rtol=2 ** -7, atol=atol)
        np.testing.assert_allclose(v[b, :, n - 1], vc[:, n - 1], rtol=2 ** -7, atol=atol)
        # untouched rows stay untouched
        if n > 1:
            assert np.array_equal(k1[b, :, : n - 1], kv.k1c[b, :, : n - 1])
        parity.check_output(h[b], ref["h"], "bf16", f"seq {b}")
        parity.check_output(h[b] - h0[b], ref["h"] - h0[b], "bf16", f"seq {b} (update only)")


def test_layer_dense_loads_flag_gives_the_same_result(ctx):
    a = run_layer(ctx, synth.TINY, 2, 128, [128, 60], seed=9)
    b = run_layer(ctx, synth.TINY, 2, 128, [128, 60], seed=9, flags=S.SPARK_DENSE_LOADS)
    np.testing.assert_allclose(a[3], b[3], rtol=0, atol=1e-5 * parity.rms(a[3]))
