"""GPU parity of spark_layer_decode with quantised storage: FP8 E4M3 FFN weights with per-neuron scales (SPARK_FFN_FP8) and an FP8
predictor slice of the cache with per-row scales (SPARK_K1C_FP8), against the CPU oracle run on the dequantised values.  The
storage rounding (E4M3 codes and scales) lives with the input generators; the oracle's layer gets it as its storage-rounding hook
for the appended row."""
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
    c = S.SparkContext(0, max_batch=8, max_cap=8192, n_q=16, hd=256)
    yield c
    assert c.device_status() == S.SPARK_OK
    c.close()


def bf16_dev(bits):
    return torch.from_numpy(bits.view(np.int16)).cuda().view(torch.bfloat16)


def quant_rows(a2d):
    bits, scale = synth.quantize_rows_e4m3(a2d)
    return bits, scale, synth.e4m3_bits_to_f32(bits).astype(np.float64) * scale[:, None].astype(np.float64)


def k1_round(rows, r):
    """Storage rounding of appended key rows [n_kv][hd]: the first r values as e4m3 with a row scale, the rest as bf16."""
    out = O.round_to_bf16(rows)
    _, _, deq = quant_rows(np.asarray(rows[:, :r], dtype=np.float32))
    out[:, :r] = deq
    return out


@pytest.mark.parametrize("shape,B,cap,lens,window,ffn8,k18", [
    (synth.TINY, 1, 128, [100], 0, True, True),
    (synth.TINY, 3, 128, [128, 1, 17], 32, True, True),
    (synth.GEMMA2_2B, 1, 2048, [2048], 0, True, True),
    (synth.GEMMA2_2B, 1, 2048, [1500], 0, False, True),
    (synth.GEMMA2_2B, 2, 1024, [700, 1024], 512, True, False),
    (synth.GEMMA2_2B, 8, 1024, [1024, 300, 77, 1, 450, 260, 1000, 512], 0, False, True),      # tensor-core projections, separate append kernel
    (synth.GEMMA2_9B, 1, 1024, [1024], 0, True, True),
])
def test_layer_with_fp8_storage_against_oracle(ctx, shape, B, cap, lens, window, ffn8, k18):
    sh = shape
    lw = synth.layer_weights(sh, 7, 0)
    kv = synth.attn_inputs(B, sh.n_q, sh.n_kv, sh.hd, sh.r_attn, cap, lens, "bf16", seed=8)
    h0 = synth.normal_f32((B, sh.d), 7, 60)
    W = {"norm1": lw.norm1, "norm2": lw.norm2, "Wqkv": synth.bf16_bits_to_f32(lw.Wqkv_bits), "Wo": synth.bf16_bits_to_f32(lw.Wo_bits),
         "K1t": synth.bf16_bits_to_f32(lw.K1t_bits), "K2t": synth.bf16_bits_to_f32(lw.K2t_bits), "Vt": synth.bf16_bits_to_f32(lw.Vt_bits)}
    dev = dict(norm1=torch.from_numpy(lw.norm1).cuda(), norm2=torch.from_numpy(lw.norm2).cuda(), Wqkv=bf16_dev(lw.Wqkv_bits), Wo=bf16_dev(lw.Wo_bits))
    flags = 0
    if ffn8:
        flags |= S.SPARK_FFN_FP8
        for name in ("K1t", "K2t", "Vt"):
            bits, scale, deq = quant_rows(W[name])
            dev[name] = torch.from_numpy(bits).cuda()
            dev[name[:2] + "s" if name != "Vt" else "Vs"] = torch.from_numpy(scale).cuda()
            W[name] = deq
    else:
        dev.update(K1t=bf16_dev(lw.K1t_bits), K2t=bf16_dev(lw.K2t_bits), Vt=bf16_dev(lw.Vt_bits))
    k1 = kv.k1c.copy()
    cache = dict(k2c=bf16_dev(kv.k2c_bits), vc=bf16_dev(kv.vc_bits))
    if k18:
        flags |= S.SPARK_K1C_FP8
        bits, scale, deq = quant_rows(kv.k1c.reshape(-1, sh.r_attn))
        cache["k1c"] = torch.from_numpy(bits.reshape(kv.k1c.shape)).cuda()
        cache["k1s"] = torch.from_numpy(scale.reshape(kv.k1c.shape[:-1])).cuda()
        k1 = deq.reshape(kv.k1c.shape)
    else:
        cache["k1c"] = bf16_dev(kv.k1c_bits)
    cfg = dict(d=sh.d, d_ff=sh.d_ff, r_ff=sh.r_ff, k_ff=sh.k_ff, n_q=sh.n_q, n_kv=sh.n_kv, hd=sh.hd, r_attn=sh.r_attn, k_attn=sh.k_attn,
               window=window, cap=cap, rms_eps=1e-6, rope_base=10000.0, flags=flags)
    layer = S.make_layer(dev, cfg, cache)
    h = torch.from_numpy(h0).cuda()
    cl = torch.tensor(lens, dtype=torch.int32, device="cuda")
    scratch = torch.empty(S.layer_scratch_floats(dict(n_q=sh.n_q, n_kv=sh.n_kv, hd=sh.hd, d=sh.d), B), device="cuda")
    S.spark_layer_decode(ctx, layer, cl, h, B, scratch)
    torch.cuda.synchronize()
    assert ctx.device_status() == S.SPARK_OK
    got = h.cpu().numpy()
    for b in range(B):
        n = lens[b]
        kc = np.concatenate([k1[b], kv.k2c[b]], axis=-1).astype(np.float64)
        vc = kv.vc[b].astype(np.float64)
        hook = (lambda rows: k1_round(rows, sh.r_attn)) if k18 else None
        last = None
        for ref in parity.layer_refs_within_band(O, h0[b], W, kc, vc, n, window, n_q=sh.n_q, n_kv=sh.n_kv, hd=sh.hd, r_attn=sh.r_attn,
                                                 k_attn=sh.k_attn, r_ff=sh.r_ff, k_ff=sh.k_ff, k_round=hook):
            try:
                parity.check_output(got[b], ref["h"], "bf16", f"seq {b}")
                parity.check_output(got[b] - h0[b], ref["h"] - h0[b], "bf16", f"seq {b} (update only)")
                last = None
                break
            except AssertionError as e:
                last = e
        if last is not None:
            raise last
        if k18:      # the appended predictor row: the oracle's row quantised by the generator's rule, equal up to one code step
            code = cache["k1c"][b, :, n - 1].cpu().numpy()
            sc = cache["k1s"][b, :, n - 1].cpu().numpy()
            deq = synth.e4m3_bits_to_f32(code).astype(np.float64) * sc[:, None]
            want = kc[:, n - 1, : sh.r_attn]
            np.testing.assert_allclose(deq, want, rtol=0.13, atol=0.02 * float(np.abs(want).max()))
            assert np.mean(np.isclose(deq, want, rtol=1e-5, atol=0)) > 0.95      # the same codes; the fp32 scale may differ in its last bit
