"""GPU parity of the opt-in execution paths of a one-token layer call: the fused persistent kernel (spark_set_fused_layer;
also through spark_stack_decode, several layers per launch) and the L2 prefetch option, each against the CPU oracle, with and
without launch overlap.  Both options are off by default (they measure slower than the kernel-per-step path on B200)."""
import numpy as np
import pytest
import torch

from oracle import spark_oracle as O
from paper_2506_06644_b200 import binding as S
from paper_2506_06644_b200 import synth
from tests import parity
from tests.test_gpu_layer import make_layer, oracle_layer

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def ctx():
    c = S.SparkContext(0, max_batch=4, max_cap=16384, n_q=16, hd=256)
    yield c
    assert c.device_status() == S.SPARK_OK
    c.close()


@pytest.mark.parametrize("overlap", [False, True])
@pytest.mark.parametrize("shape,cap,n,window", [
    (synth.TINY, 64, 40, 0), (synth.TINY, 128, 1, 0), (synth.TINY, 128, 100, 32), (synth.TINY, 64, 16, 0),
    (synth.GEMMA2_2B, 2048, 2048, 0), (synth.GEMMA2_2B, 1024, 700, 512), (synth.GEMMA2_9B, 1024, 1024, 0),
])
def test_fused_layer_kernel_against_oracle(ctx, shape, cap, n, window, overlap):
    ctx.set_fused_layer(True)
    ctx.set_launch_overlap(overlap)
    try:
        lw, kv, h0, layer, cache = make_layer(shape, 1, cap, [n], seed=5, window=window)
        h = torch.from_numpy(h0).cuda()
        cl = torch.tensor([n], dtype=torch.int32, device="cuda")
        scratch = torch.empty(S.layer_scratch_floats(dict(n_q=shape.n_q, n_kv=shape.n_kv, hd=shape.hd, d=shape.d), 1), device="cuda")
        for call in range(2):                          # the second call runs on the barrier counters the first one left
            h.copy_(torch.from_numpy(h0))
            S.spark_layer_decode(ctx, layer, cl, h, 1, scratch)
            torch.cuda.synchronize()
            assert ctx.device_status() == S.SPARK_OK
            ref, kc, vc = oracle_layer(shape, lw, kv, h0, 0, n, window)
            got_k = np.concatenate([cache["k1c"][0, :, n - 1].float().cpu().numpy(), cache["k2c"][0, :, n - 1].float().cpu().numpy()], axis=-1)
            np.testing.assert_allclose(got_k, kc[:, n - 1], rtol=2 ** -7, atol=1e-5 * parity.rms(kc[:, n - 1]))
            np.testing.assert_allclose(cache["vc"][0, :, n - 1].float().cpu().numpy(), vc[:, n - 1], rtol=2 ** -7, atol=1e-5 * parity.rms(vc[:, n - 1]))
            parity.check_output(h.cpu().numpy()[0], ref["h"], "bf16", f"call {call}")
            parity.check_output(h.cpu().numpy()[0] - h0[0], ref["h"] - h0[0], "bf16", f"call {call} (update only)")
    finally:
        ctx.set_fused_layer(False)
        ctx.set_launch_overlap(False)


@pytest.mark.parametrize("fused,prefetch", [(True, False), (False, True), (False, False)])
def test_stack_call_equals_the_layers_one_by_one(ctx, fused, prefetch):
    sh, cap, n, nl = synth.TINY, 128, 90, 3
    made = [make_layer(sh, 1, cap, [n], seed=20 + l, window=32 if l % 2 == 0 else 0) for l in range(nl)]
    h0 = made[0][2]
    ctx.set_fused_layer(fused)
    ctx.set_l2_prefetch(prefetch)
    try:
        h = torch.from_numpy(h0).cuda()
        cl = torch.tensor([n], dtype=torch.int32, device="cuda")
        scratch = torch.empty(S.layer_scratch_floats(dict(n_q=sh.n_q, n_kv=sh.n_kv, hd=sh.hd, d=sh.d), 1), device="cuda")
        S.spark_stack_decode(ctx, S.make_stack([m[3] for m in made]), cl, h, 1, scratch)
        torch.cuda.synchronize()
        assert ctx.device_status() == S.SPARK_OK
        ref = h0[0].astype(np.float64)
        for l, (lw, kv, _, _, _) in enumerate(made):
            W = {"norm1": lw.norm1, "norm2": lw.norm2, "Wqkv": synth.bf16_bits_to_f32(lw.Wqkv_bits), "Wo": synth.bf16_bits_to_f32(lw.Wo_bits),
                 "K1t": synth.bf16_bits_to_f32(lw.K1t_bits), "K2t": synth.bf16_bits_to_f32(lw.K2t_bits), "Vt": synth.bf16_bits_to_f32(lw.Vt_bits)}
            kc = np.concatenate([kv.k1c[0], kv.k2c[0]], axis=-1).astype(np.float64)
            ref = O.decoder_layer(ref, W, kc, kv.vc[0].astype(np.float64), n, n_q=sh.n_q, n_kv=sh.n_kv, hd=sh.hd, r_attn=sh.r_attn,
                                  k_attn=sh.k_attn, r_ff=sh.r_ff, k_ff=sh.k_ff, window=32 if l % 2 == 0 else 0)["h"]
        parity.check_output(h.cpu().numpy()[0], ref, "bf16")
    finally:
        ctx.set_fused_layer(False)
        ctx.set_l2_prefetch(False)
