"""GPU parity of the BENCHMARKED configuration: the decoder stack at the Gemma-2 shapes behind an 8192-token prompt, alternating
local-4096 / global layers, run the way bench.py runs it (one CUDA graph per decode step, launch overlap on), several decode steps
with the context growing by one per step -- compared layer by layer with the oracle, every layer fed the GPU's own input (so
bf16-level differences do not compound) and the GPU's own appended cache rows (checked first).  Reduced depth only: the oracle
needs about a tenth of a second per layer and token."""
import numpy as np
import pytest
import torch

from oracle import spark_oracle as O
from paper_2506_06644_b200 import binding as S
from paper_2506_06644_b200 import synth
from tests import parity

pytestmark = pytest.mark.gpu


def bf16_dev(bits):
    return torch.from_numpy(bits.view(np.int16)).cuda().view(torch.bfloat16)


def window_of(layer, ctx_len):
    return 4096 if (layer % 2 == 0 and ctx_len > 4096) else 0       # bench.py's layer pattern


class Stack:
    """n_layers layers of `shape` for B sequences with ctx_len cached tokens each, on the device and as oracle inputs."""

    def __init__(self, shape, n_layers, B, ctx_len, steps, seed):
        self.shape, self.B, self.ctx_len = shape, B, ctx_len
        self.cap = cap = ctx_len + steps + 3
        self.layers, self.W, self.kc, self.vc, self.dev_cache = [], [], [], [], []
        for l in range(n_layers):
            lw = synth.layer_weights(shape, seed, l)
            kv = synth.attn_inputs(B, shape.n_q, shape.n_kv, shape.hd, shape.r_attn, cap, [ctx_len] * B, "bf16", seed=seed + 100 + l)
            dev = dict(norm1=torch.from_numpy(lw.norm1).cuda(), norm2=torch.from_numpy(lw.norm2).cuda(), Wqkv=bf16_dev(lw.Wqkv_bits),
                       Wo=bf16_dev(lw.Wo_bits), K1t=bf16_dev(lw.K1t_bits), K2t=bf16_dev(lw.K2t_bits), Vt=bf16_dev(lw.Vt_bits))
            cache = dict(k1c=bf16_dev(kv.k1c_bits), k2c=bf16_dev(kv.k2c_bits), vc=bf16_dev(kv.vc_bits))
            cfg = dict(d=shape.d, d_ff=shape.d_ff, r_ff=shape.r_ff, k_ff=shape.k_ff, n_q=shape.n_q, n_kv=shape.n_kv, hd=shape.hd,
                       r_attn=shape.r_attn, k_attn=shape.k_attn, window=window_of(l, ctx_len), cap=cap, rms_eps=1e-6,
                       rope_base=10000.0, flags=0)
            self.layers.append(S.make_layer(dev, cfg, cache))
            self.dev_cache.append(cache)
            self.W.append({"norm1": lw.norm1, "norm2": lw.norm2, "Wqkv": synth.bf16_bits_to_f32(lw.Wqkv_bits),
                           "Wo": synth.bf16_bits_to_f32(lw.Wo_bits), "K1t": synth.bf16_bits_to_f32(lw.K1t_bits),
                           "K2t": synth.bf16_bits_to_f32(lw.K2t_bits), "Vt": synth.bf16_bits_to_f32(lw.Vt_bits)})
            self.kc.append(np.concatenate([kv.k1c, kv.k2c], axis=-1).astype(np.float64))      # [B][n_kv][cap][hd]
            self.vc.append(kv.vc.astype(np.float64))
            del lw, kv


def run_and_compare(shape, n_layers, B, ctx_len, steps, seed):
    st = Stack(shape, n_layers, B, ctx_len, steps, seed)
    sh = shape
    ctx = S.SparkContext(0, max_batch=B, max_dff=sh.d_ff, max_cap=st.cap, n_q=sh.n_q, hd=sh.hd, max_d=sh.d)
    ctx.set_launch_overlap(True)
    h = torch.empty(B, sh.d, device="cuda")
    cl = torch.zeros(B, dtype=torch.int32, device="cuda")
    cfg = dict(n_q=sh.n_q, n_kv=sh.n_kv, hd=sh.hd, d=sh.d)
    scratch = torch.empty(S.layer_scratch_floats(cfg, B), device="cuda")
    cl.fill_(ctx_len + 1)
    h.zero_()

    # one CUDA graph per prefix of the stack: replaying prefix l from the step's input gives the GPU's own input of layer l; the
    # last one is the whole stack, what bench.py replays
    side = torch.cuda.Stream()
    graphs = []
    for depth in range(1, n_layers + 1):
        with torch.cuda.stream(side):
            for lay in st.layers[:depth]:
                S.spark_layer_decode(ctx, lay, cl, h, B, scratch)
            side.synchronize()
            g = torch.cuda.CUDAGraph()
            with torch.cuda.graph(g, stream=side):
                for lay in st.layers[:depth]:
                    S.spark_layer_decode(ctx, lay, cl, h, B, scratch)
        graphs.append(g)
    torch.cuda.synchronize()
    assert ctx.device_status() == S.SPARK_OK

    worst = 0.0
    for step in range(steps):
        n = ctx_len + 1 + step                                   # valid tokens, the one being decoded included
        h_in = synth.normal_f32((B, sh.d), seed, 60 + step)
        cl.fill_(n)
        H = [h_in]
        for depth in range(1, n_layers + 1):
            h.copy_(torch.from_numpy(h_in))
            graphs[depth - 1].replay()
            torch.cuda.synchronize()
            H.append(h.cpu().numpy().copy())
        assert ctx.device_status() == S.SPARK_OK
        for l in range(n_layers):
            c = st.dev_cache[l]
            k1 = c["k1c"][:, :, n - 1].float().cpu().numpy()
            k2 = c["k2c"][:, :, n - 1].float().cpu().numpy()
            v = c["vc"][:, :, n - 1].float().cpu().numpy()
            for b in range(B):
                what = f"step {step} layer {l} seq {b}"
                # the oracle's layer; if a token sits within rounding distance of an attention threshold, also the variants with
                # that token on the other side (the threshold is discontinuous: the reading taken for the attention tests)
                last = None
                for ref in parity.layer_refs_within_band(O, H[l][b], st.W[l], st.kc[l][b], st.vc[l][b], n, window_of(l, ctx_len), n_q=sh.n_q,
                                                         n_kv=sh.n_kv, hd=sh.hd, r_attn=sh.r_attn, k_attn=sh.k_attn, r_ff=sh.r_ff, k_ff=sh.k_ff):
                    try:
                        worst = max(worst, parity.check_output(H[l + 1][b], ref["h"], "bf16", what))
                        parity.check_output(H[l + 1][b] - H[l][b], ref["h"] - H[l][b], "bf16", what + " (update only)")
                        last = None
                        break
                    except AssertionError as e:
                        last = e
                if last is not None:
                    raise last
                # appended rows: equal up to one bf16 rounding step of an fp32-vs-fp64 difference; with five or more tokens the
                # projection's inputs are a two-term bf16 split (an absolute error of about 1e-5 of the row's scale before rounding)
                got_k = np.concatenate([k1[b], k2[b]], axis=-1)
                atol = 1e-6 if B < 5 else 1e-4 * parity.rms(st.kc[l][b][:, n - 1])
                np.testing.assert_allclose(got_k, st.kc[l][b][:, n - 1], rtol=2 ** -7, atol=atol, err_msg=what)
                np.testing.assert_allclose(v[b], st.vc[l][b][:, n - 1], rtol=2 ** -7, atol=atol, err_msg=what)
                # later steps read the rows the GPU stored
                st.kc[l][b][:, n - 1] = got_k
                st.vc[l][b][:, n - 1] = v[b]
    ctx.close()
    return worst


def test_2b_stack_ctx_8192_four_layers_first_four_decode_steps():
    run_and_compare(synth.GEMMA2_2B, n_layers=4, B=1, ctx_len=8192, steps=4, seed=11)


def test_2b_stack_ctx_8192_batch_8_two_layers():
    run_and_compare(synth.GEMMA2_2B, n_layers=2, B=8, ctx_len=8192, steps=2, seed=12)


def test_9b_layer_ctx_8192():
    run_and_compare(synth.GEMMA2_9B, n_layers=2, B=1, ctx_len=8192, steps=2, seed=13)
