"""Small, self-contained launches of each kernel for profiling under ncu.

    python -m paper_2506_06644_b200.profile_cases ffn     # one-token Spark FFN, Gemma-2-2B shape
    python -m paper_2506_06644_b200.profile_cases ffn4    # four tokens (few-token kernel)
    python -m paper_2506_06644_b200.profile_cases ffn16   # sixteen tokens (tcgen05 chunk kernels)
    python -m paper_2506_06644_b200.profile_cases ffn64   # a chunk of 64 tokens (tcgen05 kernels)
    python -m paper_2506_06644_b200.profile_cases attn    # Spark attention, batch 1, context 8192
    python -m paper_2506_06644_b200.profile_cases topk    # statistical top-k, 512 rows x 65536
    python -m paper_2506_06644_b200.profile_cases layer   # four decoder layers, one token
    python -m paper_2506_06644_b200.profile_cases chunk64 # four decoder layers over a 64-token chunk of a prompt
    python -m paper_2506_06644_b200.profile_cases layer8  # four decoder layers, eight sequences
    python -m paper_2506_06644_b200.profile_cases layer_ab [9b]   # one-token layer: A/B of the execution paths, timed + phase timeline

Every case cycles over enough distinct weight sets / caches / rows to exceed the 126 MB L2, holds at
most about 1 GB on the device and launches a dozen kernels, so that a capture of two or three of
them ends by itself within a minute or two.  Inputs are seeded torch tensors made on the device
(profiling looks at time and traffic, not at values)."""
import sys

import torch

from . import binding as S
from . import synth


def _w(gen, rows, cols, fan_in):
    return (torch.randn(rows, cols, device="cuda", generator=gen) * fan_in ** -0.5).to(torch.bfloat16)


def case_ffn(B=1, sets=12):
    sh = synth.GEMMA2_2B
    gen = torch.Generator(device="cuda")
    gen.manual_seed(0)
    ctx = S.SparkContext(0, max_batch=B, max_dff=sh.d_ff, max_d=sh.d)
    ws = [(_w(gen, sh.d_ff, sh.r_ff, sh.d), _w(gen, sh.d_ff, sh.d - sh.r_ff, sh.d), _w(gen, sh.d_ff, sh.d, sh.d))
          for _ in range(sets)]
    x = torch.randn(B, sh.d, device="cuda", generator=gen)
    x = x / x.pow(2).mean(dim=1, keepdim=True).sqrt()
    y = torch.empty(B, sh.d, device="cuda")
    theta = torch.empty(B, device="cuda")
    torch.cuda.synchronize()
    for K1t, K2t, Vt in ws:
        S.spark_ffn_decode(ctx, x, B, K1t, K2t, Vt, S.SPARK_BF16, sh.d, sh.d_ff, sh.r_ff, sh.k_ff, 0, y, theta, None, None)
    torch.cuda.synchronize()
    assert ctx.device_status() == S.SPARK_OK


def case_attn(B=1, ctx_len=8192, sets=10):
    sh = synth.GEMMA2_2B
    gen = torch.Generator(device="cuda")
    gen.manual_seed(1)
    ctx = S.SparkContext(0, max_batch=B, max_cap=ctx_len, n_q=sh.n_q, hd=sh.hd)
    caches = [tuple(torch.randn(B, sh.n_kv, ctx_len, w, device="cuda", generator=gen).to(torch.bfloat16)
                    for w in (sh.r_attn, sh.hd - sh.r_attn, sh.hd)) for _ in range(sets)]
    q = torch.randn(B, sh.n_q, sh.hd, device="cuda", generator=gen) * sh.hd ** -0.5
    o = torch.empty(B, sh.n_q, sh.hd, device="cuda")
    cl = torch.full((B,), ctx_len, dtype=torch.int32, device="cuda")
    torch.cuda.synchronize()
    for k1c, k2c, vc in caches:
        S.spark_attn_decode(ctx, q, k1c, k2c, vc, S.SPARK_BF16, B, sh.n_q, sh.n_kv, sh.hd, sh.r_attn, ctx_len, cl, 0,
                            sh.k_attn, 0, o, None, None, None, 0)
    torch.cuda.synchronize()
    assert ctx.device_status() == S.SPARK_OK


def case_topk(rows=512, n=65536, k=1311, calls=6):
    gen = torch.Generator(device="cuda")
    gen.manual_seed(2)
    ctx = S.SparkContext(0)
    xs = [torch.randn(rows, n, device="cuda", generator=gen) for _ in range(3)]       # 3 x 134 MB
    theta = torch.empty(rows, device="cuda")
    count = torch.empty(rows, dtype=torch.int32, device="cuda")
    cap = 4 * k
    idx = torch.empty(rows, cap, dtype=torch.int32, device="cuda")
    val = torch.empty(rows, cap, device="cuda")
    torch.cuda.synchronize()
    for c in range(calls):          # even calls: theta and count only; odd calls: with the ordered lists
        lists = c % 2 == 1
        S.spark_stat_topk(ctx, xs[c % 3], rows, n, n, k, S.SPARK_FILL_ZERO, theta, count, idx if lists else None,
                          val if lists else None, cap if lists else 0, None)
    torch.cuda.synchronize()
    assert ctx.device_status() == S.SPARK_OK


def case_layer(n_layers=4, B=1, ctx_len=8192, steps=3, overlap=True):
    sh = synth.GEMMA2_2B
    gen = torch.Generator(device="cuda")
    gen.manual_seed(3)
    ctx = S.SparkContext(0, max_batch=B, max_dff=sh.d_ff, max_cap=ctx_len, n_q=sh.n_q, hd=sh.hd, max_d=sh.d)
    ctx.set_launch_overlap(overlap)
    nqkv = (sh.n_q + 2 * sh.n_kv) * sh.hd
    layers = []
    for _ in range(n_layers):
        w = dict(norm1=torch.ones(sh.d, device="cuda"), norm2=torch.ones(sh.d, device="cuda"),
                 Wqkv=_w(gen, nqkv, sh.d, sh.d), Wo=_w(gen, sh.d, sh.n_q * sh.hd, sh.n_q * sh.hd),
                 K1t=_w(gen, sh.d_ff, sh.r_ff, sh.d), K2t=_w(gen, sh.d_ff, sh.d - sh.r_ff, sh.d), Vt=_w(gen, sh.d_ff, sh.d, sh.d))
        cache = dict(k1c=torch.randn(B, sh.n_kv, ctx_len, sh.r_attn, device="cuda", generator=gen).to(torch.bfloat16),
                     k2c=torch.randn(B, sh.n_kv, ctx_len, sh.hd - sh.r_attn, device="cuda", generator=gen).to(torch.bfloat16),
                     vc=torch.randn(B, sh.n_kv, ctx_len, sh.hd, device="cuda", generator=gen).to(torch.bfloat16))
        cfg = dict(d=sh.d, d_ff=sh.d_ff, r_ff=sh.r_ff, k_ff=sh.k_ff, n_q=sh.n_q, n_kv=sh.n_kv, hd=sh.hd, r_attn=sh.r_attn,
                   k_attn=sh.k_attn, window=0, cap=ctx_len, rms_eps=1e-6, rope_base=10000.0, flags=0)
        layers.append((S.make_layer(w, cfg, cache), w, cache))
    h = torch.randn(B, sh.d, device="cuda", generator=gen)
    cl = torch.full((B,), ctx_len, dtype=torch.int32, device="cuda")
    scratch = torch.empty(B * (nqkv + 2 * sh.n_q * sh.hd + sh.d + 2 + sh.n_q), device="cuda")
    torch.cuda.synchronize()
    for _ in range(steps):
        for lay in layers:
            S.spark_layer_decode(ctx, lay[0], cl, h, B, scratch)
    torch.cuda.synchronize()
    assert ctx.device_status() == S.SPARK_OK


def case_chunk(n_layers=4, T=64, ctx_len=8192, steps=2):
    """Chunks of a prompt: T consecutive tokens of one sequence per layer call, behind ctx_len - T cached tokens."""
    sh = synth.GEMMA2_2B
    gen = torch.Generator(device="cuda")
    gen.manual_seed(4)
    ctx = S.SparkContext(0, max_batch=T, max_dff=sh.d_ff, max_cap=ctx_len, n_q=sh.n_q, hd=sh.hd, max_d=sh.d)
    ctx.set_launch_overlap(True)
    nqkv = (sh.n_q + 2 * sh.n_kv) * sh.hd
    layers = []
    for _ in range(n_layers):
        w = dict(norm1=torch.ones(sh.d, device="cuda"), norm2=torch.ones(sh.d, device="cuda"),
                 Wqkv=_w(gen, nqkv, sh.d, sh.d), Wo=_w(gen, sh.d, sh.n_q * sh.hd, sh.n_q * sh.hd),
                 K1t=_w(gen, sh.d_ff, sh.r_ff, sh.d), K2t=_w(gen, sh.d_ff, sh.d - sh.r_ff, sh.d), Vt=_w(gen, sh.d_ff, sh.d, sh.d))
        cache = dict(k1c=torch.randn(sh.n_kv, ctx_len, sh.r_attn, device="cuda", generator=gen).to(torch.bfloat16),
                     k2c=torch.randn(sh.n_kv, ctx_len, sh.hd - sh.r_attn, device="cuda", generator=gen).to(torch.bfloat16),
                     vc=torch.randn(sh.n_kv, ctx_len, sh.hd, device="cuda", generator=gen).to(torch.bfloat16))
        cfg = dict(d=sh.d, d_ff=sh.d_ff, r_ff=sh.r_ff, k_ff=sh.k_ff, n_q=sh.n_q, n_kv=sh.n_kv, hd=sh.hd, r_attn=sh.r_attn,
                   k_attn=sh.k_attn, window=0, cap=ctx_len, rms_eps=1e-6, rope_base=10000.0, flags=S.SPARK_SHARED_CACHE)
        layers.append((S.make_layer(w, cfg, cache), w, cache))
    h = torch.randn(T, sh.d, device="cuda", generator=gen)
    cl = torch.arange(ctx_len - T + 1, ctx_len + 1, dtype=torch.int32, device="cuda")
    scratch = torch.empty(T * (nqkv + 2 * sh.n_q * sh.hd + sh.d + 2 + sh.n_q), device="cuda")
    torch.cuda.synchronize()
    for _ in range(steps):
        for lay in layers:
            S.spark_layer_decode(ctx, lay[0], cl, h, T, scratch)
    torch.cuda.synchronize()
    assert ctx.device_status() == S.SPARK_OK


def case_layer_ab(shape_name="2b", n_layers=12, ctx_len=8192):
    """A/B of the execution paths of a one-token layer call on a 12-layer stack (CUDA-graph replay, launch overlap on, CUDA
    events): kernel-per-step (default), with L2 prefetch of the next kernel's weights, fused persistent kernel per layer and per
    stack; then the fused kernel's phase timeline (per-block cycle stamps of its last layer: median and maximum of the time
    between consecutive marks).  Prints its figures: nothing here is meant for an ncu capture."""
    import numpy as np
    sh = synth.GEMMA2_9B if shape_name == "9b" else synth.GEMMA2_2B
    gen = torch.Generator(device="cuda")
    gen.manual_seed(5)
    cap = ctx_len + 64
    ctx = S.SparkContext(0, max_batch=1, max_dff=sh.d_ff, max_cap=cap, n_q=sh.n_q, hd=sh.hd, max_d=sh.d)
    ctx.set_launch_overlap(True)
    nqkv = (sh.n_q + 2 * sh.n_kv) * sh.hd
    layers = []
    for l in range(n_layers):
        w = dict(norm1=torch.ones(sh.d, device="cuda"), norm2=torch.ones(sh.d, device="cuda"),
                 Wqkv=_w(gen, nqkv, sh.d, sh.d), Wo=_w(gen, sh.d, sh.n_q * sh.hd, sh.n_q * sh.hd),
                 K1t=_w(gen, sh.d_ff, sh.r_ff, sh.d), K2t=_w(gen, sh.d_ff, sh.d - sh.r_ff, sh.d), Vt=_w(gen, sh.d_ff, sh.d, sh.d))
        cache = dict(k1c=torch.randn(1, sh.n_kv, cap, sh.r_attn, device="cuda", generator=gen).to(torch.bfloat16),
                     k2c=torch.randn(1, sh.n_kv, cap, sh.hd - sh.r_attn, device="cuda", generator=gen).to(torch.bfloat16),
                     vc=torch.randn(1, sh.n_kv, cap, sh.hd, device="cuda", generator=gen).to(torch.bfloat16))
        cfg = dict(d=sh.d, d_ff=sh.d_ff, r_ff=sh.r_ff, k_ff=sh.k_ff, n_q=sh.n_q, n_kv=sh.n_kv, hd=sh.hd, r_attn=sh.r_attn,
                   k_attn=sh.k_attn, window=4096 if l % 2 == 0 else 0, cap=cap, rms_eps=1e-6, rope_base=10000.0, flags=0)
        layers.append(S.make_layer(w, cfg, cache))
    stack = S.make_stack(layers)
    h = torch.randn(1, sh.d, device="cuda", generator=gen)
    cl = torch.full((1,), ctx_len, dtype=torch.int32, device="cuda")
    scratch = torch.empty(S.layer_scratch_floats(dict(n_q=sh.n_q, n_kv=sh.n_kv, hd=sh.hd, d=sh.d), 1), device="cuda")

    def per_layer():
        for lay in layers:
            S.spark_layer_decode(ctx, lay, cl, h, 1, scratch)

    def stacked():
        S.spark_stack_decode(ctx, stack, cl, h, 1, scratch)

    def timed(fn, name):
        side = torch.cuda.Stream()
        with torch.cuda.stream(side):
            fn()
            side.synchronize()
            g = torch.cuda.CUDAGraph()
            with torch.cuda.graph(g, stream=side):
                fn()
        torch.cuda.synchronize()
        for _ in range(5):
            g.replay()
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for _ in range(30):
            g.replay()
        e1.record()
        torch.cuda.synchronize()
        assert ctx.device_status() == S.SPARK_OK
        print(f"{name}: {e0.elapsed_time(e1) / 30 / n_layers * 1e3:.2f} us per layer")

    ctx.set_fused_layer(False)
    timed(per_layer, "kernel per step (default)                ")
    ctx.set_l2_prefetch(True)
    timed(stacked, "kernel per step + L2 prefetch, stack call ")
    ctx.set_l2_prefetch(False)
    ctx.set_fused_layer(True)
    timed(per_layer, "fused persistent kernel, one launch/layer ")
    timed(stacked, "fused persistent kernel, one launch/stack ")
    tr = torch.zeros(ctx.grid_size * 16, dtype=torch.int64, device="cuda")
    ctx.set_phase_trace(tr)
    stacked()
    torch.cuda.synchronize()
    ctx.set_phase_trace(None)
    t = tr.cpu().numpy().reshape(-1, 16).astype(np.float64)
    names = ["start", "P1 done (QKV, rotary, append)", "G1 (grid barrier)", "P2 done (predictor scores)", "X2 (theta per head)",
             "gather landed (k2c / vc rows)", "P3 done (softmax x gate x value)", "G3", "P4 done (Wo)", "G4", "P5 done (FFN scores)",
             "X5 (theta)", "gather landed (K2t / Vt rows)", "P6 done (V u)", "G6"]
    mhz = torch.cuda.get_device_properties(0).clock_rate / 1e3 if hasattr(torch.cuda.get_device_properties(0), "clock_rate") else 1965.0
    print(f"fused kernel, last layer of the stack, time between consecutive marks over the {t.shape[0]} blocks (us at {mhz:.0f} MHz):")
    for k in range(2, 15):
        dlt = (t[:, k] - t[:, k - 1]) / mhz
        print(f"  {names[k]:34s} median {np.median(dlt):6.2f}   max {dlt.max():6.2f}")
    dl = (t[:, 14] - t[:, 2]) / mhz
    print(f"  G1 -> G6 (a layer minus its P1): median {np.median(dl):6.2f}")


CASES = {"layer_ab": case_layer_ab, "chunk64": case_chunk, "chunk64_4k": lambda: case_chunk(ctx_len=4096), "attn8x32k": lambda: case_attn(B=8, ctx_len=32768, sets=3), "layer8": lambda: case_layer(n_layers=4, B=8, steps=2), "ffn": case_ffn, "ffn4": lambda: case_ffn(B=4, sets=12), "ffn16": lambda: case_ffn(B=16, sets=12), "ffn64": lambda: case_ffn(B=64, sets=12), "attn": case_attn, "topk": case_topk, "layer": case_layer}

if __name__ == "__main__":
    name = sys.argv[1] if len(sys.argv) > 1 else ""
    if name not in CASES:
        sys.exit(f"usage: python -m paper_2506_06644_b200.profile_cases {{{'|'.join(CASES)}}}")
    CASES[name](*sys.argv[2:3]) if name == "layer_ab" else CASES[name]()
    print(f"{name}: done")
