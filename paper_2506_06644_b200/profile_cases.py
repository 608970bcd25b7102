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


CASES = {"chunk64": case_chunk, "layer8": lambda: case_layer(n_layers=4, B=8, steps=2), "ffn": case_ffn, "ffn4": lambda: case_ffn(B=4, sets=12), "ffn16": lambda: case_ffn(B=16, sets=12), "ffn64": lambda: case_ffn(B=64, sets=12), "attn": case_attn, "topk": case_topk, "layer": case_layer}

if __name__ == "__main__":
    name = sys.argv[1] if len(sys.argv) > 1 else ""
    if name not in CASES:
        sys.exit(f"usage: python -m paper_2506_06644_b200.profile_cases {{{'|'.join(CASES)}}}")
    CASES[name]()
    print(f"{name}: done")
