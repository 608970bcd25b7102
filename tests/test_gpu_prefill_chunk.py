"""GPU parity of the shared-cache mode (SPARK_SHARED_CACHE): the B tokens of a call are consecutive tokens of
one sequence -- a chunk of its prompt -- appended to one cache, token b attending to the prompt and to the
chunk's tokens up to itself.  The oracle is the decoder layer applied token by token."""
import numpy as np
import pytest
import torch

from oracle import spark_oracle as O
from paper_2506_06644_b200 import binding as S
from paper_2506_06644_b200 import synth
from tests import parity
from tests.test_gpu_layer import bf16_dev

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def ctx():
    c = S.SparkContext(0, max_batch=64)
    yield c
    assert c.device_status() == S.SPARK_OK
    c.close()


@pytest.mark.parametrize("shape,T,L0,cap,window", [
    (synth.TINY, 3, 40, 64, 0),                 # fused projection + rotary + append kernel (up to four tokens)
    (synth.TINY, 7, 20, 64, 0),                 # five and more tokens: separate append kernel
    (synth.TINY, 6, 50, 64, 16),                # local window sliding over the chunk
    (synth.GEMMA2_2B, 8, 300, 512, 0),          # FFN of the chunk on the tcgen05 path
    (synth.GEMMA2_2B, 16, 0, 64, 0),            # a chunk that starts the sequence (empty cache)
    (synth.GEMMA2_2B, 64, 100, 256, 0),         # the largest chunk a layer call takes
    (synth.TINY, 20, 10, 64, 0),                # more than sixteen tokens on the fallback kernels (shape not served by the GEMMs)
    (synth.GEMMA2_9B, 16, 40, 128, 0),          # 9B shape: 16 query / 8 KV heads, d 3584, d_ff 14336 on every tensor-core path
    (synth.GEMMA2_2B, 64, 8128, 8192, 0),       # the benchmarked chunk: 64 tokens behind 8128, global layer (gather stage) ...
    (synth.GEMMA2_2B, 64, 8128, 8192, 4096),    # ... and local layer (window 4096: dense stage)
    (synth.GEMMA2_2B, 64, 3000, 3072, 0),       # a short cache: dense stage over all rows, ragged last tile
])
def test_chunk_of_a_prompt_equals_token_by_token_decoding(ctx, shape, T, L0, cap, window):
    sh = shape
    lw = synth.layer_weights(sh, 21, 0)
    kv = synth.attn_inputs(1, sh.n_q, sh.n_kv, sh.hd, sh.r_attn, cap, [max(L0, 1)], "bf16", seed=22)
    h0 = synth.normal_f32((T, sh.d), 23, 60)
    dev = dict(norm1=torch.from_numpy(lw.norm1).cuda(), norm2=torch.from_numpy(lw.norm2).cuda(),
               Wqkv=bf16_dev(lw.Wqkv_bits), Wo=bf16_dev(lw.Wo_bits), K1t=bf16_dev(lw.K1t_bits),
               K2t=bf16_dev(lw.K2t_bits), Vt=bf16_dev(lw.Vt_bits))
    cache = dict(k1c=bf16_dev(kv.k1c_bits[0]), k2c=bf16_dev(kv.k2c_bits[0]), vc=bf16_dev(kv.vc_bits[0]))     # [n_kv][cap][.]
    cfg = dict(d=sh.d, d_ff=sh.d_ff, r_ff=sh.r_ff, k_ff=sh.k_ff, n_q=sh.n_q, n_kv=sh.n_kv, hd=sh.hd, r_attn=sh.r_attn,
               k_attn=sh.k_attn, window=window, cap=cap, rms_eps=1e-6, rope_base=10000.0, flags=S.SPARK_SHARED_CACHE)
    layer = S.make_layer(dev, cfg, cache)
    h = torch.from_numpy(h0).cuda()
    cl = torch.tensor([L0 + t + 1 for t in range(T)], dtype=torch.int32, device="cuda")
    nqkv = (sh.n_q + 2 * sh.n_kv) * sh.hd
    scratch = torch.empty(T * (nqkv + 2 * sh.n_q * sh.hd + sh.d + 2 + sh.n_q), device="cuda")
    S.spark_layer_decode(ctx, layer, cl, h, T, scratch)
    torch.cuda.synchronize()
    got = h.cpu().numpy()

    W = {"norm1": lw.norm1, "norm2": lw.norm2, "Wqkv": synth.bf16_bits_to_f32(lw.Wqkv_bits),
         "Wo": synth.bf16_bits_to_f32(lw.Wo_bits), "K1t": synth.bf16_bits_to_f32(lw.K1t_bits),
         "K2t": synth.bf16_bits_to_f32(lw.K2t_bits), "Vt": synth.bf16_bits_to_f32(lw.Vt_bits)}
    kc = np.concatenate([kv.k1c[0], kv.k2c[0]], axis=-1).astype(np.float64)
    vc = kv.vc[0].astype(np.float64)
    for t in range(T):                           # the oracle appends token t's row before token t + 1 reads the cache
        # the oracle's layer, or -- when a cached token sits within rounding distance of a head's threshold -- its variant
        # with that token on the other side (the reading taken for the attention tests: either is a correct result)
        last = None
        for ref in parity.layer_refs_within_band(O, h0[t], W, kc, vc, L0 + t + 1, window, n_q=sh.n_q, n_kv=sh.n_kv, hd=sh.hd,
                                                 r_attn=sh.r_attn, k_attn=sh.k_attn, r_ff=sh.r_ff, k_ff=sh.k_ff):
            try:
                parity.check_output(got[t], ref["h"], "bf16", f"token {t}")
                parity.check_output(got[t] - h0[t], ref["h"] - h0[t], "bf16", f"token {t} (update only)")
                last = None
                break
            except AssertionError as e:
                last = e
        if last is not None:
            raise last
    # the chunk's rows are in the one cache, the prompt's rows untouched
    k1 = cache["k1c"].float().cpu().numpy()
    v = cache["vc"].float().cpu().numpy()
    for t in range(T):
        n = L0 + t + 1
        np.testing.assert_allclose(k1[:, n - 1], kc[:, n - 1, : sh.r_attn], rtol=2 ** -7, atol=1e-4 * parity.rms(kc[:, n - 1]))
        np.testing.assert_allclose(v[:, n - 1], vc[:, n - 1], rtol=2 ** -7, atol=1e-4 * parity.rms(vc[:, n - 1]))
    if L0 > 0:
        assert np.array_equal(k1[:, :L0], kv.k1c[0][:, :L0])


def test_attention_queries_sharing_one_cache(ctx):
    # spark_attn_decode alone: eight queries over one cache, query b seeing the first L0 + b + 1 rows
    B, n_q, n_kv, hd, r, cap, L0, k_attn = 8, 8, 4, 64, 32, 256, 200, 24
    kv = synth.attn_inputs(1, n_q, n_kv, hd, r, cap, [cap], "bf16", seed=31)
    q = synth.normal_f32((B, n_q, hd), 32, 0) * hd ** -0.5
    lens = [L0 + b + 1 for b in range(B)]
    o = torch.empty(B, n_q, hd, device="cuda")
    theta = torch.empty(B, n_q, device="cuda")
    S.spark_attn_decode(ctx, torch.from_numpy(q).cuda(), bf16_dev(kv.k1c_bits[0]), bf16_dev(kv.k2c_bits[0]), bf16_dev(kv.vc_bits[0]),
                        S.SPARK_BF16, B, n_q, n_kv, hd, r, cap, torch.tensor(lens, dtype=torch.int32, device="cuda"), 0, k_attn,
                        S.SPARK_SHARED_CACHE, o, theta, None, None, 0)
    torch.cuda.synchronize()
    kc = np.concatenate([kv.k1c[0], kv.k2c[0]], axis=-1).astype(np.float64)
    vc = kv.vc[0].astype(np.float64)
    for b in range(B):
        ref = O.spark_attention(q[b].astype(np.float64), kc, vc, lens[b], k_attn, r)
        parity.check_output(o[b].cpu().numpy().reshape(-1), np.asarray(ref["o"]).reshape(-1), "bf16", f"query {b}")


@pytest.mark.parametrize("T,n_q,n_kv,hd,r,cap,L0,k_attn,window", [
    (17, 8, 4, 256, 128, 1024, 700, 64, 0),          # two query heads per KV head, tensor-core scores for the whole chunk
    (64, 8, 4, 256, 128, 640, 500, 32, 0),           # the largest chunk: 128 columns per KV head
    (40, 4, 4, 128, 64, 512, 300, 40, 100),          # one head per KV head, r = 64, a window sliding over the chunk
    (32, 8, 2, 256, 128, 256, 0, 16, 0),             # four heads per KV head; the chunk starts the sequence (identity for short rows)
    (12, 8, 4, 256, 128, 512, 400, 64, 0),           # a short chunk: per-query kernel over the shared cache
    (64, 16, 8, 256, 128, 900, 800, 48, 0),          # 9B head layout: eight KV heads, sixteen (KV head, 64 columns) groups
    (48, 16, 2, 128, 64, 700, 600, 24, 250),         # eight heads per KV head: falls back (more than 128 columns per KV head)
])
@pytest.mark.parametrize("mode", [0, 2])      # second stage: gather per (token, head) / masked dense products where the shape is served
def test_chunk_attention_on_the_tensor_cores(ctx, mode, T, n_q, n_kv, hd, r, cap, L0, k_attn, window):
    ctx.set_chunk_dense(mode)
    kv = synth.attn_inputs(1, n_q, n_kv, hd, r, cap, [cap], "bf16", seed=41)
    q = synth.normal_f32((T, n_q, hd), 42, 0) * hd ** -0.5
    lens = [L0 + t + 1 for t in range(T)]
    o = torch.full((T, n_q, hd), float("nan"), device="cuda")
    theta = torch.empty(T, n_q, device="cuda")
    count = torch.empty(T, n_q, dtype=torch.int32, device="cuda")
    S.spark_attn_decode(ctx, torch.from_numpy(q).cuda(), bf16_dev(kv.k1c_bits[0]), bf16_dev(kv.k2c_bits[0]), bf16_dev(kv.vc_bits[0]),
                        S.SPARK_BF16, T, n_q, n_kv, hd, r, cap, torch.tensor(lens, dtype=torch.int32, device="cuda"), window, k_attn,
                        S.SPARK_SHARED_CACHE, o, theta, count, None, 0)
    torch.cuda.synchronize()
    ctx.set_chunk_dense(1)
    kc = np.concatenate([kv.k1c[0], kv.k2c[0]], axis=-1).astype(np.float64)
    vc = kv.vc[0].astype(np.float64)
    og, thg, cg = o.cpu().numpy(), theta.cpu().numpy(), count.cpu().numpy()
    for t in range(T):
        ref = O.spark_attention(q[t].astype(np.float64), kc, vc, lens[t], k_attn, r, window)
        for h in range(n_q):
            lo = 0 if window <= 0 else max(0, lens[t] - window)
            s = kc[h // (n_q // n_kv), lo:lens[t], :r] @ q[t, h, :r].astype(np.float64)
            std = float(np.std(s, ddof=1)) if s.size > 1 else 1.0
            parity.check_theta(thg[t, h], ref["theta"][h], std, f"token {t} head {h}")
            near = int(np.sum(np.abs(s - ref["theta"][h]) <= 1e-4 * std)) if np.isfinite(ref["theta"][h]) else 0
            assert abs(int(cg[t, h]) - int(ref["mask"][h].sum())) <= near
        parity.check_output(og[t].reshape(-1), np.asarray(ref["o"]).reshape(-1), "bf16", f"token {t}")


@pytest.mark.parametrize("chunk,pipelined", [(64, False), (32, True)])
def test_prefill_loop_over_two_layers_and_ragged_chunks(ctx, chunk, pipelined):
    # 100 tokens in chunks of 64 (64 + 36) through two layers behind 30 cached tokens, against token-by-token decoding; the same
    # in chunks of 32 (32 + 32 + 32 + 4) with two chunks in flight on two streams and two contexts
    sh, N, L0, cap = synth.GEMMA2_2B, 100, 30, 256
    lws = [synth.layer_weights(sh, 51 + l, 0) for l in range(2)]
    kvs = [synth.attn_inputs(1, sh.n_q, sh.n_kv, sh.hd, sh.r_attn, cap, [L0], "bf16", seed=61 + l) for l in range(2)]
    h0 = synth.normal_f32((N, sh.d), 71, 60)
    layers, keep = [], []
    for lw, kv in zip(lws, kvs):
        dev = dict(norm1=torch.from_numpy(lw.norm1).cuda(), norm2=torch.from_numpy(lw.norm2).cuda(),
                   Wqkv=bf16_dev(lw.Wqkv_bits), Wo=bf16_dev(lw.Wo_bits), K1t=bf16_dev(lw.K1t_bits),
                   K2t=bf16_dev(lw.K2t_bits), Vt=bf16_dev(lw.Vt_bits))
        cache = dict(k1c=bf16_dev(kv.k1c_bits[0]), k2c=bf16_dev(kv.k2c_bits[0]), vc=bf16_dev(kv.vc_bits[0]))
        cfg = dict(d=sh.d, d_ff=sh.d_ff, r_ff=sh.r_ff, k_ff=sh.k_ff, n_q=sh.n_q, n_kv=sh.n_kv, hd=sh.hd, r_attn=sh.r_attn,
                   k_attn=sh.k_attn, window=0, cap=cap, rms_eps=1e-6, rope_base=10000.0, flags=S.SPARK_SHARED_CACHE)
        layers.append(S.make_layer(dev, cfg, cache))
        keep.append((dev, cache))
    h = torch.from_numpy(h0).cuda()
    ctx2 = S.SparkContext(0, max_batch=64) if pipelined else None
    S.spark_prefill(ctx, layers, h, L0, chunk=chunk, more_ctx=[ctx2] if ctx2 is not None else [])
    torch.cuda.synchronize()
    if ctx2 is not None:
        assert ctx2.device_status() == S.SPARK_OK
        ctx2.close()
    got = h.cpu().numpy()
    caches = [(np.concatenate([kv.k1c[0], kv.k2c[0]], axis=-1).astype(np.float64), kv.vc[0].astype(np.float64)) for kv in kvs]
    Ws = [{"norm1": lw.norm1, "norm2": lw.norm2, "Wqkv": synth.bf16_bits_to_f32(lw.Wqkv_bits), "Wo": synth.bf16_bits_to_f32(lw.Wo_bits),
           "K1t": synth.bf16_bits_to_f32(lw.K1t_bits), "K2t": synth.bf16_bits_to_f32(lw.K2t_bits), "Vt": synth.bf16_bits_to_f32(lw.Vt_bits)}
          for lw in lws]
    ref = np.zeros_like(got, dtype=np.float64)
    for t in range(N):
        x = h0[t].astype(np.float64)
        for W, (kc, vc) in zip(Ws, caches):
            x = O.decoder_layer(x, W, kc, vc, L0 + t + 1, n_q=sh.n_q, n_kv=sh.n_kv, hd=sh.hd, r_attn=sh.r_attn, k_attn=sh.k_attn,
                                r_ff=sh.r_ff, k_ff=sh.k_ff, window=0)["h"]
        ref[t] = x
    for t in range(N):
        parity.check_output(got[t], ref[t], "bf16", f"token {t}")


@pytest.mark.parametrize("mode", [0, 2])
@pytest.mark.parametrize("seed", range(6))
def test_seeded_random_shapes_of_the_chunk_attention(ctx, seed, mode):
    ctx.set_chunk_dense(mode)
    # head layouts, chunk lengths, cache fill, k and windows drawn from a seeded generator (shapes the tensor-core path serves)
    rng = np.random.default_rng(1000 + seed)
    gq = int(rng.choice([1, 2, 4])); n_kv = int(rng.choice([1, 2, 4])); n_q = gq * n_kv
    hd, r = [(256, 128), (128, 64), (192, 128)][int(rng.integers(3))]
    T = int(rng.integers(16, min(64, 128 // gq) + 1)); cap = 4 * int(rng.integers(40, 160))
    L0 = int(rng.integers(0, cap - T + 1)); k_attn = int(rng.choice([8, 40, 200])); window = int(rng.choice([0, 0, 37, 300]))
    kv = synth.attn_inputs(1, n_q, n_kv, hd, r, cap, [cap], "bf16", seed=2000 + seed)
    q = synth.normal_f32((T, n_q, hd), 3000 + seed, 0) * hd ** -0.5
    lens = [L0 + t + 1 for t in range(T)]
    o = torch.full((T, n_q, hd), float("nan"), device="cuda")
    theta = torch.empty(T, n_q, device="cuda")
    S.spark_attn_decode(ctx, torch.from_numpy(q).cuda(), bf16_dev(kv.k1c_bits[0]), bf16_dev(kv.k2c_bits[0]), bf16_dev(kv.vc_bits[0]),
                        S.SPARK_BF16, T, n_q, n_kv, hd, r, cap, torch.tensor(lens, dtype=torch.int32, device="cuda"), window, k_attn,
                        S.SPARK_SHARED_CACHE, o, theta, None, None, 0)
    torch.cuda.synchronize()
    ctx.set_chunk_dense(1)
    kc = np.concatenate([kv.k1c[0], kv.k2c[0]], axis=-1).astype(np.float64)
    vc = kv.vc[0].astype(np.float64)
    og, thg = o.cpu().numpy(), theta.cpu().numpy()
    for t in range(T):
        ref = O.spark_attention(q[t].astype(np.float64), kc, vc, lens[t], k_attn, r, window)
        for h in range(n_q):
            lo = 0 if window <= 0 else max(0, lens[t] - window)
            s = kc[h // gq, lo:lens[t], :r] @ q[t, h, :r].astype(np.float64)
            parity.check_theta(thg[t, h], ref["theta"][h], float(np.std(s, ddof=1)) if s.size > 1 else 1.0, f"token {t} head {h}")
        parity.check_output(og[t].reshape(-1), np.asarray(ref["o"]).reshape(-1), "bf16", f"token {t}")


@pytest.mark.parametrize("mode", [0, 2])
def test_rows_behind_the_chunk_may_hold_anything(ctx, mode):
    # the cache is longer than what has been written: the rows behind the chunk's last token hold NaN bit patterns; and the
    # 64-token chunk at 4000 cached rows spans several tiles with a ragged last one (8 of its tokens against the oracle)
    T, n_q, n_kv, hd, r, cap, L0, k_attn = 64, 8, 4, 256, 128, 4200, 4000, 256
    kv = synth.attn_inputs(1, n_q, n_kv, hd, r, cap, [cap], "bf16", seed=77)
    q = synth.normal_f32((T, n_q, hd), 78, 0) * hd ** -0.5
    lens = [L0 + t + 1 for t in range(T)]
    dev = []
    for bits in (kv.k1c_bits[0], kv.k2c_bits[0], kv.vc_bits[0]):
        b = bits.copy()
        b[:, L0 + T:, :] = 0x7FC0          # bf16 NaN
        dev.append(bf16_dev(b))
    ctx.set_chunk_dense(mode)
    o = torch.full((T, n_q, hd), float("nan"), device="cuda")
    theta = torch.empty(T, n_q, device="cuda")
    S.spark_attn_decode(ctx, torch.from_numpy(q).cuda(), dev[0], dev[1], dev[2], S.SPARK_BF16, T, n_q, n_kv, hd, r, cap,
                        torch.tensor(lens, dtype=torch.int32, device="cuda"), 0, k_attn, S.SPARK_SHARED_CACHE, o, theta, None, None, 0)
    torch.cuda.synchronize()
    ctx.set_chunk_dense(1)
    og = o.cpu().numpy()
    assert np.all(np.isfinite(og))
    kc = np.concatenate([kv.k1c[0], kv.k2c[0]], axis=-1).astype(np.float64)
    vc = kv.vc[0].astype(np.float64)
    for t in (0, 1, 17, 31, 32, 47, 62, 63):
        ref = O.spark_attention(q[t].astype(np.float64), kc, vc, lens[t], k_attn, r, 0)
        parity.check_output(og[t].reshape(-1), np.asarray(ref["o"]).reshape(-1), "bf16", f"token {t}")


def test_chunk_mode_is_checked(ctx):
    with pytest.raises(S.SparkError):
        ctx.set_chunk_dense(3)


def test_chunks_in_flight_give_what_one_at_a_time_gives(ctx):
    # many chunks through four layers (alternating local / global) on two streams against the plain loop: outputs and caches
    sh, N, L0, cap, n_layers, chunk = synth.GEMMA2_2B, 640, 17, 704, 4, 64
    gen = torch.Generator(device="cuda")
    gen.manual_seed(5)

    def make():
        layers, keep = [], []
        for l in range(n_layers):
            lw = synth.layer_weights(sh, 91 + l, 0)
            kv = synth.attn_inputs(1, sh.n_q, sh.n_kv, sh.hd, sh.r_attn, cap, [L0], "bf16", seed=95 + l)
            dev = dict(norm1=torch.from_numpy(lw.norm1).cuda(), norm2=torch.from_numpy(lw.norm2).cuda(),
                       Wqkv=bf16_dev(lw.Wqkv_bits), Wo=bf16_dev(lw.Wo_bits), K1t=bf16_dev(lw.K1t_bits),
                       K2t=bf16_dev(lw.K2t_bits), Vt=bf16_dev(lw.Vt_bits))
            cache = dict(k1c=bf16_dev(kv.k1c_bits[0]), k2c=bf16_dev(kv.k2c_bits[0]), vc=bf16_dev(kv.vc_bits[0]))
            cfg = dict(d=sh.d, d_ff=sh.d_ff, r_ff=sh.r_ff, k_ff=sh.k_ff, n_q=sh.n_q, n_kv=sh.n_kv, hd=sh.hd, r_attn=sh.r_attn,
                       k_attn=64, window=(200 if l % 2 == 0 else 0), cap=cap, rms_eps=1e-6, rope_base=10000.0, flags=S.SPARK_SHARED_CACHE)
            layers.append(S.make_layer(dev, cfg, cache))
            keep.append((dev, cache))
        return layers, keep

    h0 = synth.normal_f32((N, sh.d), 99, 0)
    outs = []
    for pipelined in (False, False, True):
        layers, keep = make()
        h = torch.from_numpy(h0).cuda()
        more = [S.SparkContext(0, max_batch=64) for _ in range(2)] if pipelined else []          # three chunks in flight
        S.spark_prefill(ctx, layers, h, L0, chunk=chunk, more_ctx=more)
        torch.cuda.synchronize()
        for c in more:
            assert c.device_status() == S.SPARK_OK
            c.close()
        outs.append((h.cpu().numpy(), [{k: v.float().cpu().numpy() for k, v in c.items()} for _, c in keep]))
    (ha, ca), (hb, cb), (hc, cc) = outs
    assert np.all(np.isfinite(hc))
    # Two runs of the plain loop already differ: sums reduced with atomics round differently, a rounding step flips a stored
    # bf16 cache row or puts a token on the other side of a threshold, and four layers carry that on.  Two chunks in flight
    # must not differ from the plain loop by more than the plain loop differs from itself.
    scale = parity.rms(ha)
    noise = np.abs(ha - hb).max(axis=1) / scale
    diff = np.abs(ha - hc).max(axis=1) / scale
    assert np.median(diff) <= 3 * np.median(noise) + 1e-4, (np.median(diff), np.median(noise))
    assert np.quantile(diff, 0.9) <= 3 * np.quantile(noise, 0.9) + 1e-3 and diff.max() <= 3 * noise.max() + 2e-2
    for la, lb, lc in zip(ca, cb, cc):          # the stored rows likewise
        for k in la:
            assert np.abs(la[k] - lc[k]).mean() <= 3 * np.abs(la[k] - lb[k]).mean() + 1e-4 * np.abs(la[k]).mean()


def test_pipelined_prefill_checks_its_arguments(ctx):
    sh, cap = synth.TINY, 64
    lw = synth.layer_weights(sh, 3, 0)
    kv = synth.attn_inputs(1, sh.n_q, sh.n_kv, sh.hd, sh.r_attn, cap, [4], "bf16", seed=4)
    dev = dict(norm1=torch.from_numpy(lw.norm1).cuda(), norm2=torch.from_numpy(lw.norm2).cuda(), Wqkv=bf16_dev(lw.Wqkv_bits),
               Wo=bf16_dev(lw.Wo_bits), K1t=bf16_dev(lw.K1t_bits), K2t=bf16_dev(lw.K2t_bits), Vt=bf16_dev(lw.Vt_bits))
    cache = dict(k1c=bf16_dev(kv.k1c_bits[0]), k2c=bf16_dev(kv.k2c_bits[0]), vc=bf16_dev(kv.vc_bits[0]))
    cfg = dict(d=sh.d, d_ff=sh.d_ff, r_ff=sh.r_ff, k_ff=sh.k_ff, n_q=sh.n_q, n_kv=sh.n_kv, hd=sh.hd, r_attn=sh.r_attn,
               k_attn=sh.k_attn, window=0, cap=cap, rms_eps=1e-6, rope_base=10000.0, flags=S.SPARK_SHARED_CACHE)
    layer = S.make_layer(dev, cfg, cache)
    h = torch.zeros(8, sh.d, device="cuda")
    with pytest.raises(S.SparkError) as e:          # one context twice: its workspace would be shared by concurrent kernels
        S.spark_prefill(ctx, [layer], h, 4, chunk=4, more_ctx=[ctx])
    assert e.value.status == S.SPARK_ERR_INVALID_ARG
    with pytest.raises(S.SparkError) as e:          # the same stream twice
        S.spark_prefill(ctx, [layer], h, 4, chunk=4, more_ctx=[S.SparkContext(0, max_batch=8)], more_streams=[torch.cuda.current_stream()])
    assert e.value.status == S.SPARK_ERR_INVALID_ARG
    torch.cuda.synchronize()
    assert ctx.device_status() == S.SPARK_OK
