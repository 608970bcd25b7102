#!/usr/bin/env python
"""Benchmark of the Spark decode hot path on B200.

A step decodes ONE token per sequence through the whole decoder stack: every layer is one
spark_layer_decode call (RMSNorm + dense QKV projection, rotary encoding + cache append, Spark
attention with its statistical top-k, output projection, Spark FFN with its statistical top-k).
Workload (default): Gemma-2-2B shape, 26 layers, bf16 weights and KV caches, context 8192, batch 1,
random-init weights and synthetic N(0,1) caches (seeded).  The 2.9 GB of weights and 0.9 GB of
caches are far larger than L2, so every step streams them from HBM.

Prints ONE JSON line (rank 0).  `value` is microseconds per token per layer with all inputs
resident in HBM; `e2e` is the same through the same C-ABI calls with the token's hidden state
starting and ending in pinned host memory.  `roofline` is for the dominant kernel (the fused Spark
FFN kernel): touched bytes (all of K1t plus the active rows of K2t and Vt) over its average
duration, timed with CUDA events over a loop of the same launches.  `cpu_baseline` times the fp64
oracle on the host cores on a bounded sample.  `--impl reference` times only that oracle.
The default run (2B shape, batch 1) also measures, under `stacks`, the 42-layer 9B-shape stack at
batch 1 and the 2B-shape stack at batch 8, and under `other_workloads` the remaining configurations
(batched FFN, attention at 4096 to 32768 tokens, the LM head, statistical top-k on three distributions).
"""
from __future__ import annotations

import argparse
import json
import os
import subprocess
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import numpy as np

# dram__bytes_read.sum + dram__bytes_write.sum per launch of the fused FFN kernel, from one ncu
# capture of that kernel (keyed by shape and batch); None where no capture exists.
NCU_TRAFFIC_BYTES = {("2b", 1): 25.04e6}

FALLBACK_HBM_GBS = 6650.0


def parse():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=256)
    ap.add_argument("--warmup", type=int, default=8)
    ap.add_argument("--impl", default="spark", choices=["spark", "reference"])
    ap.add_argument("--shape", default="2b", choices=["2b", "9b", "tiny"])
    ap.add_argument("--batch", type=int, default=1)
    ap.add_argument("--ctx", type=int, default=8192)
    ap.add_argument("--layers", type=int, default=0, help="0 = the shape's layer count")
    ap.add_argument("--no-dense", action="store_true", help="skip the dense-loads comparator")
    ap.add_argument("--no-cpu", action="store_true", help="skip the oracle timing")
    ap.add_argument("--overlap", type=int, default=1, help="1 = launch kernels with programmatic stream serialization")
    ap.add_argument("--no-extra", action="store_true", help="skip the other configurations (batched FFN, long-context attention, top-k)")
    ap.add_argument("--study", default="", choices=["", "batch"], help="batch: where the union of the tokens' active sets stops paying (Appendix B)")
    ap.add_argument("--no-graph", action="store_true", help="launch every kernel from the host instead of replaying a CUDA graph")
    return ap.parse_args()


def shape_of(name):
    from paper_2506_06644_b200 import synth
    return {"2b": synth.GEMMA2_2B, "9b": synth.GEMMA2_9B, "tiny": synth.TINY}[name]


def measured_peak():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(path) as f:
            return float(json.load(f)["hbm_gbs"]), "measured"
    except Exception:
        return FALLBACK_HBM_GBS, "fallback"


class ClockSampler:
    """Samples SM clocks and throttle reasons with nvidia-smi while the timed region runs."""
    FIELDS = ("clocks.sm,clocks.max.sm,clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
              "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, index):
        self.index, self.rows, self.proc = index, [], None

    def start(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", f"--id={self.index}", f"--query-gpu={self.FIELDS}",
                                          "--format=csv,noheader,nounits", "-lms", "100"],
                                         stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._read, daemon=True)
            self.thread.start()
        except Exception:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.rows.append([c.strip() for c in line.split(",")])

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        time.sleep(0.15)
        self.proc.terminate()
        try:
            self.proc.wait(timeout=2)
        except Exception:
            self.proc.kill()
        sm = [float(r[0]) for r in self.rows if r and r[0].replace(".", "").isdigit()]
        mx = [float(r[1]) for r in self.rows if len(r) > 1 and r[1].replace(".", "").isdigit()]
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        reasons = sorted({names[i] for r in self.rows if len(r) >= 6 for i in range(4) if r[2 + i] == "Active"})
        return {"sm_mhz": float(np.median(sm)) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "reasons": reasons, "samples": len(sm)}


# --------------------------------------------------------------------------------------------
# oracle timing (cpu_baseline and the reference arm)
# --------------------------------------------------------------------------------------------
def oracle_sample(shape, ctx_len, n_layers, seed=0):
    """Host inputs for `n_layers` layers of one token at context ctx_len (bf16-rounded values)."""
    from paper_2506_06644_b200 import synth
    layers = []
    for l in range(n_layers):
        lw = synth.layer_weights(shape, seed, l)
        W = {"norm1": lw.norm1, "norm2": lw.norm2, "Wqkv": synth.bf16_bits_to_f32(lw.Wqkv_bits),
             "Wo": synth.bf16_bits_to_f32(lw.Wo_bits), "K1t": synth.bf16_bits_to_f32(lw.K1t_bits),
             "K2t": synth.bf16_bits_to_f32(lw.K2t_bits), "Vt": synth.bf16_bits_to_f32(lw.Vt_bits)}
        kv = synth.attn_inputs(1, shape.n_q, shape.n_kv, shape.hd, shape.r_attn, ctx_len, [ctx_len], "bf16",
                               seed=seed + 1000 + l)
        kc = np.concatenate([kv.k1c[0], kv.k2c[0]], axis=-1).astype(np.float64)
        layers.append((W, kc, kv.vc[0].astype(np.float64)))
    h = synth.normal_f32((shape.d,), seed, 60).astype(np.float64)
    return layers, h


def oracle_run(shape, layers, h, ctx_len):
    from oracle import spark_oracle as O
    for W, kc, vc in layers:
        h = O.decoder_layer(h, W, kc, vc, ctx_len, n_q=shape.n_q, n_kv=shape.n_kv, hd=shape.hd,
                            r_attn=shape.r_attn, k_attn=shape.k_attn, r_ff=shape.r_ff, k_ff=shape.k_ff)["h"]
    return h


def host_threads():
    try:
        from threadpoolctl import threadpool_info
        n = max([p.get("num_threads", 1) for p in threadpool_info()] or [1])
    except Exception:
        n = 1
    try:
        return min(n, len(os.sched_getaffinity(0)))
    except Exception:
        return n


def run_reference(args):
    """The oracle as it stands on the host cores: each step is one layer of one token."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    shape = shape_of(args.shape)
    layers, h = oracle_sample(shape, args.ctx, 1)
    for _ in range(max(args.warmup, 1)):
        oracle_run(shape, layers, h, args.ctx)
    t0 = time.perf_counter()
    for _ in range(args.steps):
        oracle_run(shape, layers, h, args.ctx)
    dt = time.perf_counter() - t0
    us = dt / args.steps * 1e6
    cores = host_threads()
    line = {
        "impl": "reference", "metric": "us_per_token_per_layer", "value": us, "unit": "us/token/layer",
        "n_gpus": args.gpus, "steps": args.steps, "warmup": args.warmup, "ms_per_step": dt / args.steps * 1e3,
        "higher_is_better": False, "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": workload_name(args, shape), "sample": "one layer of one token per step"},
        "cpu_baseline": {"value": us, "unit": "us/token/layer", "cores": cores, "kind": "oracle",
                         "sample": f"{args.steps} steps of one decoder layer for one token at context {args.ctx}"},
        "e2e": {"value": us, "unit": "us/token/layer", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }
    print(json.dumps(line), flush=True)


def workload_name(args, shape):
    n_layers = args.layers or shape.n_layers
    return (f"gemma2-{args.shape}-shape spark decoder: {n_layers} layers x spark_layer_decode, decode of "
            f"{args.steps} tokens after a {args.ctx}-token prompt (synthetic cache), batch {args.batch}, bf16 weights+cache")


# --------------------------------------------------------------------------------------------
# N > 1: independent replicas, one process per GPU.  The step time is the slowest rank's; the
# whole-job figure counts every rank's tokens.
def max_over_ranks(ms, world, device):
    """The largest of the ranks' times (every rank gets it).  `device`: where the process group reduces."""
    import torch
    import torch.distributed as dist
    t = torch.tensor([ms], dtype=torch.float64, device=device)
    if world > 1:
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def us_per_token_per_layer(ms_total, steps, n_layers, batch, world):
    """Time of one decoder layer for one token, whole job: `world` replicas each step `batch` tokens."""
    return ms_total / steps * 1e3 / (n_layers * batch * world)


# --------------------------------------------------------------------------------------------
# the CUDA arm
# --------------------------------------------------------------------------------------------
def step_stats(events, torch):
    """Per-step times (ms) from the events recorded around every step of a timed loop."""
    per = np.array([events[i].elapsed_time(events[i + 1]) for i in range(len(events) - 1)])
    return {"mean": float(per.mean()), "median": float(np.median(per)), "min": float(per.min())}


def measure_stack(torch, S, dist, dev, rank, world, shape_name, B, ctx_len, n_layers, steps, W, overlap, no_graph, no_dense,
                  with_e2e, with_kernels):
    """Build the decoder stack of `shape_name` for B sequences behind ctx_len cached tokens, time `steps` decode steps of
    the whole stack (plus its dense-loads comparator, the end-to-end variant and the per-kernel loops), free it, and
    return the figures.  One step decodes one token per sequence through every layer."""
    shape = shape_of(shape_name)
    d, hd = shape.d, shape.hd
    cap = ctx_len + steps + W + 8                       # the prompt plus every token decoded in one timed loop
    ctx = S.SparkContext(dev.index, max_batch=B, max_dff=shape.d_ff, max_cap=cap, n_q=shape.n_q, hd=hd, max_d=d)
    ctx.set_launch_overlap(bool(overlap))
    gen = torch.Generator(device=dev)
    gen.manual_seed(1234 + rank)

    def randw(rows, cols, fan_in):
        return (torch.randn(rows, cols, device=dev, generator=gen) * (fan_in ** -0.5)).to(torch.bfloat16)

    nqkv = (shape.n_q + 2 * shape.n_kv) * hd
    layers = []
    for l in range(n_layers):
        w = dict(norm1=1.0 + 0.1 * torch.randn(d, device=dev, generator=gen),
                 norm2=1.0 + 0.1 * torch.randn(d, device=dev, generator=gen),
                 Wqkv=randw(nqkv, d, d), Wo=randw(d, shape.n_q * hd, shape.n_q * hd),
                 K1t=randw(shape.d_ff, shape.r_ff, d), K2t=randw(shape.d_ff, d - shape.r_ff, d),
                 Vt=randw(shape.d_ff, d, d))
        cache = dict(k1c=torch.randn(B, shape.n_kv, cap, shape.r_attn, device=dev, generator=gen).to(torch.bfloat16),
                     k2c=torch.randn(B, shape.n_kv, cap, hd - shape.r_attn, device=dev, generator=gen).to(torch.bfloat16),
                     vc=torch.randn(B, shape.n_kv, cap, hd, device=dev, generator=gen).to(torch.bfloat16))
        window = 4096 if (l % 2 == 0 and ctx_len > 4096) else 0      # local / global layers alternate
        cfg = dict(d=d, d_ff=shape.d_ff, r_ff=shape.r_ff, k_ff=shape.k_ff, n_q=shape.n_q, n_kv=shape.n_kv, hd=hd,
                   r_attn=shape.r_attn, k_attn=shape.k_attn, window=window, cap=cap, rms_eps=1e-6,
                   rope_base=10000.0, flags=0)
        cfg_dense = dict(cfg, flags=S.SPARK_DENSE_LOADS)
        layers.append((S.make_layer(w, cfg, cache), S.make_layer(w, cfg_dense, cache), w, cache))
    h_init = torch.randn(B, d, device=dev, generator=gen)
    h = torch.empty_like(h_init)
    cl = torch.full((B,), ctx_len + 1, dtype=torch.int32, device=dev)   # valid tokens, the one being decoded included
    scratch = torch.empty(S.layer_scratch_floats(dict(n_q=shape.n_q, n_kv=shape.n_kv, hd=hd, d=d), B), device=dev)
    h_host_in = h_init.cpu().pin_memory()
    h_host_out = torch.empty_like(h_host_in).pin_memory()
    # QKV (+ rotary, append: a kernel of their own for B >= 5), attention, output projection, FFN; for B >= 5 the projections
    # are two kernels each (prep, tcgen05 GEMM) and the FFN four (prep, scores, activation, output)
    kernels_per_layer = 4 if B <= 4 else 10

    def stack(which):
        for lay in layers:
            S.spark_layer_decode(ctx, lay[which], cl, h, B, scratch)

    # The library only enqueues kernels on the caller's stream, so a whole decode step can be
    # captured once into a CUDA graph and replayed per token (what a serving loop would do).
    graphs = {}
    side = torch.cuda.Stream()

    def capture_of(calls):
        with torch.cuda.stream(side):
            calls()                                        # warm-up outside capture (first-call set-up)
            side.synchronize()
            g = torch.cuda.CUDAGraph()
            with torch.cuda.graph(g, stream=side):
                calls()
        torch.cuda.synchronize()
        return g

    def capture():
        graphs.clear()
        if no_graph:
            return
        for which in ((0,) if no_dense else (0, 1)):
            graphs[which] = capture_of(lambda: stack(which))

    capture()
    overlap_on = bool(overlap)
    if overlap_on:
        # Launch overlap needs the GPU to itself (its blocks must all become resident).  Try it once; if a
        # block gave up waiting, go back to ordinary cooperative launches and say so in the result.
        for g in graphs.values():
            g.replay()
        stack(0)
        if ctx.device_status() != S.SPARK_OK:
            overlap_on = False
            ctx.set_launch_overlap(False)
            capture()

    def run_stack(which):
        if which in graphs:
            graphs[which].replay()
        else:
            stack(which)

    # One step decodes one token per sequence: the context grows by one (the lengths live on the device,
    # so the replayed graph follows them); every timed loop starts again right after the prompt.
    def step(which=0):
        h.copy_(h_init)                                   # device-to-device copy of the token's input
        run_stack(which)
        cl.add_(1)

    def step_e2e():
        h.copy_(h_host_in, non_blocking=True)             # pinned host -> device
        run_stack(0)
        cl.add_(1)
        h_host_out.copy_(h, non_blocking=True)            # device -> pinned host
        torch.cuda.current_stream().synchronize()

    def timed(fn, nsteps, warmup, reset=True):
        """Total ms of nsteps calls of fn (max over ranks) and the per-step statistics of this rank."""
        if reset:
            cl.fill_(ctx_len + 1)
        for _ in range(warmup):
            fn()
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()
        ev = [torch.cuda.Event(enable_timing=True) for _ in range(nsteps + 1)]
        ev[0].record()
        for i in range(nsteps):
            fn()
            ev[i + 1].record()
        torch.cuda.synchronize()
        if world > 1:
            dist.barrier()
        return max_over_ranks(ev[0].elapsed_time(ev[-1]), world, dev), step_stats(ev, torch)

    sampler = ClockSampler(dev.index)
    sampler.start()
    ms_total, st_total = timed(step, steps, W)
    clocks = sampler.stop()
    ms_e2e = timed(step_e2e, steps, W)[0] if with_e2e else None
    ms_dense, st_dense = (None, None) if no_dense else timed(lambda: step(1), steps, W)
    status = ctx.device_status()
    assert status == S.SPARK_OK, f"device status {status}"
    assert torch.isfinite(h).all()

    # ---- the kernels of a layer one by one, each as a CUDA graph of n_layers launches over the layers' own weights and
    #      caches (more data than L2 holds): FFN, attention, the two projections ------------------------------------
    peak, peak_kind = measured_peak()
    out = {"shape": shape_name, "batch": B, "ctx": ctx_len, "n_layers": n_layers, "kernels_per_layer": kernels_per_layer,
           "overlap_on": overlap_on, "ms_total": ms_total, "steps_ms": st_total, "ms_e2e": ms_e2e, "ms_dense": ms_dense,
           "steps_ms_dense": st_dense, "clocks": clocks,
           "h2d_bytes_per_step": int(h_host_in.numel() * 4), "d2h_bytes_per_step": int(h_host_out.numel() * 4)}
    xn = torch.nn.functional.normalize(h_init, dim=1) * (d ** 0.5)
    y = torch.empty_like(xn)
    cnt = torch.zeros(B, dtype=torch.int32, device=dev)
    idx = torch.zeros(B, shape.d_ff, dtype=torch.int32, device=dev)
    unions = []
    for lay in layers[: min(4, n_layers)]:
        w = lay[2]
        S.spark_ffn_decode(ctx, xn, B, w["K1t"], w["K2t"], w["Vt"], S.SPARK_BF16, d, shape.d_ff, shape.r_ff,
                           shape.k_ff, 0, y, None, cnt, idx)
        torch.cuda.synchronize()
        ids = torch.cat([idx[b, : int(cnt[b])] for b in range(B)])
        unions.append(int(torch.unique(ids).numel()))
    union = float(np.mean(unions))
    out["union_rows"] = union
    out["layer_touched_bytes"] = touched_layer_bytes(shape, B, ctx_len, union if B <= 4 else shape.d_ff, n_layers)
    if with_kernels:
        def loop_us(calls):
            g = None if no_graph else capture_of(calls)
            ms, st = timed(lambda: g.replay() if g is not None else calls(), steps, W, reset=False)
            return {"us_per_launch": ms * 1e3 / (steps * n_layers), "median_us": st["median"] * 1e3 / n_layers,
                    "min_us": st["min"] * 1e3 / n_layers}

        def entry(name, t, nbytes):
            t.update({"kernel": name, "bound": "hbm", "touched_bytes_per_launch": nbytes, "unit": "GB/s", "peak": peak,
                      "achieved": nbytes / (t["us_per_launch"] * 1e-6) / 1e9,
                      "frac": nbytes / (t["us_per_launch"] * 1e-6) / 1e9 / peak, "peak_kind": f"of {peak_kind}"})
            return t

        def ffn_calls():
            for lay in layers:
                w = lay[2]
                S.spark_ffn_decode(ctx, xn, B, w["K1t"], w["K2t"], w["Vt"], S.SPARK_BF16, d, shape.d_ff, shape.r_ff,
                                   shape.k_ff, 0, y, None, None, None)
        cl.fill_(ctx_len + 1)
        rows_read = union if B <= 4 else shape.d_ff
        out["ffn"] = entry(("ffn1_kernel" if B == 1 else "ffn_few_kernel" if B <= 4 else "ffn_tc_{prep,scores,act,out}_kernel") +
                           " (spark_ffn_decode)", loop_us(ffn_calls), shape.d_ff * shape.r_ff * 2 + rows_read * (2 * d - shape.r_ff) * 2)

        qa = torch.randn(B, shape.n_q, hd, device=dev, generator=gen) / (hd ** 0.5)
        oa = torch.empty(B, shape.n_q, hd, device=dev)

        def attn_calls():
            for l, lay in enumerate(layers):
                c = lay[3]
                win = 4096 if (l % 2 == 0 and ctx_len > 4096) else 0
                S.spark_attn_decode(ctx, qa, c["k1c"], c["k2c"], c["vc"], S.SPARK_BF16, B, shape.n_q, shape.n_kv, hd,
                                    shape.r_attn, cap, cl, win, shape.k_attn, 0, oa, None, None, None, 0)
        avg_ctx = (min(ctx_len, 4096) + ctx_len) / 2 if ctx_len > 4096 else ctx_len
        attn_bytes = B * (shape.n_kv * avg_ctx * shape.r_attn * 2 +
                          shape.n_q * min(shape.k_attn, avg_ctx) * ((hd - shape.r_attn) + hd) * 2)
        out["attn"] = entry("attn_kernel (spark_attn_decode)", loop_us(attn_calls), attn_bytes)

        yq = torch.empty(B, nqkv, device=dev)
        yo = torch.empty(B, d, device=dev)
        xo = torch.randn(B, shape.n_q * hd, device=dev, generator=gen)

        def qkv_calls():
            for lay in layers:
                S.spark_dense_gemv(ctx, xn, B, lay[2]["Wqkv"], S.SPARK_BF16, d, nqkv, None, yq)

        def wo_calls():
            for lay in layers:
                S.spark_dense_gemv(ctx, xo, B, lay[2]["Wo"], S.SPARK_BF16, shape.n_q * hd, d, None, yo)
        out["qkv_proj"] = entry("gemv_kernel / gemm_tc_kernel on Wqkv (spark_dense_gemv; the layer fuses norm, rotary, append)",
                                loop_us(qkv_calls), nqkv * d * 2)
        out["o_proj"] = entry("gemv_kernel / gemm_tc_kernel on Wo (spark_dense_gemv)", loop_us(wo_calls), d * shape.n_q * hd * 2)
        assert ctx.device_status() == S.SPARK_OK
    ctx.close()
    del layers, graphs
    torch.cuda.empty_cache()
    return out


def stack_summary(m, world, peak):
    """The reported figures of one measured stack (see measure_stack)."""
    steps_ms = m["steps_ms"]
    per = 1e3 / (m["n_layers"] * m["batch"] * world)          # ms per step -> us per token per layer
    n = m["n_layers"]
    us_layer_call = steps_ms["mean"] * 1e3 / n
    touched = m["layer_touched_bytes"]
    s = {"workload": f"gemma2-{m['shape']}-shape spark decoder, {n} layers, batch {m['batch']}, context {m['ctx']} "
                     "(local 4096 / global layers alternate), one CUDA graph replay per decode step",
         "us_per_token_per_layer": steps_ms["mean"] * per, "median_us_per_token_per_layer": steps_ms["median"] * per,
         "min_us_per_token_per_layer": steps_ms["min"] * per, "ms_per_step": steps_ms["mean"],
         "tokens_per_s": m["batch"] * world / (steps_ms["mean"] * 1e-3),
         "layer_touched_mb": touched / 1e6, "layer_gbs_touched": touched / (us_layer_call * 1e-6) / 1e9,
         "layer_frac_of_measured_peak": touched / (us_layer_call * 1e-6) / 1e9 / peak,
         "layer_frac_of_8tbs": touched / (us_layer_call * 1e-6) / 8e12,
         "union_rows_ffn": m["union_rows"], "launch_overlap": m["overlap_on"]}
    if m["ms_dense"] is not None:
        s["dense_loads"] = {"us_per_token_per_layer": m["steps_ms_dense"]["mean"] * per,
                            "median_us_per_token_per_layer": m["steps_ms_dense"]["median"] * per,
                            "speedup_spark_vs_dense_loads": m["ms_dense"] / m["ms_total"]}
    for k in ("ffn", "attn", "qkv_proj", "o_proj"):
        if k in m:
            s[k] = m[k]
    return s


def run_spark(args):
    import torch
    import torch.distributed as dist

    from paper_2506_06644_b200 import binding as S

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    if world > 1:
        dist.init_process_group("nccl", device_id=dev)

    shape = shape_of(args.shape)
    n_layers = args.layers or shape.n_layers
    B, ctx_len = args.batch, args.ctx
    W = max(args.warmup, 3)
    m = measure_stack(torch, S, dist, dev, rank, world, args.shape, B, ctx_len, n_layers, args.steps, W, args.overlap,
                      args.no_graph, args.no_dense, with_e2e=True, with_kernels=True)
    peak, peak_kind = measured_peak()
    line = None
    if rank == 0:
        s = stack_summary(m, world, peak)
        per = 1e3 / (n_layers * B * world)
        ffn = m["ffn"]
        line = {
            "metric": "us_per_token_per_layer", "value": us_per_token_per_layer(m["ms_total"], args.steps, n_layers, B, world),
            "unit": "us/token/layer", "n_gpus": world, "steps": args.steps, "warmup": W, "ms_per_step": m["ms_total"] / args.steps,
            "higher_is_better": False, "scaling": "weak", "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
            "config": {"workload": workload_name(args, shape), "l2": "weights+caches (>3 GB) exceed L2; no flush needed",
                       "parallelism": f"replicas x{world}" if world > 1 else "single GPU",
                       "launch": ("host launches" if args.no_graph else "one CUDA graph replay per decode step") +
                                 (", programmatic dependent launches (spark_set_launch_overlap)" if m["overlap_on"] else ""),
                       "local_window": 4096, "k_ff": shape.k_ff, "k_attn": shape.k_attn},
            "median_us_per_token_per_layer": s["median_us_per_token_per_layer"],
            "min_us_per_token_per_layer": s["min_us_per_token_per_layer"],
            "tokens_per_s": B * world * args.steps / (m["ms_total"] * 1e-3),
            "layer_touched_mb": s["layer_touched_mb"], "layer_gbs_touched": s["layer_gbs_touched"],
            "layer_frac_of_measured_peak": s["layer_frac_of_measured_peak"], "layer_frac_of_8tbs": s["layer_frac_of_8tbs"],
            "dense": None if m["ms_dense"] is None else {
                "us_per_token_per_layer": m["ms_dense"] / args.steps * per,
                "median_us_per_token_per_layer": m["steps_ms_dense"]["median"] * per,
                "speedup_spark_vs_dense": m["ms_dense"] / m["ms_total"]},
            "e2e": {"value": m["ms_e2e"] / args.steps * per, "unit": "us/token/layer",
                    "h2d_bytes_per_step": m["h2d_bytes_per_step"], "d2h_bytes_per_step": m["d2h_bytes_per_step"]},
            "gpu_launches": args.steps * n_layers * m["kernels_per_layer"],
            "clocks": m["clocks"],
            "roofline": {"kernel": ffn["kernel"], "bound": "hbm", "achieved": ffn["achieved"], "peak": peak, "unit": "GB/s",
                         "frac": ffn["frac"], "traffic": NCU_TRAFFIC_BYTES.get((args.shape, B)), "peak_kind": f"of {peak_kind}",
                         "us_per_launch": ffn["us_per_launch"], "median_us": ffn["median_us"], "min_us": ffn["min_us"],
                         "touched_bytes_per_launch": ffn["touched_bytes_per_launch"], "union_rows": m["union_rows"]},
            "roofline_attention": dict(m["attn"], traffic=None),
            "kernels": {k: m[k] for k in ("qkv_proj", "attn", "o_proj", "ffn")},
        }
        if not args.no_extra and world == 1 and args.shape == "2b" and B == 1:
            # the other halves of the target, in the same run: the 9B-shape stack at batch 1 and the 2B-shape stack at
            # batch 8 (eight sequences with their own 8192-token caches), each with its dense-loads comparator
            ex_steps = max(min(args.steps, 24), 4)
            line["stacks"] = []
            for shp, bb in (("9b", 1), ("2b", 8)):
                mm = measure_stack(torch, S, dist, dev, rank, world, shp, bb, ctx_len, shape_of(shp).n_layers, ex_steps, W,
                                   args.overlap, args.no_graph, False, with_e2e=False, with_kernels=True)
                line["stacks"].append(stack_summary(mm, world, peak))
            line["other_workloads"] = other_workloads(torch, S, peak, max(args.steps // 4, 4), W, with_oracle=not args.no_cpu)
        if not args.no_cpu and world == 1:
            line["cpu_baseline"] = cpu_baseline(args, shape)
    if world > 1:
        dist.barrier()
        dist.destroy_process_group()
    if line is not None:
        print(json.dumps(line), flush=True)


def other_workloads(torch, S, peak, steps, warmup, with_oracle=True):
    """The other configurations of the method, each timed alone with CUDA events around a CUDA graph of
    back-to-back launches that cycle over more data than L2 holds.  GB/s are touched bytes."""
    from paper_2506_06644_b200 import synth
    dev = torch.device("cuda", torch.cuda.current_device())
    gen = torch.Generator(device=dev)
    gen.manual_seed(99)
    sh = synth.GEMMA2_2B
    out = []

    def time_graph(calls, n_launch):
        side = torch.cuda.Stream()
        with torch.cuda.stream(side):
            calls()
            side.synchronize()
            g = torch.cuda.CUDAGraph()
            with torch.cuda.graph(g, stream=side):
                calls()
        torch.cuda.synchronize()
        for _ in range(warmup):
            g.replay()
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for _ in range(steps):
            g.replay()
        e1.record()
        torch.cuda.synchronize()
        return e0.elapsed_time(e1) * 1e3 / (steps * n_launch)

    def entry(name, us, nbytes, dense_us=None):
        e = {"workload": name, "us_per_launch": us, "touched_mb": nbytes / 1e6, "gbs_touched": nbytes / us / 1e3,
             "frac_of_measured_peak": nbytes / us / 1e3 / peak}
        if dense_us is not None:
            e["dense_loads_us_per_launch"] = dense_us
            e["speedup_vs_dense_loads"] = dense_us / us
        out.append(e)

    # -- Spark FFN, 4, 16 and 64 tokens, Gemma-2-2B shape, 8 weight sets (580 MB); from five tokens on the path reads every
    #    weight row (tcgen05 chunk kernels), so SPARK_DENSE_LOADS is the same run and the bytes are all of the weights
    def w(rows, cols):
        return (torch.randn(rows, cols, device=dev, generator=gen) * sh.d ** -0.5).to(torch.bfloat16)
    sets = [(w(sh.d_ff, sh.r_ff), w(sh.d_ff, sh.d - sh.r_ff), w(sh.d_ff, sh.d)) for _ in range(8)]
    for B in (4, 16, 64):
        ctx = S.SparkContext(dev.index, max_batch=B, max_dff=sh.d_ff, max_d=sh.d)
        ctx.set_launch_overlap(True)
        x = torch.randn(B, sh.d, device=dev, generator=gen)
        y = torch.empty(B, sh.d, device=dev)
        cnt = torch.zeros(B, dtype=torch.int32, device=dev)
        idx = torch.zeros(B, sh.d_ff, dtype=torch.int32, device=dev)
        S.spark_ffn_decode(ctx, x, B, *sets[0], S.SPARK_BF16, sh.d, sh.d_ff, sh.r_ff, sh.k_ff, 0, y, None, cnt, idx)
        torch.cuda.synchronize()
        union = int(torch.unique(torch.cat([idx[b, : int(cnt[b])] for b in range(B)])).numel())
        res = []
        for flags in (0, S.SPARK_DENSE_LOADS) if B <= 4 else (0,):
            def calls():
                for k1, k2, v in sets:
                    S.spark_ffn_decode(ctx, x, B, k1, k2, v, S.SPARK_BF16, sh.d, sh.d_ff, sh.r_ff, sh.k_ff, flags, y, None, None, None)
            res.append(time_graph(calls, len(sets)))
        assert ctx.device_status() == S.SPARK_OK
        rows_read = union if B <= 4 else sh.d_ff
        entry(f"spark_ffn_decode gemma2-2b shape, {B} tokens (union of active sets {union} of {sh.d_ff}" +
              (")" if B <= 4 else "; every row read)"), res[0],
              sh.d_ff * sh.r_ff * 2 + rows_read * (2 * sh.d - sh.r_ff) * 2, res[1] if B <= 4 else None)
        ctx.close()
    del sets

    # -- Spark FFN, one token, at the paper's iso-parameter width (Section 4: d_ff 13824, k 1106), 6 weight sets (600 MB)
    dffw, kw = 13824, 1106

    def ww(rows, cols):
        return (torch.randn(rows, cols, device=dev, generator=gen) * sh.d ** -0.5).to(torch.bfloat16)
    sets = [(ww(dffw, sh.r_ff), ww(dffw, sh.d - sh.r_ff), ww(dffw, sh.d)) for _ in range(6)]
    ctx = S.SparkContext(dev.index, max_batch=1, max_dff=dffw, max_d=sh.d)
    ctx.set_launch_overlap(True)
    x = torch.randn(1, sh.d, device=dev, generator=gen)
    y = torch.empty(1, sh.d, device=dev)
    cnt = torch.zeros(1, dtype=torch.int32, device=dev)
    S.spark_ffn_decode(ctx, x, 1, *sets[0], S.SPARK_BF16, sh.d, dffw, sh.r_ff, kw, 0, y, None, cnt, None)
    torch.cuda.synchronize()
    nact = int(cnt[0])
    res = []
    for flags in (0, S.SPARK_DENSE_LOADS):
        def calls():
            for k1, k2, v in sets:
                S.spark_ffn_decode(ctx, x, 1, k1, k2, v, S.SPARK_BF16, sh.d, dffw, sh.r_ff, kw, flags, y, None, None, None)
        res.append(time_graph(calls, len(sets)))
    assert ctx.device_status() == S.SPARK_OK
    entry(f"spark_ffn_decode at the paper's width: d {sh.d}, d_ff {dffw}, r {sh.r_ff}, k {kw}, 1 token ({nact} active)", res[0],
          dffw * sh.r_ff * 2 + nact * (2 * sh.d - sh.r_ff) * 2, res[1])
    ctx.close()
    del sets

    # -- Spark FFN, one token, FP8 E4M3 weights with one scale per neuron (quantisation on top of sparsity), 12 sets
    def q8(rows, cols):
        wf = torch.randn(rows, cols, device=dev, generator=gen) * sh.d ** -0.5
        sc = wf.abs().amax(dim=1) / 448.0
        return (wf / sc[:, None]).to(torch.float8_e4m3fn).view(torch.uint8), sc
    sets = [(q8(sh.d_ff, sh.r_ff), q8(sh.d_ff, sh.d - sh.r_ff), q8(sh.d_ff, sh.d)) for _ in range(12)]
    ctx = S.SparkContext(dev.index, max_batch=1, max_dff=sh.d_ff, max_d=sh.d)
    ctx.set_launch_overlap(True)
    x = torch.randn(1, sh.d, device=dev, generator=gen)
    y = torch.empty(1, sh.d, device=dev)
    cnt = torch.zeros(1, dtype=torch.int32, device=dev)
    (a, a_s), (b, b_s), (c, c_s) = sets[0]
    S.spark_ffn_decode_fp8(ctx, x, 1, a, a_s, b, b_s, c, c_s, sh.d, sh.d_ff, sh.r_ff, sh.k_ff, 0, y, None, cnt, None)
    torch.cuda.synchronize()
    nact = int(cnt[0])
    res = []
    for flags in (0, S.SPARK_DENSE_LOADS):
        def calls():
            for (a, a_s), (b, b_s), (c, c_s) in sets:
                S.spark_ffn_decode_fp8(ctx, x, 1, a, a_s, b, b_s, c, c_s, sh.d, sh.d_ff, sh.r_ff, sh.k_ff, flags, y, None, None, None)
        res.append(time_graph(calls, len(sets)))
    assert ctx.device_status() == S.SPARK_OK
    entry(f"spark_ffn_decode_fp8 gemma2-2b shape, 1 token, FP8 E4M3 weights + per-neuron scales ({nact} active)", res[0],
          sh.d_ff * sh.r_ff + nact * (2 * sh.d - sh.r_ff) + sh.d_ff * 4 + nact * 8, res[1])
    ctx.close()
    del sets

    # -- Spark attention, long contexts
    for B, L, nsets in ((1, 4096, 24), (1, 16384, 6), (1, 32768, 4), (8, 32768, 2)):
        ctx = S.SparkContext(dev.index, max_batch=B, max_cap=L, n_q=sh.n_q, hd=sh.hd)
        ctx.set_launch_overlap(True)
        caches = [tuple(torch.randn(B, sh.n_kv, L, wd, device=dev, generator=gen).to(torch.bfloat16)
                        for wd in (sh.r_attn, sh.hd - sh.r_attn, sh.hd)) for _ in range(nsets)]
        q = torch.randn(B, sh.n_q, sh.hd, device=dev, generator=gen) * sh.hd ** -0.5
        o = torch.empty(B, sh.n_q, sh.hd, device=dev)
        cl = torch.full((B,), L, dtype=torch.int32, device=dev)
        res = []
        for flags in (0, S.SPARK_DENSE_LOADS):
            def calls():
                for rep in range(2):
                    for k1c, k2c, vc in caches:
                        S.spark_attn_decode(ctx, q, k1c, k2c, vc, S.SPARK_BF16, B, sh.n_q, sh.n_kv, sh.hd, sh.r_attn, L, cl, 0,
                                            sh.k_attn, flags, o, None, None, None, 0)
            res.append(time_graph(calls, 2 * nsets))
        assert ctx.device_status() == S.SPARK_OK
        nbytes = B * (sh.n_kv * L * sh.r_attn * 2 + sh.n_q * sh.k_attn * (2 * sh.hd - sh.r_attn) * 2)
        entry(f"spark_attn_decode 8q/4kv heads hd 256, context {L}, batch {B}, k_attn {sh.k_attn}", res[0], nbytes, res[1])
        if (B, L) not in ((1, 16384), (8, 32768)):
            ctx.close()
            del caches
            continue
        # the same with the predictor slice of the cache in FP8 E4M3 (one scale per cached row)
        q8c = []
        for k1c, k2c, vc in caches:
            kf = k1c.float()
            sc = kf.abs().amax(dim=-1).clamp_min(1e-30) / 448.0
            q8c.append(((kf / sc[..., None]).to(torch.float8_e4m3fn).view(torch.uint8), sc, k2c, vc))
            del kf

        def calls8():
            for rep in range(2):
                for k1q, k1s, k2c, vc in q8c:
                    S.spark_attn_decode_fp8k(ctx, q, k1q, k1s, k2c, vc, B, sh.n_q, sh.n_kv, sh.hd, sh.r_attn, L, cl, 0, sh.k_attn, 0,
                                             o, None, None, None, 0)
        us8 = time_graph(calls8, 2 * nsets)
        assert ctx.device_status() == S.SPARK_OK
        nbytes8 = B * (sh.n_kv * L * (sh.r_attn + 4) + sh.n_q * sh.k_attn * (2 * sh.hd - sh.r_attn) * 2)
        entry(f"spark_attn_decode_fp8k (FP8 predictor slice), context {L}, batch {B}, k_attn {sh.k_attn}", us8, nbytes8)
        # the whole cache in FP8 E4M3: the gathered rows of the selected tokens are halved too
        def quant(t):
            tf = t.float()
            sc = tf.abs().amax(dim=-1).clamp_min(1e-30) / 448.0
            return (tf / sc[..., None]).to(torch.float8_e4m3fn).view(torch.uint8), sc
        q8kv = [(k1q, k1s) + quant(k2c) + quant(vc) for k1q, k1s, k2c, vc in q8c]

        def calls8kv():
            for rep in range(2):
                for k1q, k1s, k2q, k2s, vq, vs in q8kv:
                    S.spark_attn_decode_fp8kv(ctx, q, k1q, k1s, k2q, k2s, vq, vs, B, sh.n_q, sh.n_kv, sh.hd, sh.r_attn, L, cl, 0, sh.k_attn,
                                              0, o, None, None, None, 0)
        us8kv = time_graph(calls8kv, 2 * nsets)
        assert ctx.device_status() == S.SPARK_OK
        nbytes8kv = B * (sh.n_kv * L * (sh.r_attn + 4) + sh.n_q * sh.k_attn * (2 * sh.hd - sh.r_attn + 8))
        entry(f"spark_attn_decode_fp8kv (whole cache FP8), context {L}, batch {B}, k_attn {sh.k_attn}", us8kv, nbytes8kv)
        ctx.close()
        del caches, q8c, q8kv

    # -- eight layers of the decoder at batch 8 (eight sequences, 8192-token synthetic caches each)
    B, L, nl = 8, 8192, 8
    ctx = S.SparkContext(dev.index, max_batch=B, max_dff=sh.d_ff, max_cap=L, n_q=sh.n_q, hd=sh.hd, max_d=sh.d)
    ctx.set_launch_overlap(True)
    nqkv = (sh.n_q + 2 * sh.n_kv) * sh.hd

    def wm(rows, cols, fan_in):
        return (torch.randn(rows, cols, device=dev, generator=gen) * fan_in ** -0.5).to(torch.bfloat16)
    stacks = {0: [], S.SPARK_DENSE_LOADS: []}
    for l in range(nl):
        wts = dict(norm1=torch.ones(sh.d, device=dev), norm2=torch.ones(sh.d, device=dev), Wqkv=wm(nqkv, sh.d, sh.d),
                   Wo=wm(sh.d, sh.n_q * sh.hd, sh.n_q * sh.hd), K1t=wm(sh.d_ff, sh.r_ff, sh.d), K2t=wm(sh.d_ff, sh.d - sh.r_ff, sh.d),
                   Vt=wm(sh.d_ff, sh.d, sh.d))
        cache = dict(k1c=torch.randn(B, sh.n_kv, L, sh.r_attn, device=dev, generator=gen).to(torch.bfloat16),
                     k2c=torch.randn(B, sh.n_kv, L, sh.hd - sh.r_attn, device=dev, generator=gen).to(torch.bfloat16),
                     vc=torch.randn(B, sh.n_kv, L, sh.hd, device=dev, generator=gen).to(torch.bfloat16))
        for flags in stacks:
            cfg = dict(d=sh.d, d_ff=sh.d_ff, r_ff=sh.r_ff, k_ff=sh.k_ff, n_q=sh.n_q, n_kv=sh.n_kv, hd=sh.hd, r_attn=sh.r_attn,
                       k_attn=sh.k_attn, window=4096 if l % 2 == 0 else 0, cap=L, rms_eps=1e-6, rope_base=10000.0, flags=flags)
            stacks[flags].append((S.make_layer(wts, cfg, cache), wts, cache))
    h = torch.randn(B, sh.d, device=dev, generator=gen)
    cl = torch.full((B,), L, dtype=torch.int32, device=dev)
    scratch = torch.empty(B * (nqkv + 2 * sh.n_q * sh.hd + sh.d + 2 + sh.n_q), device=dev)
    res = []
    for flags in (0, S.SPARK_DENSE_LOADS):
        def calls():
            for lay in stacks[flags]:
                S.spark_layer_decode(ctx, lay[0], cl, h, B, scratch)
        res.append(time_graph(calls, nl))
    assert ctx.device_status() == S.SPARK_OK
    lens = [4096 if l % 2 == 0 else L for l in range(nl)]
    nbytes = sum((nqkv * sh.d + sh.d * sh.n_q * sh.hd + sh.d_ff * sh.r_ff) * 2 +
                 B * (sh.n_kv * n * sh.r_attn * 2 + sh.n_q * sh.k_attn * (2 * sh.hd - sh.r_attn) * 2) for n in lens) / nl
    out.append({"workload": f"spark_layer_decode gemma2-2b shape, batch {B}, context {L} (local 4096 / global), {nl} layers: "
                            "per layer; touched bytes without the FFN's gathered rows",
                "us_per_launch": res[0], "us_per_token_per_layer": res[0] / B, "touched_mb": nbytes / 1e6,
                "gbs_touched": nbytes / res[0] / 1e3, "frac_of_measured_peak": nbytes / res[0] / 1e3 / peak,
                "dense_loads_us_per_launch": res[1], "speedup_vs_dense_loads": res[1] / res[0]})
    ctx.close()

    # -- the same layers with quantised storage (the paper's closing section: quantisation compounds with activation sparsity):
    #    FP8 E4M3 predictor slice of the cache with row scales at batch 1 and 8; at batch 1 also FP8 FFN weights with per-neuron scales
    ctx = S.SparkContext(dev.index, max_batch=8, max_dff=sh.d_ff, max_cap=L, n_q=sh.n_q, hd=sh.hd, max_d=sh.d)
    ctx.set_launch_overlap(True)

    def q8rows(t):
        tf = t.float()
        sc = tf.abs().amax(dim=-1).clamp_min(1e-30) / 448.0
        return (tf / sc[..., None]).to(torch.float8_e4m3fn).view(torch.uint8), sc
    for Bq in (1, 8):
        qlayers = []
        for l, (_, wts, cache) in enumerate(stacks[0]):
            k1q, k1s = q8rows(cache["k1c"][:Bq])
            cq = dict(k1c=k1q.contiguous(), k1s=k1s.contiguous(), k2c=cache["k2c"][:Bq].contiguous(), vc=cache["vc"][:Bq].contiguous())
            wq = dict(wts)
            flags = S.SPARK_K1C_FP8
            if Bq <= 4:
                flags |= S.SPARK_FFN_FP8
                for nm, sn in (("K1t", "K1s"), ("K2t", "K2s"), ("Vt", "Vs")):
                    wq[nm], wq[sn] = q8rows(wts[nm])
            cfg = dict(d=sh.d, d_ff=sh.d_ff, r_ff=sh.r_ff, k_ff=sh.k_ff, n_q=sh.n_q, n_kv=sh.n_kv, hd=sh.hd, r_attn=sh.r_attn,
                       k_attn=sh.k_attn, window=4096 if l % 2 == 0 else 0, cap=L, rms_eps=1e-6, rope_base=10000.0, flags=flags)
            cfg_b = dict(cfg, flags=0)
            cb = dict(k1c=cache["k1c"][:Bq].contiguous(), k2c=cq["k2c"], vc=cq["vc"])
            qlayers.append((S.make_layer(wq, cfg, cq), S.make_layer(wts, cfg_b, cb), wq, cq, cb))
        hq = torch.randn(Bq, sh.d, device=dev, generator=gen)
        clq = torch.full((Bq,), L, dtype=torch.int32, device=dev)
        scq = torch.empty(S.layer_scratch_floats(dict(n_q=sh.n_q, n_kv=sh.n_kv, hd=sh.hd, d=sh.d), Bq), device=dev)
        r8 = []
        for which in (0, 1):
            def calls():
                for lay in qlayers:
                    S.spark_layer_decode(ctx, lay[which], clq, hq, Bq, scq)
            r8.append(time_graph(calls, nl))
        assert ctx.device_status() == S.SPARK_OK
        out.append({"workload": f"spark_layer_decode gemma2-2b shape with quantised storage, batch {Bq}, context {L}, {nl} layers: FP8 predictor "
                                "slice of the cache" + (" and FP8 FFN weights" if Bq <= 4 else " (FFN weights bf16: the chunk kernels take bf16)") +
                                "; per layer, beside the bf16 layer on the same inputs",
                    "us_per_launch": r8[0], "us_per_token_per_layer": r8[0] / Bq, "bf16_us_per_launch": r8[1],
                    "speedup_vs_bf16_storage": r8[1] / r8[0]})
        del qlayers
    ctx.close()

    # -- the same eight layers over chunks of a prompt: T consecutive tokens of ONE sequence per call (SPARK_SHARED_CACHE),
    #    appended behind 8192 - T cached tokens, every token attending causally; per-layer caches [n_kv][L][.]
    ctx = S.SparkContext(dev.index, max_batch=64, max_dff=sh.d_ff, max_cap=L, n_q=sh.n_q, hd=sh.hd, max_d=sh.d)
    ctx.set_launch_overlap(True)
    chunk_layers = []
    for l, (_, wts, cache) in enumerate(stacks[0]):
        one = {k: v[0] for k, v in cache.items()}             # the first sequence's cache of that layer
        cfg = dict(d=sh.d, d_ff=sh.d_ff, r_ff=sh.r_ff, k_ff=sh.k_ff, n_q=sh.n_q, n_kv=sh.n_kv, hd=sh.hd, r_attn=sh.r_attn,
                   k_attn=sh.k_attn, window=4096 if l % 2 == 0 else 0, cap=L, rms_eps=1e-6, rope_base=10000.0,
                   flags=S.SPARK_SHARED_CACHE)
        chunk_layers.append((S.make_layer(wts, cfg, one), wts, one))
    for T in (16, 64):
        hc = torch.randn(T, sh.d, device=dev, generator=gen)
        clc = torch.arange(L - T + 1, L + 1, dtype=torch.int32, device=dev)
        scratch_c = torch.empty(T * (nqkv + 2 * sh.n_q * sh.hd + sh.d + 2 + sh.n_q), device=dev)

        def chunk_calls():
            for lay in chunk_layers:
                S.spark_layer_decode(ctx, lay[0], clc, hc, T, scratch_c)
        us_chunk = time_graph(chunk_calls, nl)
        assert ctx.device_status() == S.SPARK_OK
        out.append({"workload": f"spark_layer_decode over a chunk of a prompt: {T} consecutive tokens of one sequence per call "
                                f"(shared cache, causal), context {L}, {nl} layers: per layer",
                    "us_per_launch": us_chunk, "us_per_token_per_layer": us_chunk / T})
    # -- a whole prompt: 4096 tokens from an empty cache through the eight layers in 64-token chunks (binding.spark_prefill:
    #    host loop, 64 x 8 layer calls of 13 kernels), timed with events around the loop
    Np = 4096
    hp = torch.randn(Np, sh.d, device=dev, generator=gen)
    lay_only = [c[0] for c in chunk_layers]
    S.spark_prefill(ctx, lay_only, hp[:256].clone(), 0, chunk=64)          # warm-up
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    S.spark_prefill(ctx, lay_only, hp, 0, chunk=64)
    e1.record()
    torch.cuda.synchronize()
    assert ctx.device_status() == S.SPARK_OK
    ms_pre = e0.elapsed_time(e1)
    out.append({"workload": f"spark_prefill: {Np} tokens from an empty cache through {nl} layers in 64-token chunks (host launches)",
                "us_per_launch": ms_pre * 1e3 / (Np // 64 * nl), "us_per_token_per_layer": ms_pre * 1e3 / (Np * nl),
                "prompt_tokens_per_s_per_layer_stack": Np / (ms_pre * 1e-3)})
    # -- the same prompt with two and three chunks in flight (spark_prefill_pipelined: a stream and a context per chunk in
    #    flight, a wavefront over (chunk, layer)); the caches are overwritten from row 0 again
    more = [S.SparkContext(dev.index, max_batch=64, max_dff=sh.d_ff, max_cap=L, n_q=sh.n_q, hd=sh.hd, max_d=sh.d) for _ in range(2)]
    sides = [torch.cuda.Stream(device=dev) for _ in more]
    for c in more:
        c.set_launch_overlap(True)
    for n_in in (2, 3):
        S.spark_prefill(ctx, lay_only, hp[:256].clone(), 0, chunk=64, more_ctx=more[:n_in - 1], more_streams=sides[:n_in - 1])      # warm-up
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        S.spark_prefill(ctx, lay_only, hp, 0, chunk=64, more_ctx=more[:n_in - 1], more_streams=sides[:n_in - 1])
        e1.record()
        torch.cuda.synchronize()
        assert ctx.device_status() == S.SPARK_OK and all(c.device_status() == S.SPARK_OK for c in more)
        ms_pipe = e0.elapsed_time(e1)
        out.append({"workload": f"spark_prefill_pipelined: the same {Np}-token prompt, {n_in} chunks in flight on {n_in} streams (host launches)",
                    "us_per_launch": ms_pipe * 1e3 / (Np // 64 * nl), "us_per_token_per_layer": ms_pipe * 1e3 / (Np * nl),
                    "prompt_tokens_per_s_per_layer_stack": Np / (ms_pipe * 1e-3), "speedup_vs_one_chunk_at_a_time": ms_pre / ms_pipe})
    for c in more:
        c.close()
    ctx.close()
    del stacks, chunk_layers

    # -- the LM head as a plain GEMV over the tied embedding (256000 x d, bf16: 1.18 GB at the 2B shape, 1.84 GB at 9B), one token
    for name, dm in (("2b", synth.GEMMA2_2B.d), ("9b", synth.GEMMA2_9B.d)):
        vocab = synth.GEMMA2_2B.vocab
        ctx = S.SparkContext(dev.index, max_batch=1, max_d=dm)
        ctx.set_launch_overlap(True)
        E = torch.randn(vocab, dm, device=dev, generator=gen).to(torch.bfloat16)
        xh = torch.randn(1, dm, device=dev, generator=gen)
        logits = torch.empty(1, vocab, device=dev)
        us = time_graph(lambda: [S.spark_dense_gemv(ctx, xh, 1, E, S.SPARK_BF16, dm, vocab, None, logits) for _ in range(2)], 2)
        assert ctx.device_status() == S.SPARK_OK
        entry(f"LM head: spark_dense_gemv {vocab} x {dm} bf16 (gemma2-{name} shape), one token", us, vocab * dm * 2)
        ctx.close()
        del E

    # -- statistical top-k, 4096 rows x 65536 (1.07 GB read per launch): three distributions x k/n in {2, 8, 25} %
    ctx = S.SparkContext(dev.index)
    rows, n = 4096, 65536
    theta = torch.empty(rows, device=dev)
    count = torch.empty(rows, dtype=torch.int32, device=dev)

    def draw(dist):
        if dist == "N(0,1)":
            return torch.randn(rows, n, device=dev, generator=gen)
        if dist == "Laplace(0,1)":
            u = torch.rand(rows, n, device=dev, generator=gen)
            return torch.where(u < 0.5, torch.log(2 * u), -torch.log(2 * (1 - u))).clamp_(-80, 80)
        z = torch.randn(rows, n, device=dev, generator=gen)                  # Student-t(4) = Z / sqrt(chi2_4 / 4)
        chi = torch.zeros(rows, n, device=dev)
        for _ in range(4):
            chi += torch.randn(rows, n, device=dev, generator=gen) ** 2
        return z / torch.sqrt(chi / 4)

    for dist in ("N(0,1)", "Laplace(0,1)", "Student-t(4)"):
        xs = draw(dist)
        for kk in (1311, 5243, 16384):
            us = time_graph(lambda: S.spark_stat_topk(ctx, xs, rows, n, n, kk, S.SPARK_FILL_ZERO, theta, count, None, None, 0, None), 1)
            entry(f"spark_stat_topk {rows} x {n} fp32 {dist}, k/n = {kk / n:.0%}, theta + count", us, rows * n * 4)
            c = count.float()
            out[-1].update({"k": kk, "selected_mean": float(c.mean()), "selected_std": float(c.std()),
                            "selected_min": int(count.min()), "selected_max": int(count.max())})
            if with_oracle:          # theta of eight sampled rows against the oracle (relative to max(|theta|, std) of the row)
                from oracle import spark_oracle as O
                worst = 0.0
                for rr in range(0, rows, rows // 8):
                    xr = xs[rr].cpu().numpy()
                    th, mask, _ = O.stat_topk(xr, kk)
                    worst = max(worst, abs(float(theta[rr]) - th) / max(abs(th), float(np.std(xr.astype(np.float64), ddof=1))))
                    assert abs(int(count[rr]) - int(mask.sum())) <= 2
                out[-1]["theta_max_rel_err_vs_oracle_8_rows"] = worst
        if dist == "N(0,1)":
            yd = torch.empty(rows, n, device=dev)
            us = time_graph(lambda: S.spark_stat_topk(ctx, xs, rows, n, n, 5243, S.SPARK_FILL_ZERO, theta, count, None, None, 0, yd), 1)
            entry(f"spark_stat_topk {rows} x {n} fp32 N(0,1), k/n = 8%, dense output (Eq. 10)", us, 2 * rows * n * 4)
            del yd
            cap = 4 * 1311
            idx = torch.empty(rows, cap, dtype=torch.int32, device=dev)
            val = torch.empty(rows, cap, device=dev)
            us = time_graph(lambda: S.spark_stat_topk(ctx, xs, rows, n, n, 1311, S.SPARK_FILL_ZERO, theta, count, idx, val, cap, None), 1)
            entry(f"spark_stat_topk {rows} x {n} fp32 N(0,1), k/n = 2%, ordered index and value lists", us,
                  rows * n * 4 + int(count.sum().item()) * 8)
            del idx, val
        del xs
    assert ctx.device_status() == S.SPARK_OK
    ctx.close()
    return out



def touched_layer_bytes(shape, B, ctx_len, union_ffn, n_layers):
    """Algorithmic bytes of one layer: dense projections, full predictor slices, active rows."""
    d, hd = shape.d, shape.hd
    proj = ((shape.n_q + 2 * shape.n_kv) * hd * d + d * shape.n_q * hd) * 2
    ffn = shape.d_ff * shape.r_ff * 2 + union_ffn * (2 * d - shape.r_ff) * 2
    win_local = min(ctx_len, 4096)
    avg_ctx = (win_local + ctx_len) / 2 if ctx_len > 4096 else ctx_len
    attn = B * (shape.n_kv * avg_ctx * shape.r_attn * 2 +
                shape.n_q * min(shape.k_attn, avg_ctx) * ((hd - shape.r_attn) + hd) * 2)
    return proj + ffn + attn


def cpu_baseline(args, shape):
    """The oracle as it stands on the host cores: all the threads its numpy build uses, and pinned to one thread."""
    n_l = 2
    layers, h = oracle_sample(shape, args.ctx, n_l)
    oracle_run(shape, layers[:1], h, args.ctx)            # touch the pages once

    def timed_reps(budget_s, max_reps):
        reps, t0 = 0, time.perf_counter()
        while True:
            oracle_run(shape, layers, h, args.ctx)
            reps += 1
            if time.perf_counter() - t0 > budget_s or reps >= max_reps:
                break
        return (time.perf_counter() - t0) / (reps * n_l) * 1e6, reps

    us_all, reps = timed_reps(10.0, 40)
    out = {"value": us_all, "unit": "us/token/layer", "cores": host_threads(), "kind": "oracle",
           "sample": f"{reps} x {n_l} decoder layers of one token at context {args.ctx} (fp64 numpy)"}
    try:
        from threadpoolctl import threadpool_limits
        with threadpool_limits(limits=1):
            us_one, reps1 = timed_reps(6.0, 10)
        out["single_thread"] = {"value": us_one, "unit": "us/token/layer", "cores": 1,
                                "sample": f"{reps1} x {n_l} decoder layers, numpy limited to one thread"}
    except Exception:
        pass
    return out


def batch_study(args):
    """Spark FFN over 1..64 tokens at the 2B shape, independent and correlated tokens (a common direction plus 30 % individual
    noise: what a speculative-verify batch looks like), sparse against SPARK_DENSE_LOADS, 8 rotating weight sets, CUDA-graph
    replay with launch overlap.  From five tokens on the library reads every row (tensor-core chunk kernels), so both columns are
    the same kernels there.  Prints one JSON line."""
    import torch

    from paper_2506_06644_b200 import binding as S
    from paper_2506_06644_b200 import synth
    dev = torch.device("cuda", 0)
    torch.cuda.set_device(0)
    gen = torch.Generator(device=dev)
    gen.manual_seed(7)
    sh = synth.GEMMA2_2B

    def w(rows, cols):
        return (torch.randn(rows, cols, device=dev, generator=gen) * sh.d ** -0.5).to(torch.bfloat16)
    sets = [(w(sh.d_ff, sh.r_ff), w(sh.d_ff, sh.d - sh.r_ff), w(sh.d_ff, sh.d)) for _ in range(8)]
    rows = []
    for B in (1, 2, 3, 4, 8, 16, 64):
        ctx = S.SparkContext(0, max_batch=B, max_dff=sh.d_ff, max_d=sh.d)
        ctx.set_launch_overlap(True)
        for kind in ("independent", "correlated"):
            x = torch.randn(B, sh.d, device=dev, generator=gen)
            if kind == "correlated":
                x = torch.randn(1, sh.d, device=dev, generator=gen) + 0.3 * x
            x = x / x.pow(2).mean(dim=1, keepdim=True).sqrt()
            y = torch.empty(B, sh.d, device=dev)
            cnt = torch.zeros(B, dtype=torch.int32, device=dev)
            idx = torch.zeros(B, sh.d_ff, dtype=torch.int32, device=dev)
            S.spark_ffn_decode(ctx, x, B, *sets[0], S.SPARK_BF16, sh.d, sh.d_ff, sh.r_ff, sh.k_ff, 0, y, None, cnt, idx)
            torch.cuda.synchronize()
            union = int(torch.unique(torch.cat([idx[b, : int(cnt[b])] for b in range(B)])).numel())
            us = []
            for flags in (0, S.SPARK_DENSE_LOADS):
                def calls():
                    for k1, k2, v in sets:
                        S.spark_ffn_decode(ctx, x, B, k1, k2, v, S.SPARK_BF16, sh.d, sh.d_ff, sh.r_ff, sh.k_ff, flags, y, None, None, None)
                side = torch.cuda.Stream()
                with torch.cuda.stream(side):
                    calls()
                    side.synchronize()
                    g = torch.cuda.CUDAGraph()
                    with torch.cuda.graph(g, stream=side):
                        calls()
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
                us.append(e0.elapsed_time(e1) * 1e3 / (30 * len(sets)))
            assert ctx.device_status() == S.SPARK_OK
            rows.append({"tokens": B, "inputs": kind, "union_rows": union, "union_frac": union / sh.d_ff, "sparse_us": us[0],
                         "dense_loads_us": us[1], "speedup": us[1] / us[0], "us_per_token": us[0] / B})
            if B == 1:
                break
        ctx.close()
    print(json.dumps({"study": "batch", "shape": "gemma2-2b FFN (d 2304, d_ff 9216, r 1024, k 737)", "rows": rows}), flush=True)


def main():
    args = parse()
    if args.study == "batch":
        return batch_study(args)
    if args.impl == "reference":
        run_reference(args)
    else:
        run_spark(args)


if __name__ == "__main__":
    main()
