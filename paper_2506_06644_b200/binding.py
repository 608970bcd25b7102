"""ctypes binding of libspark_b200.so: argument marshalling only.

Every function below has the name and the argument order of its C entry point in
include/spark.h and does nothing but turn torch tensors into device pointers, pass the
current CUDA stream, and raise on a non-zero status.  torch is used for device memory and
streams; every step of the computation runs in the library's kernels.  There is no CPU
fallback: a missing library or a missing GPU is an error.
"""
from __future__ import annotations

import ctypes as C
import os
from dataclasses import dataclass

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libspark_b200.so")

SPARK_OK = 0
SPARK_ERR_INVALID_ARG, SPARK_ERR_UNSUPPORTED, SPARK_ERR_WORKSPACE, SPARK_ERR_CUDA = 1, 2, 3, 4
SPARK_ERR_TIMEOUT, SPARK_ERR_OVERFLOW, SPARK_ERR_NONFINITE = 5, 6, 7
SPARK_F32, SPARK_BF16, SPARK_FP8_E4M3 = 0, 1, 2
SPARK_FILL_ZERO, SPARK_FILL_NEGINF = 0, 1
SPARK_GELU_TANH, SPARK_GELU_ERF, SPARK_DENSE_LOADS, SPARK_SHARED_CACHE, SPARK_CHECK_FINITE = 0, 1, 2, 4, 8
SPARK_FFN_FP8, SPARK_K1C_FP8 = 16, 32

EXPORTS = [
    "spark_status_string", "spark_normal_upper_quantile", "spark_workspace_bytes", "spark_create",
    "spark_destroy", "spark_device_status", "spark_grid_size", "spark_set_phase_trace", "spark_set_launch_overlap", "spark_stat_topk", "spark_ffn_decode",
    "spark_attn_decode", "spark_dense_gemv", "spark_layer_decode", "spark_ffn_decode_noalloc", "spark_ffn_decode_fp8", "spark_attn_decode_fp8k",
    "spark_stat_moments", "spark_stat_merge", "spark_stat_select",
    "spark_set_wait_limit", "spark_debug_expect_arrivals", "spark_noalloc_status",
    "spark_stack_decode", "spark_set_fused_layer", "spark_set_l2_prefetch", "spark_prefill", "spark_attn_decode_fp8kv", "spark_set_chunk_dense", "spark_prefill_pipelined",
]


class SparkError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        super().__init__(f"{where}: status {status} ({status_string(status)})")


class _LayerWeights(C.Structure):
    _fields_ = [(n, C.c_void_p) for n in ("norm1", "norm2", "Wqkv", "Wo", "K1t", "K2t", "Vt", "K1s", "K2s", "Vs")]


class _LayerCfg(C.Structure):
    _fields_ = [(n, C.c_int64) for n in ("d", "d_ff", "r_ff", "k_ff", "n_q", "n_kv", "hd", "r_attn", "k_attn",
                                         "window", "cap")] + \
               [("rms_eps", C.c_float), ("rope_base", C.c_float), ("flags", C.c_int)]


class _KvCache(C.Structure):
    _fields_ = [(n, C.c_void_p) for n in ("k1c", "k2c", "vc", "k1s")]


_lib = None


def lib() -> C.CDLL:
    """Load the shared library (built in-tree by paper_2506_06644_b200.build); fail loudly if absent."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(LIB_PATH):
        raise RuntimeError(f"{LIB_PATH} is missing: run `python -m paper_2506_06644_b200.build` "
                           "(there is no fallback path)")
    L = C.CDLL(LIB_PATH)
    vp, i64, i32, f64 = C.c_void_p, C.c_int64, C.c_int, C.c_double
    sig = {
        "spark_status_string": (C.c_char_p, [i32]),
        "spark_normal_upper_quantile": (f64, [f64]),
        "spark_workspace_bytes": (C.c_size_t, [i64] * 6),
        "spark_create": (i32, [C.POINTER(vp), i32, vp, C.c_size_t]),
        "spark_destroy": (i32, [vp]),
        "spark_device_status": (i32, [vp, vp, C.POINTER(i32)]),
        "spark_grid_size": (i32, [vp]),
        "spark_set_phase_trace": (i32, [vp, vp, i64]),
        "spark_set_launch_overlap": (i32, [vp, i32]),
        "spark_set_wait_limit": (i32, [vp, vp, i64]),
        "spark_debug_expect_arrivals": (i32, [vp, i32]),
        "spark_noalloc_status": (i32, [vp, C.POINTER(i32)]),
        "spark_stat_topk": (i32, [vp, vp, i64, i64, i64, i64, i32, vp, vp, vp, vp, i64, vp, vp]),
        "spark_stat_moments": (i32, [vp, vp, i64, i64, i64, vp, vp]),
        "spark_stat_merge": (i32, [vp, vp, i64, i64, i64, i64, vp, vp, vp]),
        "spark_stat_select": (i32, [vp, vp, i64, i64, i64, vp, i32, vp, vp, vp, i64, vp, vp]),
        "spark_ffn_decode": (i32, [vp, vp, i64, vp, vp, vp, i32, i64, i64, i64, i64, i32, vp, vp, vp, vp, vp]),
        "spark_ffn_decode_noalloc": (i32, [vp, i64, vp, vp, vp, i32, i64, i64, i64, i64, i32, vp, vp, vp]),
        "spark_ffn_decode_fp8": (i32, [vp, vp, i64, vp, vp, vp, vp, vp, vp, i64, i64, i64, i64, i32, vp, vp, vp, vp, vp]),
        "spark_attn_decode": (i32, [vp, vp, vp, vp, vp, i32, i64, i64, i64, i64, i64, i64, vp, i64, i64, i32,
                                    vp, vp, vp, vp, i64, vp]),
        "spark_attn_decode_fp8k": (i32, [vp, vp, vp, vp, vp, vp, i64, i64, i64, i64, i64, i64, vp, i64, i64, i32,
                                         vp, vp, vp, vp, i64, vp]),
        "spark_attn_decode_fp8kv": (i32, [vp, vp, vp, vp, vp, vp, vp, vp, i64, i64, i64, i64, i64, i64, vp, i64, i64, i32,
                                          vp, vp, vp, vp, i64, vp]),
        "spark_dense_gemv": (i32, [vp, vp, i64, vp, i32, i64, i64, vp, vp, vp]),
        "spark_stack_decode": (i32, [vp, C.POINTER(_LayerWeights), C.POINTER(_LayerCfg), C.POINTER(_KvCache), i64,
                                     vp, vp, i64, vp, vp]),
        "spark_set_fused_layer": (i32, [vp, i32]),
        "spark_set_chunk_dense": (i32, [vp, i32]),
        "spark_prefill": (i32, [vp, C.POINTER(_LayerWeights), C.POINTER(_LayerCfg), C.POINTER(_KvCache), i64, vp, i64, i64, i64, vp, vp, vp]),
        "spark_prefill_pipelined": (i32, [C.POINTER(vp), C.POINTER(vp), C.POINTER(vp), i64, C.POINTER(_LayerWeights), C.POINTER(_LayerCfg),
                                          C.POINTER(_KvCache), i64, vp, i64, i64, i64, vp]),
        "spark_set_l2_prefetch": (i32, [vp, i32]),
        "spark_layer_decode": (i32, [vp, C.POINTER(_LayerWeights), C.POINTER(_LayerCfg), C.POINTER(_KvCache),
                                     vp, vp, i64, vp, vp]),
    }
    assert sorted(sig) == sorted(EXPORTS)
    for name, (res, args) in sig.items():
        fn = getattr(L, name, None)       # a missing symbol surfaces at its first call
        if fn is not None:
            fn.restype, fn.argtypes = res, args
    _lib = L
    return L


def status_string(status: int) -> str:
    return lib().spark_status_string(status).decode()


def spark_normal_upper_quantile(p: float) -> float:
    return lib().spark_normal_upper_quantile(p)


def _ptr(t) -> int | None:
    if t is None:
        return None
    if not t.is_cuda or not t.is_contiguous():
        raise ValueError("tensors passed to the library must be contiguous CUDA tensors")
    return t.data_ptr()


def _stream() -> int:
    return torch.cuda.current_stream().cuda_stream


def _check(status: int, where: str):
    if status != SPARK_OK:
        raise SparkError(status, where)


def _dtype_code(t: torch.Tensor) -> int:
    if t.dtype == torch.float32:
        return SPARK_F32
    if t.dtype == torch.bfloat16:
        return SPARK_BF16
    raise ValueError(f"unsupported weight dtype {t.dtype}")


def spark_workspace_bytes(max_batch: int, max_dff: int, max_cap: int, n_q: int, hd: int, max_d: int) -> int:
    return lib().spark_workspace_bytes(max_batch, max_dff, max_cap, n_q, hd, max_d)


class SparkContext:
    """spark_create / spark_destroy around a torch-allocated workspace."""

    def __init__(self, device: int = 0, max_batch: int = 16, max_dff: int = 16384, max_cap: int = 32768,
                 n_q: int = 16, hd: int = 256, max_d: int = 4096):
        if not torch.cuda.is_available():
            raise RuntimeError("the Spark decode library needs a CUDA device (no CPU fallback)")
        self.device = device
        nbytes = spark_workspace_bytes(max_batch, max_dff, max_cap, n_q, hd, max_d)
        with torch.cuda.device(device):
            self.workspace = torch.zeros(nbytes + 256, dtype=torch.uint8, device=f"cuda:{device}")
            base = self.workspace.data_ptr()
            self._ws_ptr = (base + 255) // 256 * 256
            h = C.c_void_p()
            _check(lib().spark_create(C.byref(h), device, self._ws_ptr, nbytes), "spark_create")
        self.handle = h

    def device_status(self) -> int:
        out = C.c_int(0)
        _check(lib().spark_device_status(self.handle, _stream(), C.byref(out)), "spark_device_status")
        return out.value

    def set_phase_trace(self, trace):
        """trace: int64/uint64 CUDA tensor of grid_size * 16 entries, or None to switch tracing off."""
        n = 0 if trace is None else trace.numel()
        _check(lib().spark_set_phase_trace(self.handle, _ptr(trace), n), "spark_set_phase_trace")
        self._trace = trace

    def set_launch_overlap(self, on: bool):
        """Launch every kernel of this context so that it may start under the tail of the kernel before it."""
        _check(lib().spark_set_launch_overlap(self.handle, 1 if on else 0), "spark_set_launch_overlap")

    def set_wait_limit(self, cycles: int):
        """Bound of the waits between thread blocks in SM cycles (0 = the default of about two seconds)."""
        _check(lib().spark_set_wait_limit(self.handle, _stream(), cycles), "spark_set_wait_limit")

    def set_fused_layer(self, on: bool):
        """One-token layer calls: the fused persistent kernel, or the kernel-per-step path (default)."""
        _check(lib().spark_set_fused_layer(self.handle, 1 if on else 0), "spark_set_fused_layer")

    def set_chunk_dense(self, mode: int):
        """Prompt chunks, second stage of the attention: 0 gather per (token, head), 1 masked dense products on the tensor
        cores where they measured faster (default), 2 wherever they serve the shape."""
        _check(lib().spark_set_chunk_dense(self.handle, int(mode)), "spark_set_chunk_dense")

    def set_l2_prefetch(self, on: bool):
        """Kernels of a one-token layer call ask L2 for the next kernel's weights (default off: it measured slower)."""
        _check(lib().spark_set_l2_prefetch(self.handle, 1 if on else 0), "spark_set_l2_prefetch")

    def debug_expect_arrivals(self, extra: int):
        """Test hook: the one-token FFN kernel waits for `extra` arrivals that never come (0 = off)."""
        _check(lib().spark_debug_expect_arrivals(self.handle, extra), "spark_debug_expect_arrivals")

    @property
    def grid_size(self) -> int:
        return lib().spark_grid_size(self.handle)

    def close(self):
        if self.handle is not None:
            lib().spark_destroy(self.handle)
            self.handle = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass


def spark_stat_moments(ctx: SparkContext, x, rows, n, ld, moments):
    _check(lib().spark_stat_moments(ctx.handle, _ptr(x), rows, n, ld, _ptr(moments), _stream()), "spark_stat_moments")


def spark_stat_merge(ctx: SparkContext, parts, m, rows, k, n_total, theta, merged):
    _check(lib().spark_stat_merge(ctx.handle, _ptr(parts), m, rows, k, n_total, _ptr(theta), _ptr(merged), _stream()),
           "spark_stat_merge")


def spark_stat_select(ctx: SparkContext, x, rows, n, ld, theta_in, fill, count, idx, val, idx_cap, y_dense):
    _check(lib().spark_stat_select(ctx.handle, _ptr(x), rows, n, ld, _ptr(theta_in), fill, _ptr(count), _ptr(idx), _ptr(val),
                                   idx_cap, _ptr(y_dense), _stream()), "spark_stat_select")


def spark_stat_topk(ctx: SparkContext, x, rows, n, ld, k, fill, theta, count, idx, val, idx_cap, y_dense):
    _check(lib().spark_stat_topk(ctx.handle, _ptr(x), rows, n, ld, k, fill, _ptr(theta), _ptr(count), _ptr(idx),
                                 _ptr(val), idx_cap, _ptr(y_dense), _stream()), "spark_stat_topk")


def spark_ffn_decode(ctx: SparkContext, x, B, K1t, K2t, Vt, wdtype, d, d_ff, r, k, flags, y, theta, count, idx):
    _check(lib().spark_ffn_decode(ctx.handle, _ptr(x), B, _ptr(K1t), _ptr(K2t), _ptr(Vt), wdtype, d, d_ff, r, k,
                                  flags, _ptr(y), _ptr(theta), _ptr(count), _ptr(idx), _stream()), "spark_ffn_decode")


def spark_ffn_decode_fp8(ctx: SparkContext, x, B, K1t, K1s, K2t, K2s, Vt, Vs, d, d_ff, r, k, flags, y, theta, count, idx):
    _check(lib().spark_ffn_decode_fp8(ctx.handle, _ptr(x), B, _ptr(K1t), _ptr(K1s), _ptr(K2t), _ptr(K2s), _ptr(Vt), _ptr(Vs), d,
                                      d_ff, r, k, flags, _ptr(y), _ptr(theta), _ptr(count), _ptr(idx), _stream()), "spark_ffn_decode_fp8")


def spark_ffn_decode_noalloc(x, B, K1t, K2t, Vt, wdtype, d, d_ff, r, k, flags, y, theta):
    """spark_ffn_decode for callers that must not allocate: no context, no workspace; the kernel's
    inter-block state lives in a fixed array inside the library (see include/spark.h).  B <= 16."""
    _check(lib().spark_ffn_decode_noalloc(_ptr(x), B, _ptr(K1t), _ptr(K2t), _ptr(Vt), wdtype, d, d_ff, r, k, flags,
                                          _ptr(y), _ptr(theta), _stream()), "spark_ffn_decode_noalloc")


def spark_noalloc_status() -> int:
    """Device status of the no-allocation entry point on the current device (resets its state after an error)."""
    out = C.c_int(0)
    _check(lib().spark_noalloc_status(_stream(), C.byref(out)), "spark_noalloc_status")
    return out.value


def spark_attn_decode(ctx: SparkContext, q, k1c, k2c, vc, kvdtype, B, n_q, n_kv, hd, r, cap, ctx_len, window,
                      k_attn, flags, o, theta, count, idx, idx_cap):
    _check(lib().spark_attn_decode(ctx.handle, _ptr(q), _ptr(k1c), _ptr(k2c), _ptr(vc), kvdtype, B, n_q, n_kv, hd,
                                   r, cap, _ptr(ctx_len), window, k_attn, flags, _ptr(o), _ptr(theta), _ptr(count),
                                   _ptr(idx), idx_cap, _stream()), "spark_attn_decode")


def spark_attn_decode_fp8k(ctx: SparkContext, q, k1c, k1s, k2c, vc, B, n_q, n_kv, hd, r, cap, ctx_len, window, k_attn, flags,
                           o, theta, count, idx, idx_cap):
    _check(lib().spark_attn_decode_fp8k(ctx.handle, _ptr(q), _ptr(k1c), _ptr(k1s), _ptr(k2c), _ptr(vc), B, n_q, n_kv, hd, r, cap,
                                        _ptr(ctx_len), window, k_attn, flags, _ptr(o), _ptr(theta), _ptr(count), _ptr(idx), idx_cap,
                                        _stream()), "spark_attn_decode_fp8k")


def spark_attn_decode_fp8kv(ctx: SparkContext, q, k1c, k1s, k2c, k2s, vc, vs, B, n_q, n_kv, hd, r, cap, ctx_len, window, k_attn, flags,
                            o, theta, count, idx, idx_cap):
    _check(lib().spark_attn_decode_fp8kv(ctx.handle, _ptr(q), _ptr(k1c), _ptr(k1s), _ptr(k2c), _ptr(k2s), _ptr(vc), _ptr(vs), B, n_q, n_kv,
                                         hd, r, cap, _ptr(ctx_len), window, k_attn, flags, _ptr(o), _ptr(theta), _ptr(count), _ptr(idx),
                                         idx_cap, _stream()), "spark_attn_decode_fp8kv")


def spark_dense_gemv(ctx: SparkContext, x, B, Wt, wdtype, n_in, n_out, y_add, y):
    _check(lib().spark_dense_gemv(ctx.handle, _ptr(x), B, _ptr(Wt), wdtype, n_in, n_out, _ptr(y_add), _ptr(y),
                                  _stream()), "spark_dense_gemv")


@dataclass
class LayerHandles:
    """Host-side structs of spark_layer_decode, built once per layer (they only hold pointers)."""
    weights: _LayerWeights
    cfg: _LayerCfg
    cache: _KvCache
    keep: tuple            # tensors kept alive


def make_layer(weights: dict, cfg: dict, cache: dict) -> LayerHandles:
    w = _LayerWeights(**{k: _ptr(weights.get(k)) for k in ("norm1", "norm2", "Wqkv", "Wo", "K1t", "K2t", "Vt", "K1s", "K2s", "Vs")})
    c = _LayerCfg(**cfg)
    kv = _KvCache(**{k: _ptr(cache.get(k)) for k in ("k1c", "k2c", "vc", "k1s")})
    return LayerHandles(w, c, kv, (weights, cache))


def spark_layer_decode(ctx: SparkContext, layer: LayerHandles, ctx_len, h, B, scratch):
    _check(lib().spark_layer_decode(ctx.handle, C.byref(layer.weights), C.byref(layer.cfg), C.byref(layer.cache),
                                    _ptr(ctx_len), _ptr(h), B, _ptr(scratch), _stream()), "spark_layer_decode")


@dataclass
class StackHandles:
    """Host arrays of the per-layer structs of spark_stack_decode (they only hold pointers)."""
    weights: object
    cfgs: object
    caches: object
    n_layers: int
    keep: tuple


def make_stack(layers) -> StackHandles:
    """layers: LayerHandles of the stack's layers, first to last."""
    n = len(layers)
    w = (_LayerWeights * n)(*[l.weights for l in layers])
    c = (_LayerCfg * n)(*[l.cfg for l in layers])
    kv = (_KvCache * n)(*[l.cache for l in layers])
    return StackHandles(w, c, kv, n, tuple(layers))


def spark_stack_decode(ctx: SparkContext, stack: StackHandles, ctx_len, h, B, scratch):
    _check(lib().spark_stack_decode(ctx.handle, stack.weights, stack.cfgs, stack.caches, stack.n_layers, _ptr(ctx_len), _ptr(h), B,
                                    _ptr(scratch), _stream()), "spark_stack_decode")


def layer_scratch_floats(cfg: dict, B: int) -> int:
    """fp32 elements of scratch spark_layer_decode needs for B tokens."""
    nqkv = (cfg["n_q"] + 2 * cfg["n_kv"]) * cfg["hd"]
    return B * (nqkv + 2 * cfg["n_q"] * cfg["hd"] + cfg["d"] + 2 + cfg["n_q"])


def spark_prefill(ctx: SparkContext, layers, h, start: int, chunk: int = 64, more_ctx=(), more_streams=None):
    """Run a prompt through a stack of layers chunk by chunk (the C entry point of the same name; argument marshalling only).
    With further contexts in more_ctx (and optionally as many further torch streams) that many more chunks are in flight at
    a time: spark_prefill_pipelined.

    layers: LayerHandles made with SPARK_SHARED_CACHE in cfg["flags"] and caches [n_kv][cap][.]; h [N][d] fp32 holds the
    prompt's N embeddings and is replaced in place by the stack's outputs; the tokens are appended to each layer's
    cache at rows start .. start + N - 1 (start = tokens already cached).  chunk <= 64 tokens go through the stack
    together; later chunks see the earlier ones through the caches."""
    if not 1 <= chunk <= 64:
        raise ValueError("chunk must be 1..64")
    N = h.shape[0]
    stack = make_stack(layers)
    cfg = {k: getattr(layers[0].cfg, k) for k in ("n_q", "n_kv", "hd", "d")}
    scratch = torch.empty(layer_scratch_floats(cfg, min(chunk, N)), dtype=torch.float32, device=h.device)
    more_ctx = list(more_ctx) if not isinstance(more_ctx, SparkContext) else [more_ctx]
    if more_ctx:
        n = 1 + len(more_ctx)
        ctxs = [ctx] + more_ctx
        scratches = [scratch] + [torch.empty_like(scratch) for _ in more_ctx]
        side = list(more_streams) if more_streams is not None else [torch.cuda.Stream(device=h.device) for _ in more_ctx]
        streams = [_stream()] + [s.cuda_stream for s in side]
        len_buf = torch.empty(n * chunk, dtype=torch.int32, device=h.device)
        arr = lambda vals: (C.c_void_p * n)(*vals)
        _check(lib().spark_prefill_pipelined(arr([c.handle.value for c in ctxs]), arr([_ptr(t) for t in scratches]), arr(streams), n,
                                             stack.weights, stack.cfgs, stack.caches, stack.n_layers, _ptr(h), N, start, chunk,
                                             _ptr(len_buf)), "spark_prefill_pipelined")
        # the temporaries are used on the other streams too: keep the caching allocator from handing them out early
        for s in side:
            for t in scratches + [len_buf]:
                t.record_stream(s)
        return h
    len_buf = torch.empty(chunk, dtype=torch.int32, device=h.device)
    _check(lib().spark_prefill(ctx.handle, stack.weights, stack.cfgs, stack.caches, stack.n_layers, _ptr(h), N, start, chunk,
                               _ptr(len_buf), _ptr(scratch), _stream()), "spark_prefill")
    return h
