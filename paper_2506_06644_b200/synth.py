"""Seeded synthetic inputs for the Spark decode path.

This module only draws numbers and rounds them to their storage type.  It holds
none of the method's arithmetic (no threshold, no activation, no product), so
the CUDA library's tests and the CPU oracle's tests can both be fed from it
without sharing any computation.  Everything is generated on the host with
numpy; callers upload what they need.

Storage rounding: bf16 tensors are produced by rounding fp32 draws to bf16 with
round-to-nearest-even once, here.  A bf16 tensor is returned as a pair
(bits uint16, widened fp32 values); both sides of a parity test read the same
bits.

Shapes follow the Gemma-2-shaped workloads of the paper's Section 4
("Implementation details"): model width d, FFN width d_ff, predictor width r,
sparsity k ~ 8 % of d_ff; attention with head_dim 256, predictor slice 128 and
k_attn = 256 tokens per query head.
"""
from __future__ import annotations

from dataclasses import dataclass

import numpy as np


# ----------------------------------------------------------------------------
# storage rounding
# ----------------------------------------------------------------------------
def f32_to_bf16_bits(a: np.ndarray) -> np.ndarray:
    """Round fp32 to bf16 (nearest, ties to even); returns the uint16 patterns."""
    a = np.ascontiguousarray(a, dtype=np.float32)
    u = a.view(np.uint32)
    lsb = (u >> np.uint32(16)) & np.uint32(1)
    rounded = u + np.uint32(0x7FFF) + lsb
    return (rounded >> np.uint32(16)).astype(np.uint16)


def bf16_bits_to_f32(bits: np.ndarray) -> np.ndarray:
    """Widen bf16 bit patterns to fp32 (exact)."""
    bits = np.ascontiguousarray(bits, dtype=np.uint16)
    return (bits.astype(np.uint32) << np.uint32(16)).view(np.float32)


def f32_to_e4m3_bits(a: np.ndarray) -> np.ndarray:
    """Round fp32 to FP8 E4M3 (1-4-3 bits, bias 7, largest finite 448, no infinities; nearest, ties to even,
    magnitudes beyond 448 saturate); returns the uint8 patterns.  NaN -> 0x7f."""
    a = np.ascontiguousarray(a, dtype=np.float32).astype(np.float64)
    sign = np.signbit(a).astype(np.uint8) << np.uint8(7)
    mag = np.minimum(np.abs(a), 448.0)
    # subnormal codes (and zero): multiples of 2^-9 below 2^-6
    sub = np.rint(mag * 512.0)
    m, e = np.frexp(np.where(mag > 0, mag, 1.0))                  # mag = m * 2^e, m in [0.5, 1)
    expo = e - 1
    mant = np.rint((2.0 * m - 1.0) * 8.0)
    carry = mant >= 8
    mant = np.where(carry, 0, mant)
    expo = np.where(carry, expo + 1, expo)
    code = np.where(mag < 2.0 ** -6, sub, (expo + 7) * 8 + mant)
    code = np.minimum(code, 0x7E).astype(np.uint8)
    out = sign | code
    return np.where(np.isnan(a), np.uint8(0x7F), out).astype(np.uint8)


def e4m3_bits_to_f32(bits: np.ndarray) -> np.ndarray:
    """Widen FP8 E4M3 bit patterns to fp32 (exact); 0x7f / 0xff are NaN."""
    bits = np.ascontiguousarray(bits, dtype=np.uint8)
    codes = np.arange(256)
    e, m = (codes >> 3) & 15, codes & 7
    val = np.where(e == 0, m * 2.0 ** -9, (1.0 + m / 8.0) * 2.0 ** (e - 7.0))
    val = np.where(codes & 0x80, -val, val)
    val[[0x7F, 0xFF]] = np.nan
    return val.astype(np.float32)[bits]


def quantize_rows_e4m3(W: np.ndarray):
    """Per-row scaled FP8 storage of a weight matrix: W[i, :] ~ scale[i] * e4m3(bits[i, :]) with
    scale[i] = max|W[i, :]| / 448 (1 for an all-zero row).  Returns (bits uint8, scale float32)."""
    W = np.ascontiguousarray(W, dtype=np.float32)
    amax = np.abs(W).max(axis=1)
    scale = np.where(amax > 0, amax / np.float32(448.0), np.float32(1.0)).astype(np.float32)
    bits = f32_to_e4m3_bits(W / scale[:, None])
    return bits, scale


def _rng(seed: int, stream: int) -> np.random.Generator:
    # One independent stream per tensor, so that adding a tensor to a workload
    # does not change the others.
    return np.random.Generator(np.random.PCG64(np.random.SeedSequence([seed, stream])))


def normal_f32(shape, seed: int, stream: int, scale: float = 1.0) -> np.ndarray:
    g = _rng(seed, stream)
    out = g.standard_normal(size=shape, dtype=np.float32)
    if scale != 1.0:
        out *= np.float32(scale)
    return out


def laplace_f32(shape, seed: int, stream: int) -> np.ndarray:
    """Laplace(0, 1): density exp(-|x|)/2."""
    g = _rng(seed, stream)
    return g.laplace(0.0, 1.0, size=shape).astype(np.float32)


def student_t_f32(shape, seed: int, stream: int, dof: float = 4.0) -> np.ndarray:
    g = _rng(seed, stream)
    return g.standard_t(dof, size=shape).astype(np.float32)


def rows_f32(dist: str, rows: int, n: int, seed: int, stream: int = 0) -> np.ndarray:
    """Rows for the standalone statistical top-k workload: 'normal', 'laplace' or 'student_t4'."""
    if dist == "normal":
        return normal_f32((rows, n), seed, stream)
    if dist == "laplace":
        return laplace_f32((rows, n), seed, stream)
    if dist == "student_t4":
        return student_t_f32((rows, n), seed, stream, 4.0)
    raise ValueError(f"unknown distribution {dist!r}")


# ----------------------------------------------------------------------------
# Spark FFN workload
# ----------------------------------------------------------------------------
@dataclass
class FfnInputs:
    """One Spark-FFN problem in the library's HBM layout (neuron-major).

    K1t[d_ff][r], K2t[d_ff][d-r], Vt[d_ff][d] are the transposes of the paper's
    K1 (r x d_ff), K2 ((d-r) x d_ff) and V (d x d_ff): one neuron's weights are
    one contiguous row.  For wdtype == 'bf16' the *_bits arrays hold the storage
    bits and the fp32 arrays hold exactly those values widened.
    """
    d: int
    d_ff: int
    r: int
    k: int
    wdtype: str
    x: np.ndarray            # [B][d] fp32
    K1t: np.ndarray          # fp32 values (storage-rounded)
    K2t: np.ndarray
    Vt: np.ndarray
    K1t_bits: np.ndarray | None = None
    K2t_bits: np.ndarray | None = None
    Vt_bits: np.ndarray | None = None


def ffn_inputs(d: int, d_ff: int, r: int, k: int, batch: int, wdtype: str = "bf16",
               seed: int = 0, unit_rms_x: bool = True) -> FfnInputs:
    """Weights ~ N(0, 1/d); x ~ N(0, 1), each token optionally rescaled to RMS 1."""
    if wdtype not in ("f32", "bf16"):
        raise ValueError(wdtype)
    s = 1.0 / np.sqrt(d)
    K1t = normal_f32((d_ff, r), seed, 1, s)
    K2t = normal_f32((d_ff, d - r), seed, 2, s)
    Vt = normal_f32((d_ff, d), seed, 3, s)
    x = normal_f32((batch, d), seed, 4)
    if unit_rms_x:
        rms = np.sqrt(np.mean(x.astype(np.float64) ** 2, axis=1, keepdims=True))
        x = (x / rms).astype(np.float32)
    out = FfnInputs(d, d_ff, r, k, wdtype, x, K1t, K2t, Vt)
    if wdtype == "bf16":
        out.K1t_bits = f32_to_bf16_bits(K1t)
        out.K2t_bits = f32_to_bf16_bits(K2t)
        out.Vt_bits = f32_to_bf16_bits(Vt)
        out.K1t = bf16_bits_to_f32(out.K1t_bits)
        out.K2t = bf16_bits_to_f32(out.K2t_bits)
        out.Vt = bf16_bits_to_f32(out.Vt_bits)
    return out


# ----------------------------------------------------------------------------
# Spark attention workload
# ----------------------------------------------------------------------------
@dataclass
class AttnInputs:
    """One Spark-attention decode problem in the library's cache layout.

    k1c[B][n_kv][cap][r], k2c[B][n_kv][cap][hd-r], vc[B][n_kv][cap][hd]; the
    first ctx_len[b] token rows of sequence b are valid.  q[B][n_q][hd] fp32 is
    used as given (already position-encoded and scaled).
    """
    n_q: int
    n_kv: int
    hd: int
    r: int
    cap: int
    kvdtype: str
    q: np.ndarray
    ctx_len: np.ndarray      # int32 [B]
    k1c: np.ndarray          # fp32 values (storage-rounded)
    k2c: np.ndarray
    vc: np.ndarray
    k1c_bits: np.ndarray | None = None
    k2c_bits: np.ndarray | None = None
    vc_bits: np.ndarray | None = None


def attn_inputs(batch: int, n_q: int, n_kv: int, hd: int, r: int, cap: int, ctx_len,
                kvdtype: str = "bf16", seed: int = 0, q_scale: float | None = None) -> AttnInputs:
    """KV cache ~ N(0, 1); q ~ N(0, 1) * q_scale (default 1/sqrt(hd))."""
    if kvdtype not in ("f32", "bf16"):
        raise ValueError(kvdtype)
    if q_scale is None:
        q_scale = 1.0 / np.sqrt(hd)
    ctx = np.asarray(ctx_len, dtype=np.int32).reshape(-1)
    if ctx.size == 1 and batch > 1:
        ctx = np.repeat(ctx, batch)
    assert ctx.size == batch and int(ctx.max(initial=0)) <= cap
    k1c = normal_f32((batch, n_kv, cap, r), seed, 11)
    k2c = normal_f32((batch, n_kv, cap, hd - r), seed, 12)
    vc = normal_f32((batch, n_kv, cap, hd), seed, 13)
    q = normal_f32((batch, n_q, hd), seed, 14, q_scale)
    out = AttnInputs(n_q, n_kv, hd, r, cap, kvdtype, q, ctx, k1c, k2c, vc)
    if kvdtype == "bf16":
        out.k1c_bits = f32_to_bf16_bits(k1c)
        out.k2c_bits = f32_to_bf16_bits(k2c)
        out.vc_bits = f32_to_bf16_bits(vc)
        out.k1c = bf16_bits_to_f32(out.k1c_bits)
        out.k2c = bf16_bits_to_f32(out.k2c_bits)
        out.vc = bf16_bits_to_f32(out.vc_bits)
    return out


# ----------------------------------------------------------------------------
# decoder-layer workload
# ----------------------------------------------------------------------------
@dataclass
class LayerShape:
    d: int
    d_ff: int
    r_ff: int
    k_ff: int
    n_q: int
    n_kv: int
    hd: int
    r_attn: int
    k_attn: int
    n_layers: int
    vocab: int


GEMMA2_2B = LayerShape(d=2304, d_ff=9216, r_ff=1024, k_ff=737, n_q=8, n_kv=4, hd=256,
                       r_attn=128, k_attn=256, n_layers=26, vocab=256000)
# The paper gives no predictor width for a 9B-shaped model; d/2 = 1792 is a
# multiple of 256 as its Section 4 requires of r.
GEMMA2_9B = LayerShape(d=3584, d_ff=14336, r_ff=1792, k_ff=1147, n_q=16, n_kv=8, hd=256,
                       r_attn=128, k_attn=256, n_layers=42, vocab=256000)
TINY = LayerShape(d=256, d_ff=1024, r_ff=128, k_ff=82, n_q=4, n_kv=2, hd=64,
                  r_attn=32, k_attn=16, n_layers=2, vocab=512)


@dataclass
class LayerWeights:
    """bf16 weights of one decoder layer, output-major ([n_out][n_in])."""
    shape: LayerShape
    norm1: np.ndarray        # [d] fp32
    norm2: np.ndarray        # [d] fp32
    Wqkv_bits: np.ndarray    # [(n_q + 2 n_kv) hd][d]
    Wo_bits: np.ndarray      # [d][n_q hd]
    K1t_bits: np.ndarray     # [d_ff][r_ff]
    K2t_bits: np.ndarray     # [d_ff][d - r_ff]
    Vt_bits: np.ndarray      # [d_ff][d]


def layer_weights(shape: LayerShape, seed: int, layer: int) -> LayerWeights:
    """Random-init weights ~ N(0, 1/fan_in), rounded to bf16; norm weights ~ 1 + 0.1 N(0,1)."""
    base = 100 + 16 * layer
    d, hd = shape.d, shape.hd
    nqkv = (shape.n_q + 2 * shape.n_kv) * hd

    def w(rows, cols, stream, fan_in):
        return f32_to_bf16_bits(normal_f32((rows, cols), seed, base + stream, 1.0 / np.sqrt(fan_in)))

    return LayerWeights(
        shape=shape,
        norm1=(1.0 + 0.1 * normal_f32((d,), seed, base + 0)).astype(np.float32),
        norm2=(1.0 + 0.1 * normal_f32((d,), seed, base + 1)).astype(np.float32),
        Wqkv_bits=w(nqkv, d, 2, d),
        Wo_bits=w(d, shape.n_q * hd, 3, shape.n_q * hd),
        K1t_bits=w(shape.d_ff, shape.r_ff, 4, d),
        K2t_bits=w(shape.d_ff, d - shape.r_ff, 5, d),
        Vt_bits=w(shape.d_ff, d, 6, d),
    )
