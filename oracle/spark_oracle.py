"""CPU oracle for the Spark Transformer decode step -- TEST INFRASTRUCTURE ONLY.

A plain, slow, fp64 restatement of what the paper defines: statistical top-k
(Section 3, Eq. 9-11), Spark FFN (Section 2.1, Eq. 2), Spark attention
(Section 2.2, Eq. 7) and the minimal pre-norm decoder layer around them
(Section 4, "Implementation details").  It exists so that the CUDA library can
be checked against something written independently from the paper.  Only the
tests, the smoke check and the benchmark's cpu_baseline / reference arm may
import it; it shares no code with the CUDA path and imports nothing from the
library package.  The sparse steps are computed DENSELY here (every neuron,
every token, with explicit zeros / -inf), never through an index list.

Inputs are the storage-rounded values (bf16 weights / caches are rounded once
by the input generator and widened); all arithmetic below is fp64.

Parity pins (tests/test_oracle_*.py): the quantile against printed constants
and scipy.special.ndtri; mean/std against numpy; two hand-worked examples under
tests/golden/; threshold-set == sort-based top-count set; Theorem 1's count
bound and the Gaussian / Laplace closed-form selected fractions; the
zero-inactive-rows and k >= n invariants; attention special cases against
torch.nn.functional.scaled_dot_product_attention; GELU / softplus / RMSNorm
against torch library routines; RoPE against its rotation identities.
Parity unpinned: the CHOICE of layer structure in `decoder_layer` (the paper
says only "Gemma-2 recipe"); each of its steps is pinned separately.
"""
from __future__ import annotations

import math

import numpy as np

F64 = np.float64


# ----------------------------------------------------------------------------
# Section 3: statistical top-k
# ----------------------------------------------------------------------------
def gaussian_upper_quantile(p: float) -> float:
    """z such that a standard normal exceeds z with probability p, i.e. Q(1 - p).

    Q is the standard Gaussian quantile of Eq. 11.  Solved as
    0.5 * erfc(z / sqrt(2)) = p by bisection (the upper-tail form keeps small p
    free of cancellation).
    """
    if not (0.0 < p < 1.0):
        raise ValueError("p must lie strictly between 0 and 1")
    if p == 0.5:
        return 0.0                 # symmetry; erfc is flat to rounding around 0
    lo, hi = -40.0, 40.0           # tail(lo) ~ 1 > p > tail(hi) ~ 0
    for _ in range(200):           # far more halvings than fp64 can resolve
        mid = 0.5 * (lo + hi)
        if 0.5 * math.erfc(mid / math.sqrt(2.0)) > p:
            lo = mid
        else:
            hi = mid
    return 0.5 * (lo + hi)


def mean_std(x: np.ndarray) -> tuple[float, float]:
    """Sample mean and Bessel-corrected standard deviation (text below Eq. 11)."""
    x = np.asarray(x, dtype=F64)
    n = x.size
    mean = float(np.sum(x) / n)
    std = float(np.sqrt(np.sum((x - mean) ** 2) / (n - 1)))
    return mean, std


def threshold(x: np.ndarray, k: int) -> float:
    """theta(x, k) = mean(x) + std(x) * Q(1 - k/d)   (Eq. 11)."""
    x = np.asarray(x, dtype=F64)
    n = x.size
    mean, std = mean_std(x)
    return mean + std * gaussian_upper_quantile(k / n)


def stat_topk(x: np.ndarray, k: int, fill: str = "zero"):
    """Statistical top-k of one vector (Eq. 9-10) and its -inf variant (Section 3).

    Returns (theta, mask, out): mask[i] = x[i] > theta (strict: soft-thresholding
    gives 0 at equality), out[i] = x[i] - theta on the mask and 0 ('zero') or
    -inf ('neginf') elsewhere.

    Readings where the paper is silent: k >= d keeps every entry unshifted
    (theta = -inf), because "keep the largest k values" with k >= d removes
    nothing and the literal formula would shift by -inf; k <= 0 keeps nothing.
    """
    x = np.asarray(x, dtype=F64).reshape(-1)
    n = x.size
    off = 0.0 if fill == "zero" else -np.inf
    if fill not in ("zero", "neginf"):
        raise ValueError(fill)
    if k >= n:
        return -np.inf, np.ones(n, dtype=bool), x.copy()
    if k <= 0:
        return np.inf, np.zeros(n, dtype=bool), np.full(n, off)
    theta = threshold(x, k)
    mask = x > theta
    out = np.where(mask, x - theta, off)
    return theta, mask, out


# ----------------------------------------------------------------------------
# statistical top-k of a vector sharded over m devices (appendix on distributed
# training: "global" and "local" statistical top-k)
# ----------------------------------------------------------------------------
def shard_moments(x: np.ndarray) -> tuple[float, float, float]:
    """What one device computes of its part: (count, mean, sum of squared deviations from its mean).

    Reading: the paper has the devices exchange "mean and variance"; the count is carried along so
    that parts of unequal length combine correctly, and the sum of squared deviations stands for
    the variance (variance x count) so that no convention about its divisor is needed."""
    x = np.asarray(x, dtype=F64).reshape(-1)
    mean = float(np.sum(x) / x.size)
    return float(x.size), mean, float(np.sum((x - mean) ** 2))


def combine_moments(parts) -> tuple[float, float, float]:
    """Moments of the whole vector from the parts' moments: the weighted mean, and the law of total
    variance (within-part deviations plus the parts' squared distances to the global mean)."""
    n = sum(p[0] for p in parts)
    mean = sum(p[0] * p[1] for p in parts) / n
    m2 = sum(p[2] + p[0] * (p[1] - mean) ** 2 for p in parts)
    return n, mean, m2


def stat_topk_sharded_global(shards, k: int, fill: str = "zero"):
    """Global statistical top-k: every device combines all parts' moments into mean and Bessel-corrected
    std of the whole vector, forms theta (Eq. 11 with d = total length) and thresholds its own part.
    Returns (theta, [mask per shard], [out per shard])."""
    shards = [np.asarray(s, dtype=F64).reshape(-1) for s in shards]
    n, mean, m2 = combine_moments([shard_moments(s) for s in shards])
    off = 0.0 if fill == "zero" else -np.inf
    if k >= n:
        return -np.inf, [np.ones(s.size, dtype=bool) for s in shards], [s.copy() for s in shards]
    theta = mean + math.sqrt(m2 / (n - 1)) * gaussian_upper_quantile(k / n)
    masks = [s > theta for s in shards]
    return theta, masks, [np.where(m, s - theta, off) for s, m in zip(shards, masks)]


def stat_topk_sharded_local(shards, k: int, fill: str = "zero"):
    """Local statistical top-k: each device applies the operator to its own part with k' = k / m
    (reading: integer division, at least 1).  Returns a list of (theta, mask, out) per shard."""
    kk = max(1, k // len(shards))
    return [stat_topk(s, kk, fill) for s in shards]


# ----------------------------------------------------------------------------
# activations
# ----------------------------------------------------------------------------
_erf = np.vectorize(math.erf, otypes=[F64])


def gelu(a: np.ndarray, form: str = "tanh") -> np.ndarray:
    """GELU of Hendrycks & Gimpel: 'erf' is a * Phi(a); 'tanh' is their tanh form
    0.5 a (1 + tanh(sqrt(2/pi) (a + 0.044715 a^3))), the one Gemma uses."""
    a = np.asarray(a, dtype=F64)
    if form == "erf":
        return 0.5 * a * (1.0 + _erf(a / math.sqrt(2.0)))
    if form == "tanh":
        return 0.5 * a * (1.0 + np.tanh(math.sqrt(2.0 / math.pi) * (a + 0.044715 * a ** 3)))
    raise ValueError(form)


def softplus(a: np.ndarray) -> np.ndarray:
    """log(1 + exp(a)), written so that it neither overflows nor loses small values."""
    a = np.asarray(a, dtype=F64)
    return np.maximum(a, 0.0) + np.log1p(np.exp(-np.abs(a)))


# ----------------------------------------------------------------------------
# Section 2.1: Spark FFN
# ----------------------------------------------------------------------------
def spark_ffn(q, K1, K2, V, k: int, r: int, gelu_form: str = "tanh"):
    """Spark-FFN(q; K1, K2, V, k, r) = V . ( GELU(Top_k(K1^T q[:r])) * (K2^T q[r:]) )   (Eq. 2).

    K1 is r x d_ff, K2 is (d - r) x d_ff, V is d x d_ff (the paper's
    orientation).  Top_k is statistical top-k with zero fill, so GELU sees the
    shifted survivors s_i - theta and GELU(0) = 0 elsewhere.
    Returns dict(y, theta, mask, s, u).
    """
    q = np.asarray(q, dtype=F64).reshape(-1)
    K1 = np.asarray(K1, dtype=F64)
    K2 = np.asarray(K2, dtype=F64)
    V = np.asarray(V, dtype=F64)
    d = q.size
    assert K1.shape[0] == r and K2.shape[0] == d - r and V.shape[0] == d
    s = K1.T @ q[:r]                              # predictor, every neuron
    theta, mask, a = stat_topk(s, k, "zero")
    g = gelu(a, gelu_form)                        # zero off the mask
    t = K2.T @ q[r:]                              # every neuron (dense on purpose)
    u = g * t
    y = V @ u
    return {"y": y, "theta": theta, "mask": mask, "s": s, "u": u}


# ----------------------------------------------------------------------------
# Section 2.2: Spark attention
# ----------------------------------------------------------------------------
def spark_attention_head(q, K, V, k_attn: int, r: int, mask_override=None):
    """One head of Eq. 7: V . ( softmax(Top_k^{(-inf)}(K1^T q[:r])) * softplus(K2^T q[r:]) ).

    K, V are d_attn x n_ctx (one column per token, the paper's orientation);
    K1 = first r rows of K, K2 = the rest.  No logit scale is applied here: q is
    used as given.  No renormalisation after the softplus gate (the equation
    has none).  An empty selection gives a zero output ("attends to nothing").
    mask_override, if given, replaces the selected set (used by the parity
    harness when an entry sits within rounding distance of theta).
    Returns dict(o, theta, mask, s).
    """
    q = np.asarray(q, dtype=F64).reshape(-1)
    K = np.asarray(K, dtype=F64)
    V = np.asarray(V, dtype=F64)
    n = K.shape[1]
    s = K[:r, :].T @ q[:r]
    theta, mask, a = stat_topk(s, k_attn, "neginf")
    if mask_override is not None:
        mask = np.asarray(mask_override, dtype=bool)
        a = np.where(mask, s - (theta if np.isfinite(theta) else 0.0), -np.inf)
    if not mask.any():
        return {"o": np.zeros(V.shape[0]), "theta": theta, "mask": mask, "s": s}
    e = np.exp(a - np.max(a))                     # exp(-inf) = 0 off the mask
    w = e / np.sum(e)
    gate = softplus(K[r:, :].T @ q[r:])           # every token (dense on purpose)
    o = V @ (w * gate)
    return {"o": o, "theta": theta, "mask": mask, "s": s}


def spark_attention(q, kcache, vcache, ctx_len: int, k_attn: int, r: int, window: int = 0,
                    mask_override=None):
    """Spark attention for one sequence with grouped KV heads.

    q[n_q][hd]; kcache[n_kv][cap][hd], vcache[n_kv][cap][hd] token-major; the
    first ctx_len rows are valid and the newest token is row ctx_len - 1 (it
    attends to itself).  Query head h reads KV head h // (n_q // n_kv); every
    query head runs its own top-k.  window > 0 keeps only the newest `window`
    tokens (the local-attention layers of Section 4); 0 means all.
    Returns dict(o[n_q][hd], theta[n_q], mask[n_q][ctx_len]) with mask False
    outside the window.
    """
    q = np.asarray(q, dtype=F64)
    n_q, hd = q.shape
    n_kv = kcache.shape[0]
    group = n_q // n_kv
    lo = 0 if window <= 0 else max(0, ctx_len - window)
    o = np.zeros((n_q, hd))
    theta = np.zeros(n_q)
    mask = np.zeros((n_q, ctx_len), dtype=bool)
    for h in range(n_q):
        g = h // group
        K = np.asarray(kcache[g, lo:ctx_len, :], dtype=F64).T
        V = np.asarray(vcache[g, lo:ctx_len, :], dtype=F64).T
        mo = None if mask_override is None else np.asarray(mask_override[h])[lo:ctx_len]
        res = spark_attention_head(q[h], K, V, k_attn, r, mo)
        o[h] = res["o"]
        theta[h] = res["theta"]
        mask[h, lo:ctx_len] = res["mask"]
    return {"o": o, "theta": theta, "mask": mask}


def standard_attention_head(q, K, V):
    """Standard-Attention(q; K, V) = V . softmax(K^T q)   (Eq. 6), no scale."""
    q = np.asarray(q, dtype=F64).reshape(-1)
    z = np.asarray(K, dtype=F64).T @ q
    e = np.exp(z - np.max(z))
    return np.asarray(V, dtype=F64) @ (e / np.sum(e))


# ----------------------------------------------------------------------------
# FLOP counts the paper prints (Eq. 3, 4, 8 and the FLOPs-per-token table)
# ----------------------------------------------------------------------------
def ffn_flops_dense(d: int, d_ff: int) -> int:
    return 4 * d * d_ff                                         # Eq. 3


def ffn_flops_spark(d: int, d_ff: int, r: int, k: int) -> int:
    return 2 * r * d_ff + 2 * (d - r) * k + 2 * d * k           # Eq. 4


def attn_flops_dense(d_attn: int, n_ctx: int) -> int:
    return 4 * d_attn * n_ctx                                   # text below Eq. 6


def attn_flops_spark(d_attn: int, n_ctx: int, k_attn: int, r: int) -> int:
    ka = min(k_attn, n_ctx)
    return 2 * r * n_ctx + 2 * (d_attn - r) * ka + 2 * d_attn * ka   # Eq. 8 at general r


# ----------------------------------------------------------------------------
# Section 4: the layer around the two operators
# ----------------------------------------------------------------------------
def rmsnorm(h, w, eps: float = 1e-6):
    """h / sqrt(mean(h^2) + eps) * w."""
    h = np.asarray(h, dtype=F64)
    return h / np.sqrt(np.mean(h * h) + eps) * np.asarray(w, dtype=F64)


def rope_part(v, pos: int, base: float = 10000.0):
    """Rotary position embedding of one m-dim vector on its own m/2 pairs (i, i + m/2),
    pair i rotated by the angle pos * base^(-2i/m)."""
    v = np.asarray(v, dtype=F64)
    m = v.shape[-1]
    half = m // 2
    ang = pos * base ** (-2.0 * np.arange(half) / m)
    c, s = np.cos(ang), np.sin(ang)
    a, b = v[..., :half], v[..., half:]
    return np.concatenate([a * c - b * s, a * s + b * c], axis=-1)


def rope_split(v, pos: int, r: int, base: float = 10000.0):
    """Position-encode v[:r] and v[r:] separately (Section 4: the encoding is applied to
    q[:r], q[r:], and to the columns of K1 and of K2)."""
    v = np.asarray(v, dtype=F64)
    return np.concatenate([rope_part(v[..., :r], pos, base), rope_part(v[..., r:], pos, base)], axis=-1)


def round_to_bf16(a):
    """Nearest-even rounding of fp64 values to bf16-representable values (cache storage)."""
    a32 = np.asarray(a, dtype=np.float32)
    u = a32.view(np.uint32)
    u = (u + np.uint32(0x7FFF) + ((u >> np.uint32(16)) & np.uint32(1))) & np.uint32(0xFFFF0000)
    return u.view(np.float32).astype(F64)


def decoder_layer(h, W, kcache, vcache, ctx_len: int, *, n_q: int, n_kv: int, hd: int,
                  r_attn: int, k_attn: int, r_ff: int, k_ff: int, window: int = 0,
                  gelu_form: str = "tanh", eps: float = 1e-6, cache_bf16: bool = True,
                  rope_base: float = 10000.0, attn_mask_override=None, k_round=None):
    """One pre-norm decoder layer for one new token of one sequence.

        a  = RMSNorm(h; norm1);  [q|k|v] = Wqkv a
        q, k position-encoded on each half at position ctx_len - 1;  q *= 1/sqrt(hd)
        k, v stored as cache row ctx_len - 1 (rounded to bf16 when cache_bf16)
        h += Wo . SparkAttention(q; cache)
        h += SparkFFN(RMSNorm(h; norm2))

    W: dict(norm1[d], norm2[d], Wqkv[(n_q+2 n_kv) hd][d], Wo[d][n_q hd],
            K1t[d_ff][r_ff], K2t[d_ff][d-r_ff], Vt[d_ff][d])  (storage-rounded values).
    kcache / vcache: [n_kv][cap][hd] fp64 arrays, modified in place.
    ctx_len counts the new token.  k_round, if given, is the storage rounding of the appended key rows
    ([n_kv][hd] -> the values a quantised cache holds; the rule itself belongs to whoever defines the
    storage format) and replaces the bf16 rounding of k.  attn_mask_override, if given, is handed to spark_attention (the
    parity harness's way of following the other side's choice for a token within rounding distance of
    the attention threshold).  Returns dict(h, attn, ffn, q).
    """
    h = np.asarray(h, dtype=F64).copy()
    pos = ctx_len - 1
    a = rmsnorm(h, W["norm1"], eps)
    qkv = np.asarray(W["Wqkv"], dtype=F64) @ a
    q = qkv[: n_q * hd].reshape(n_q, hd)
    kn = qkv[n_q * hd:(n_q + n_kv) * hd].reshape(n_kv, hd)
    vn = qkv[(n_q + n_kv) * hd:].reshape(n_kv, hd)
    q = rope_split(q, pos, r_attn, rope_base) / math.sqrt(hd)
    kn = rope_split(kn, pos, r_attn, rope_base)
    if cache_bf16:
        kn, vn = round_to_bf16(kn), round_to_bf16(vn)
    if k_round is not None:
        kn = np.asarray(k_round(rope_split(qkv[n_q * hd:(n_q + n_kv) * hd].reshape(n_kv, hd), pos, r_attn, rope_base)), dtype=F64)
    kcache[:, pos, :] = kn
    vcache[:, pos, :] = vn
    att = spark_attention(q, kcache, vcache, ctx_len, k_attn, r_attn, window, attn_mask_override)
    h = h + np.asarray(W["Wo"], dtype=F64) @ att["o"].reshape(-1)
    b = rmsnorm(h, W["norm2"], eps)
    ffn = spark_ffn(b, np.asarray(W["K1t"], dtype=F64).T, np.asarray(W["K2t"], dtype=F64).T,
                    np.asarray(W["Vt"], dtype=F64).T, k_ff, r_ff, gelu_form)
    h = h + ffn["y"]
    return {"h": h, "attn": att, "ffn": ffn, "q": q, "x_ffn": b}
