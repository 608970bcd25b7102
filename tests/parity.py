"""Comparison rules shared by the GPU parity tests.

Tolerances (written here once, used by every test):
  * theta: |theta_gpu - theta_oracle| <= 1e-5 * max(|theta_oracle|, std_oracle)  (fp32 threshold)
  * active sets: identical except for entries with |x_i - theta| <= 1e-4 * std
  * outputs: max|err| <= 2e-2 * RMS(oracle output) for bf16 weights with fp32 accumulation,
             max|err| <= 1e-5 * RMS(oracle output) for fp32 weights
"""
import numpy as np

THETA_RTOL = 1e-5
BAND = 1e-4
# "split2": exact (bf16-representable) weights met by activations that the tensor-core kernels feed as a two-term
# bf16 split (16 mantissa bits): every product carries a relative error of up to 2^-17 = 7.6e-6, the largest of
# tens of thousands of outputs lands near 1e-5 of the RMS; 4e-5 leaves a factor of four.
OUT_TOL = {"bf16": 2e-2, "f32": 1e-5, "split2": 4e-5}


def rms(a):
    a = np.asarray(a, dtype=np.float64)
    return float(np.sqrt(np.mean(a * a))) if a.size else 0.0


def check_theta(theta_gpu, theta_or, std_or, what=""):
    theta_gpu, theta_or = float(theta_gpu), float(theta_or)
    if not np.isfinite(theta_or):
        assert theta_gpu == theta_or, f"{what}: theta {theta_gpu} vs {theta_or}"
        return
    err = abs(theta_gpu - theta_or) / max(abs(theta_or), std_or)
    assert err <= THETA_RTOL, f"{what}: theta {theta_gpu} vs {theta_or} (rel {err:.2e})"


def check_set(idx_gpu, mask_or, scores, theta_or, std_or, what=""):
    """idx_gpu: iterable of selected positions; mask_or: oracle's boolean mask; scores: fp64 values
    the oracle thresholded.  Returns the symmetric difference (all of it inside the band)."""
    got = np.zeros(mask_or.shape[0], dtype=bool)
    idx_gpu = np.asarray(idx_gpu, dtype=np.int64)
    assert idx_gpu.size == np.unique(idx_gpu).size, f"{what}: duplicate indices"
    assert idx_gpu.size == 0 or (idx_gpu.min() >= 0 and idx_gpu.max() < mask_or.shape[0]), f"{what}: index out of range"
    got[idx_gpu] = True
    diff = np.flatnonzero(got != mask_or)
    if diff.size:
        dist = np.abs(np.asarray(scores, dtype=np.float64)[diff] - theta_or)
        assert np.all(dist <= BAND * std_or), \
            f"{what}: {diff.size} set differences outside the band (worst {dist.max() / std_or:.2e} std)"
    return diff


def check_output(y_gpu, y_or, kind, what=""):
    y_gpu = np.asarray(y_gpu, dtype=np.float64)
    y_or = np.asarray(y_or, dtype=np.float64)
    assert y_gpu.shape == y_or.shape, f"{what}: shape {y_gpu.shape} vs {y_or.shape}"
    assert np.all(np.isfinite(y_gpu)), f"{what}: non-finite output"
    scale = rms(y_or)
    err = float(np.max(np.abs(y_gpu - y_or))) if y_or.size else 0.0
    tol = OUT_TOL[kind] * scale if scale > 0 else 1e-30
    assert err <= tol, f"{what}: max|err| {err:.3e} > {OUT_TOL[kind]:g} * RMS {scale:.3e}"
    return err / scale if scale > 0 else 0.0


def layer_refs_within_band(O, h_in, W, kc, vc, n, window, **shape_kw):
    """The oracle's decoder layer, then -- lazily -- its variants in which attended tokens whose predictor score lies within
    BAND * std of their head's threshold are toggled (at most four such tokens: sixteen variants).  The -inf threshold of the
    attention is discontinuous, so either side of the band is a correct result; a GPU output must match one of them."""
    ref = O.decoder_layer(h_in, W, kc, vc, n, window=window, **shape_kw)
    yield ref
    n_q, n_kv, r = shape_kw["n_q"], shape_kw["n_kv"], shape_kw["r_attn"]
    lo = 0 if window <= 0 else max(0, n - window)
    near = []
    for h in range(n_q):
        th = ref["attn"]["theta"][h]
        if not np.isfinite(th):
            continue
        s = kc[h // (n_q // n_kv), lo:n, :r] @ ref["q"][h, :r]
        std = float(np.std(s, ddof=1))
        near += [(h, lo + int(t)) for t in np.flatnonzero(np.abs(s - th) <= BAND * std)]
    near = near[:4]
    for combo in range(1, 1 << len(near)):
        mask = ref["attn"]["mask"].copy()
        for i, (h, t) in enumerate(near):
            if combo >> i & 1:
                mask[h, t] = not mask[h, t]
        yield O.decoder_layer(h_in, W, kc, vc, n, window=window, attn_mask_override=mask, **shape_kw)
