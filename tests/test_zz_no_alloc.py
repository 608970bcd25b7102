"""GPU test of spark_ffn_decode_noalloc, the FFN entry point for callers that cannot allocate
device memory (its inter-block state is a fixed array inside the library instead of a workspace
the caller would have to cudaMalloc).  It must give what the oracle gives and what spark_ffn_decode
gives, must not move device memory, and its first call in a process may go to any stream.  The file
name sorts last on purpose: a run that stops at the first failure has then already run everything else.
"""
import os
import subprocess
import sys

import numpy as np
import pytest
import torch

from oracle import spark_oracle as O
from paper_2506_06644_b200 import binding as S
from paper_2506_06644_b200 import synth
from tests import parity

pytestmark = pytest.mark.gpu
ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _weights(p, wd):
    if wd == "f32":
        return tuple(torch.from_numpy(a).cuda() for a in (p.K1t, p.K2t, p.Vt))
    f = lambda bits: torch.from_numpy(bits.view(np.int16)).cuda().view(torch.bfloat16)
    return f(p.K1t_bits), f(p.K2t_bits), f(p.Vt_bits)


def _oracle(p, b, k, r):
    return O.spark_ffn(p.x[b], p.K1t.astype(np.float64).T, p.K2t.astype(np.float64).T, p.Vt.astype(np.float64).T, k, r)


# B = 1: one-token kernel; 3: few-token kernel; 5 with d_ff % 128 != 0 and 16: union-gather tensor-core kernel (the context call
# of the second takes the tcgen05 chunk kernels instead); 2 with fp32 weights: the generic kernel
@pytest.mark.parametrize("B,d,d_ff,r,k,wd", [(1, 512, 3000, 256, 240, "bf16"), (5, 512, 3000, 256, 240, "bf16"),
                                              (3, 512, 3000, 256, 240, "bf16"), (16, 512, 3072, 256, 246, "bf16"),
                                              (2, 256, 1024, 128, 82, "f32")])
def test_noalloc_matches_the_oracle_and_the_workspace_entry_point_twice_in_a_row(B, d, d_ff, r, k, wd):
    p = synth.ffn_inputs(d, d_ff, r, k, B, wd, seed=21 + B)
    K1t, K2t, Vt = _weights(p, wd)
    code = S.SPARK_F32 if wd == "f32" else S.SPARK_BF16
    x = torch.from_numpy(p.x).cuda()
    ctx = S.SparkContext(0, max_batch=16, max_dff=d_ff, max_d=d)
    y_ref = torch.empty((B, d), device="cuda")
    th_ref = torch.empty(B, device="cuda")
    S.spark_ffn_decode(ctx, x, B, K1t, K2t, Vt, code, d, d_ff, r, k, 0, y_ref, th_ref, None, None)
    torch.cuda.synchronize()
    assert ctx.device_status() == S.SPARK_OK
    refs = [_oracle(p, b, k, r) for b in range(B)]
    scale = float(y_ref.pow(2).mean().sqrt())
    assert scale > 0
    # the two entry points may take different kernels (tcgen05 chunk kernels with a workspace, union-gather without): both feed
    # the tensor cores a two-term split of the activations, so they agree to that split's error
    same_kernels = not (wd == "bf16" and B >= 5 and d_ff % 128 == 0)
    for call in range(2):                      # the second call runs on the state the first one left
        y = torch.full((B, d), float("nan"), device="cuda")
        th = torch.full((B,), float("nan"), device="cuda")
        free0 = torch.cuda.mem_get_info()[0]
        S.spark_ffn_decode_noalloc(x, B, K1t, K2t, Vt, code, d, d_ff, r, k, 0, y, th)
        torch.cuda.synchronize()
        assert torch.cuda.mem_get_info()[0] == free0, "device memory moved across the call"
        assert S.spark_noalloc_status() == S.SPARK_OK
        yh, thh = y.cpu().numpy(), th.cpu().numpy()
        for b in range(B):                     # against the oracle, at the library's tolerances
            std = float(np.std(refs[b]["s"], ddof=1))
            parity.check_theta(thh[b], refs[b]["theta"], std, f"call {call} token {b}")
            parity.check_output(yh[b], refs[b]["y"], "f32" if wd == "f32" else "bf16", f"call {call} token {b}")
        tol_th, tol_y = (1e-6, 1e-5) if same_kernels else (1e-5, 1e-4)
        assert float((th - th_ref).abs().max()) <= tol_th * max(1.0, float(th_ref.abs().max())), f"call {call}"
        err = float((y - y_ref).abs().max())
        assert err <= tol_y * scale, f"call {call}: max|diff| {err:.3e} vs RMS {scale:.3e}"
    ctx.close()


_FIRST_CALL = r"""
import sys
sys.path.insert(0, {root!r})
import numpy as np, torch
from oracle import spark_oracle as O
from paper_2506_06644_b200 import binding as S, synth
d, d_ff, r, k = 512, 3000, 256, 240
p = synth.ffn_inputs(d, d_ff, r, k, 1, "bf16", seed=5)
f = lambda bits: torch.from_numpy(bits.view(np.int16)).cuda().view(torch.bfloat16)
K1t, K2t, Vt = f(p.K1t_bits), f(p.K2t_bits), f(p.Vt_bits)
x = torch.from_numpy(p.x).cuda()
y = torch.full((1, d), float("nan"), device="cuda")
th = torch.full((1,), float("nan"), device="cuda")
torch.cuda.synchronize()
side = torch.cuda.Stream()                     # a non-blocking stream: nothing orders it behind the default stream
with torch.cuda.stream(side):
    # the very first call of the library in this process, on the side stream
    S.spark_ffn_decode_noalloc(x, 1, K1t, K2t, Vt, S.SPARK_BF16, d, d_ff, r, k, 0, y, th)
    S.spark_ffn_decode_noalloc(x, 1, K1t, K2t, Vt, S.SPARK_BF16, d, d_ff, r, k, 0, y, th)
    assert S.spark_noalloc_status() == S.SPARK_OK
ref = O.spark_ffn(p.x[0], p.K1t.astype(np.float64).T, p.K2t.astype(np.float64).T, p.Vt.astype(np.float64).T, k, r)
err = float(np.max(np.abs(y.cpu().numpy()[0] - ref["y"]))) / float(np.sqrt(np.mean(ref["y"] ** 2)))
assert err <= 2e-2, err
assert abs(float(th[0]) - ref["theta"]) <= 1e-5 * max(abs(ref["theta"]), float(np.std(ref["s"], ddof=1)))
print("FIRST_CALL_OK")
"""


def test_first_call_of_a_fresh_process_may_go_to_a_side_stream():
    res = subprocess.run([sys.executable, "-c", _FIRST_CALL.format(root=ROOT)], capture_output=True, text=True, timeout=600)
    assert res.returncode == 0 and "FIRST_CALL_OK" in res.stdout, res.stdout[-2000:] + res.stderr[-2000:]


def test_noalloc_rejects_more_tokens_than_its_static_state_serves():
    d, d_ff, r = 64, 128, 32
    B = 17
    x = torch.zeros((B, d), device="cuda")
    w1 = torch.zeros((d_ff, r), device="cuda")
    w2 = torch.zeros((d_ff, d - r), device="cuda")
    v = torch.zeros((d_ff, d), device="cuda")
    y = torch.zeros((B, d), device="cuda")
    with pytest.raises(S.SparkError) as e:
        S.spark_ffn_decode_noalloc(x, B, w1, w2, v, S.SPARK_F32, d, d_ff, r, 10, 0, y, None)
    assert e.value.status == S.SPARK_ERR_UNSUPPORTED
