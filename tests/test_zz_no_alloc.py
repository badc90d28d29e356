"""The allocation-free GEMM entry point gives the same results as the regular one.

lp_gemm_bf16_static is for callers that may not call cudaMalloc where they launch work (a serving
or real-time loop that must not take the driver's allocator lock, a plug-in whose host has handed
out the whole device-memory budget); it keeps its problem table in a fixed array inside the
library.  Checked here: two calls in a row (the second with other problems, so the array still
holds the first call's table when it starts; the outputs are cleared in between, so each call's
results are its own) against lp_gemm_bf16 on the same inputs and against the CPU oracle's Linear
layer, the status poll, and that an oversized request is refused.  This file sorts last on purpose: a run that stops at the
first failure has then already run every other test.
"""
import numpy as np
import pytest
import torch

import lp_synth
from oracle import layers as OL
from paper_2012_03837_b200 import binding as lp

pytestmark = pytest.mark.gpu


def make(M, N, K, seed):
    """Forward, input-gradient and weight-gradient products of one Linear layer, two output sets."""
    g = np.random.default_rng(seed)
    bf = lambda a: torch.from_numpy(lp_synth.bf16_round(a.astype(np.float32))).cuda().to(torch.bfloat16).contiguous()
    x, W, dy = bf(g.standard_normal((M, K))), bf(g.standard_normal((N, K)) / np.sqrt(K)), bf(g.standard_normal((M, N)))
    b = torch.from_numpy(g.standard_normal(N).astype(np.float32)).cuda()
    outs = []
    for _ in range(2):
        outs.append(dict(y=torch.zeros(M, N, dtype=torch.bfloat16, device="cuda"),
                         dx=torch.zeros(M, K, dtype=torch.bfloat16, device="cuda"),
                         dW=torch.zeros(N, K, dtype=torch.float32, device="cuda")))

    def descs(o):
        return [dict(A=x, B=W, C=o["y"], bias=b, M=M, N=N, K=K, a_ms=K, a_ks=1, b_ns=K, b_ks=1, ldc=N, act=1),
                dict(A=dy, B=W, C=o["dx"], M=M, N=K, K=N, a_ms=N, a_ks=1, b_ns=1, b_ks=K, ldc=K),
                dict(A=dy, B=x, C=o["dW"], M=N, N=K, K=M, a_ms=1, a_ks=N, b_ns=1, b_ks=K, ldc=K, out_f32=1)]
    return (x, W, dy, b), outs, descs


def compare(ref, got):
    for k in ref:
        a, b = got[k].float().cpu().numpy(), ref[k].float().cpu().numpy()
        assert np.abs(b).max() > 0
        assert np.abs(a - b).max() <= 1e-2 * np.abs(b).max(), k


def compare_oracle(keep, got):
    """Against the oracle's Linear layer (App. A.1): y = relu(x W^T + b), dx = dy W, dW = dy^T x."""
    x, W, dy, b = (t.float().cpu().numpy().astype(np.float64) for t in keep)
    y, cache = OL.linear_fwd(x, W, b)
    y = np.maximum(y, 0.0)
    dx, dW, _ = OL.linear_bwd(dy, cache)
    for k, ref in (("y", y), ("dx", dx), ("dW", dW)):
        a = got[k].float().cpu().numpy()
        assert np.abs(a - ref).max() <= 1e-2 * np.abs(ref).max(), k


def clear(o):
    for t in o.values():
        t.zero_()


def test_static_entry_matches_regular_entry_on_two_calls_in_a_row():
    keep1, outs1, d1 = make(264, 520, 136, 11)       # ragged: tensor-core kernel, partial tiles
    keep2, outs2, d2 = make(40, 24, 200, 12)         # too small for the tensor-core kernel: FP32-ALU kernel
    keep3, outs3, d3 = make(384, 256, 320, 13)
    lp.lp_gemm_bf16(d1(outs1[0]) + d3(outs3[0]), 0)
    lp.lp_gemm_bf16(d2(outs2[0]), 0)
    torch.cuda.synchronize()
    lp.lp_gemm_bf16_static(d1(outs1[1]) + d3(outs3[1]))     # first call: does the one-time set-up
    lp.lp_gemm_static_poll()                                 # synchronises; no device-side wait gave up
    compare(outs1[0], outs1[1])
    compare(outs3[0], outs3[1])
    compare_oracle(keep1, outs1[1])
    compare_oracle(keep3, outs3[1])
    clear(outs1[1])                                          # what the second call leaves is its own work
    lp.lp_gemm_bf16_static(d2(outs2[1]) + d1(outs1[1]))     # second call reuses the array
    lp.lp_gemm_static_poll()
    compare(outs1[0], outs1[1])
    compare(outs2[0], outs2[1])
    compare_oracle(keep1, outs1[1])
    compare_oracle(keep2, outs2[1])


def test_static_entry_rejects_more_problems_than_its_table_holds():
    keep, outs, d = make(128, 256, 64, 5)
    too_many = (d(outs[0]) * 22)[:lp.LP_GEMM_STATIC_MAX + 1]
    with pytest.raises(lp.LpError) as e:
        lp.lp_gemm_bf16_static(too_many)
    assert e.value.code == -2 and "64" in str(e.value)
    lp.lp_gemm_bf16_static(d(outs[1]))               # still usable afterwards
    torch.cuda.synchronize()
