"""Micro-benchmark of the grouped bf16 GEMM through the C ABI (lp_gemm_bf16): the Linear-layer
products of the transformer workloads in forward, input-gradient and weight-gradient form.

    python -m paper_2012_03837_b200.kernel_bench [--shape qkv|out|ffn1|ffn2|head|all] [--form fwd|dgrad|wgrad|all]
                                                 [--d 1024] [--rows 8192] [--vocab 32768] [--groups 4] [--reps 10]
                                                 [--epilogue none|model]
    python -m paper_2012_03837_b200.kernel_bench --shape attn [--batch 64] [--seq 512] [--heads 16] [--reps 10]

Prints one JSON line per (shape, form): milliseconds per launch and TFLOP/s (2*M*N*K per problem; attention:
4 (forward) or 10 (backward) x batch x heads x 64 x T(T+1)/2).
Inputs are larger than the L2 cache in total, so every launch streams its operands from HBM.
"""
from __future__ import annotations

import argparse
import json

import torch

from . import binding as lp


def shapes(d, ffn, vocab):
    return {"qkv": (3 * d, d), "out": (d, d), "ffn1": (ffn, d), "ffn2": (d, ffn), "head": (vocab, d)}


# fused epilogue of each product in the transformer block (--epilogue model): (bias, residual, activation)
EPI_NONE, EPI_GELU, EPI_GELU_GRAD = 0, 2, 4
MODEL_EPILOGUE = {("qkv", "fwd"): (True, False, EPI_NONE), ("out", "fwd"): (True, True, EPI_NONE),
                  ("ffn1", "fwd"): (True, False, EPI_GELU), ("ffn2", "fwd"): (True, True, EPI_NONE),
                  ("head", "fwd"): (True, False, EPI_NONE), ("ffn2", "dgrad"): (False, False, EPI_GELU_GRAD)}


def descs(form, rows, n_out, n_in, groups, epilogue=(False, False, EPI_NONE)):
    """`groups` independent Linear layers y = x W^T with x [rows, n_in], W [n_out, n_in]."""
    out, keep = [], []
    bf = dict(dtype=torch.bfloat16, device="cuda")
    bias, resid, act = epilogue
    for _ in range(groups):
        x = torch.randn(rows, n_in, **bf)
        W = torch.randn(n_out, n_in, **bf) * 0.02
        dy = torch.randn(rows, n_out, **bf)
        if form == "fwd":
            c = torch.empty(rows, n_out, **bf)
            d = dict(A=x, B=W, C=c, M=rows, N=n_out, K=n_in, a_ms=n_in, a_ks=1, b_ns=n_in, b_ks=1, ldc=n_out, act=act)
            if bias:
                d["bias"] = torch.randn(n_out, dtype=torch.float32, device="cuda")
            if resid:
                d["resid"] = torch.randn(rows, n_out, **bf)
            if act == EPI_GELU:
                d["C2"] = torch.empty(rows, n_out, **bf)
            keep += [v for v in d.values() if torch.is_tensor(v)]
            out.append(d)
        elif form == "dgrad":
            c = torch.empty(rows, n_in, **bf)
            d = dict(A=dy, B=W, C=c, M=rows, N=n_in, K=n_out, a_ms=n_out, a_ks=1, b_ns=1, b_ks=n_in, ldc=n_in, act=act)
            if act == EPI_GELU_GRAD:
                d["aux"] = torch.randn(rows, n_in, **bf)
                keep.append(d["aux"])
            out.append(d)
        else:
            c = torch.empty(n_out, n_in, dtype=torch.float32, device="cuda")
            out.append(dict(A=dy, B=x, C=c, M=n_out, N=n_in, K=rows, a_ms=1, a_ks=n_out, b_ns=1, b_ks=n_in, ldc=n_in, out_f32=1))
        keep += [x, W, dy, c]
    return out, keep


def attention(a):
    """Causal attention (lp_attention_bf16) forward and backward on [batch, seq, 3 * 64 * heads]."""
    B, T, H = a.batch, a.seq, a.heads
    d = 64 * H
    bf = dict(dtype=torch.bfloat16, device="cuda")
    qkv, dout = torch.randn(B, T, 3 * d, **bf), torch.randn(B, T, d, **bf)
    o, dqkv = torch.empty(B, T, d, **bf), torch.empty(B, T, 3 * d, **bf)
    lse = torch.empty(B, H, T, dtype=torch.float32, device="cuda")
    delta = torch.empty_like(lse)
    pairs = B * H * 64.0 * T * (T + 1) / 2
    for form, name, mult in ((lp.LP_ATTN_FORWARD, "fwd", 4.0), (lp.LP_ATTN_BACKWARD, "bwd", 10.0)):
        for _ in range(2):
            lp.lp_attention_bf16(form, qkv, o, lse, dout, dqkv, delta, B, T, H)
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for _ in range(a.reps):
            lp.lp_attention_bf16(form, qkv, o, lse, dout, dqkv, delta, B, T, H)
        e1.record()
        torch.cuda.synchronize()
        ms = e0.elapsed_time(e1) / a.reps          # each call synchronises: includes ~20 us of host latency
        print(json.dumps(dict(shape="attn", form=name, batch=B, seq=T, heads=H, ms_per_call=ms, tflops=mult * pairs / ms / 1e9)))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--shape", default="all")
    ap.add_argument("--form", default="all")
    ap.add_argument("--d", type=int, default=1024)
    ap.add_argument("--rows", type=int, default=8192)
    ap.add_argument("--vocab", type=int, default=32768)
    ap.add_argument("--groups", type=int, default=4)
    ap.add_argument("--reps", type=int, default=10)
    ap.add_argument("--backend", type=int, default=0)
    ap.add_argument("--epilogue", default="none", choices=["none", "model"],
                    help="model: the bias / residual / GELU / GELU' epilogue that product has in the transformer block")
    ap.add_argument("--batch", type=int, default=64)
    ap.add_argument("--seq", type=int, default=512)
    ap.add_argument("--heads", type=int, default=16)
    a = ap.parse_args()
    if a.shape == "attn":
        attention(a)
        return
    sh = shapes(a.d, 4 * a.d, a.vocab)
    names = list(sh) if a.shape == "all" else [a.shape]
    forms = ["fwd", "dgrad", "wgrad"] if a.form == "all" else [a.form]
    stream = torch.cuda.current_stream().cuda_stream
    for name in names:
        n_out, n_in = sh[name]
        groups = max(1, a.groups // 4) if name == "head" else a.groups
        for form in forms:
            epi = MODEL_EPILOGUE.get((name, form), (False, False, EPI_NONE)) if a.epilogue == "model" else (False, False, EPI_NONE)
            ds, keep = descs(form, a.rows, n_out, n_in, groups, epi)
            for _ in range(3):
                used = lp.lp_gemm_bf16(ds, a.backend, stream)
            torch.cuda.synchronize()
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            for _ in range(a.reps):
                lp.lp_gemm_bf16(ds, a.backend, stream)
            e1.record()
            torch.cuda.synchronize()
            ms = e0.elapsed_time(e1) / a.reps
            flops = 2.0 * a.rows * n_out * n_in * groups
            print(json.dumps(dict(shape=name, form=form, rows=a.rows, n_out=n_out, n_in=n_in, groups=groups,
                                  tensor_core_problems=used, ms_per_launch=ms, tflops=flops / ms / 1e9)))
            del ds, keep
            torch.cuda.empty_cache()


if __name__ == "__main__":
    main()
