"""The tensor-core attention kernels (lp_attention_bf16) against the oracle's causal attention (App. B.2's
transformer layers), forward and backward, element by element: sequence lengths that end inside a tile, span
several 128-row tiles, and the lengths of the two transformer workloads."""
import numpy as np
import pytest
import torch

import lp_synth
from oracle import layers as OL
from paper_2012_03837_b200 import binding as lp

pytestmark = pytest.mark.gpu


def run_case(B, T, H, seed):
    g = np.random.default_rng(seed)
    d = 64 * H
    qkv = lp_synth.bf16_round(g.standard_normal((B, T, 3 * d)).astype(np.float32) * 1.5)
    dout = lp_synth.bf16_round(g.standard_normal((B, T, d)).astype(np.float32))
    dev = torch.device("cuda:0")
    t_qkv = torch.from_numpy(qkv).to(dev).to(torch.bfloat16).contiguous()
    t_do = torch.from_numpy(dout).to(dev).to(torch.bfloat16).contiguous()
    t_o = torch.full((B, T, d), float("nan"), dtype=torch.bfloat16, device=dev)
    t_lse = torch.full((B, H, T), float("nan"), dtype=torch.float32, device=dev)
    t_dqkv = torch.full((B, T, 3 * d), float("nan"), dtype=torch.bfloat16, device=dev)
    t_delta = torch.full((B, H, T), float("nan"), dtype=torch.float32, device=dev)
    lp.lp_attention_bf16(lp.LP_ATTN_FORWARD, t_qkv, t_o, t_lse, None, None, None, B, T, H)
    o_ref, cache = OL.attention_fwd(qkv.astype(np.float64), H)
    o = t_o.float().cpu().numpy()
    assert np.all(np.isfinite(o))
    assert np.abs(o - o_ref).max() <= 2e-2 * np.abs(o_ref).max(), ("o", np.abs(o - o_ref).max(), np.abs(o_ref).max())
    # the saved statistic: log2 of the softmax denominator, in base-2 score units
    q, k = cache[0], cache[1]
    s2 = (q @ k.transpose(0, 1, 3, 2)) * (0.125 * np.log2(np.e))
    s2 = np.where(np.triu(np.ones((T, T), dtype=bool), 1), -np.inf, s2)
    m = s2.max(axis=-1)
    lse_ref = m + np.log2(np.exp2(s2 - m[..., None]).sum(axis=-1))
    assert np.abs(t_lse.cpu().numpy() - lse_ref).max() <= 2e-3 * max(1.0, np.abs(lse_ref).max())

    lp.lp_attention_bf16(lp.LP_ATTN_BACKWARD, t_qkv, t_o, t_lse, t_do, t_dqkv, t_delta, B, T, H)
    # the backward of the oracle at the forward output as the kernels see it (o rounded to bf16 enters delta only)
    dqkv_ref = OL.attention_bwd(dout.astype(np.float64), cache)
    dqkv = t_dqkv.float().cpu().numpy()
    assert np.all(np.isfinite(dqkv))
    for name, sl in (("dq", slice(0, d)), ("dk", slice(d, 2 * d)), ("dv", slice(2 * d, 3 * d))):
        a, r = dqkv[..., sl], dqkv_ref[..., sl]
        assert np.abs(a - r).max() <= 2e-2 * np.abs(r).max(), (name, np.abs(a - r).max(), np.abs(r).max())
    delta_ref = (dout.astype(np.float64) * o.astype(np.float64)).reshape(B, T, H, 64).sum(-1).transpose(0, 2, 1)
    assert np.abs(t_delta.cpu().numpy() - delta_ref).max() <= 1e-3 * max(1.0, np.abs(delta_ref).max())


@pytest.mark.parametrize("B,T,H", [(1, 64, 1), (2, 128, 2), (1, 200, 2), (3, 136, 1), (2, 37, 3), (1, 1, 1),
                                   (2, 256, 2), (1, 512, 2), (1, 700, 1)])
def test_attention_matches_the_oracle(B, T, H):
    run_case(B, T, H, seed=100 + T)


def test_causal_future_tokens_do_not_matter():
    """Changing positions after t leaves the outputs up to t bit-identical."""
    B, T, H, d = 1, 300, 2, 128
    g = np.random.default_rng(5)
    qkv = torch.from_numpy(lp_synth.bf16_round(g.standard_normal((B, T, 3 * d)).astype(np.float32))).cuda().to(torch.bfloat16)
    o1 = torch.zeros(B, T, d, dtype=torch.bfloat16, device="cuda")
    o2 = torch.zeros_like(o1)
    lse = torch.zeros(B, H, T, dtype=torch.float32, device="cuda")
    lp.lp_attention_bf16(lp.LP_ATTN_FORWARD, qkv, o1, lse, None, None, None, B, T, H)
    qkv2 = qkv.clone()
    qkv2[:, 150:, :] = -qkv2[:, 150:, :] * 2
    lp.lp_attention_bf16(lp.LP_ATTN_FORWARD, qkv2, o2, lse, None, None, None, B, T, H)
    assert torch.equal(o1[:, :150], o2[:, :150]) and not torch.equal(o1[:, 150:], o2[:, 150:])
