"""Parity at the full sizes of the five workloads, in the launch configuration bench.py times.

c1 runs in test_gpu_parity.py.  c2 runs all ten steps against the oracle.  c3 and c4 run three steps
(an oracle step costs 10-20 s of CPU there).  c5 (55 TFLOP per step) is checked on what the oracle can
compute one by one: chunks 0 and 1 of the 24 (their weights do not depend on the chunks above them, so a
two-chunk oracle with the same seeded weights reproduces them exactly), plus properties that hold at
any size (initial losses near ln V for every chunk, first Adam step bounded by the learning rate).
"""
import math

import numpy as np
import pytest

import lp_synth
from oracle.local_step import LocalUpdateOracle
from paper_2012_03837_b200 import binding as lp
from tests import lp_testlib as T
from tests.test_gpu_parity import check

pytestmark = pytest.mark.gpu


def test_c2_wide_mlp_full_size_fp32_storage():
    """The c2 network and schedule with fp32 storage (FP32-ALU kernels).  This shows how ill-conditioned the
    workload is: Adam's first step moves every weight by +-1e-3 (a thirtieth of the He-normal scale 0.031)
    whatever its gradient's size, the losses fall to ln 1000 within ten steps, and fp32 summation-order
    differences alone grow to 2.5e-2 of the weight norm and 5e-3 of a loss (a transient that follows
    minibatch 1 down the pipeline).  No implementation whose rounding order differs from the oracle's can do
    better, so these bounds, not 1e-3, are what this network admits."""
    check(lp_synth.config("c2", dtype="fp32"), steps=10, grads_first=False, w_tol=5e-2, v_tol=0.5, loss_tol=1e-2)


def test_c2_wide_mlp_bf16_full_size():
    # On top of the above, bf16 activation rounding flips ReLU decisions behind up to 14 layers: measured
    # 5.6e-2 of the weight norm at chunk 7 (1.5e-2 at chunk 0) and 3e-2 on one loss of the same transient.
    check(lp_synth.config("c2"), steps=10, grads_first=False, w_tol=1e-1, v_tol=0.6, loss_tol=5e-2)


def test_c3_transformer_bf16_full_size():
    check(lp_synth.config("c3"), steps=3, grads_first=False)


def test_c4_resnet_bf16_full_size():
    check(lp_synth.config("c4"), steps=3, grads_first=False, v_tol=0.3)


def test_c5_large_transformer_sampled_chunks():
    cfg = lp_synth.config("c5")
    small = lp_synth.config("c5", blocks_per_chunk=[1, 1])
    p_small = lp_synth.init_params(small)
    params = lp_synth.init_params(cfg)
    for n, a in p_small.items():                     # same seeded stream per tensor index
        assert np.array_equal(a, params[n]), n
    gm = T.GpuModel(cfg, params)
    del params
    x, y = lp_synth.minibatch(cfg, 0)
    losses = gm.step(x, y)                           # pipelined step 0: priming forward + one update of all 24 chunks
    # logits of a fresh head are N(0, s^2) with s^2 = 0.02^2 * d_model (LayerNorm output has unit variance), so
    # the expected loss is ln V + s^2 / 2 (log-normal mean of the partition function)
    expect0 = math.log(cfg["vocab"]) + 0.5 * 0.02 ** 2 * cfg["d_model"]
    assert np.all(np.abs(losses - expect0) < 0.05), losses

    orc = LocalUpdateOracle(small, p_small, dtype=np.float32)
    ol = orc.step(x, y, "pipelined")
    print("c5 step-0 losses chunk 0/1: gpu", losses[:2], "oracle", ol)
    assert np.all(np.abs(losses[:2] - ol) / np.abs(ol) <= 2e-2)

    worst_g, worst_w = 0.0, 0.0
    for n in p_small:
        i, info = gm.index[n]
        g = np.empty(info["shape"], np.float32)
        w = np.empty(info["shape"], np.float32)
        lp.lp_get_tensor(gm.h, i, lp.LP_GRAD, g, gm.stream)
        lp.lp_get_tensor(gm.h, i, lp.LP_MASTER, w, gm.stream)
        ge = T.tensor_rel_err(T.strip_key_bias(n, g), T.strip_key_bias(n, orc.last_grads[n]))
        worst_g = max(worst_g, ge)
        # first Adam step: |dw| = lr |g| / (|g| + eps) <= lr
        dw = np.abs(w.astype(np.float64) - p_small[n].astype(np.float64)).max()
        assert dw <= cfg["optim"]["lr"] * (1 + 1e-3), (n, dw)
        if w.ndim == 2:
            we = np.linalg.norm(w.astype(np.float64) - orc.p[n]) / np.linalg.norm(orc.p[n])
            worst_w = max(worst_w, we)
    print("c5 chunk 0/1: worst first-step gradient error", worst_g, "worst matrix error after the update", worst_w)
    assert worst_g <= 0.35
    assert worst_w <= 2e-2
    # one more step keeps every loss finite and in the neighbourhood of the initial value (chunks k > 0 now see
    # minibatch 0 again, one chunk further down, with the labels they have just trained on: their loss drops ~0.4)
    losses2 = gm.step(*lp_synth.minibatch(cfg, 1))
    assert np.all(np.isfinite(losses2)) and np.all(np.abs(losses2 - expect0) < 1.0), losses2
    gm.close()
