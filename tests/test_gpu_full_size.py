"""Parity at the full sizes of the five workloads, in the launch configuration bench.py times.

c1 runs in test_gpu_parity.py.  c2, c3 and c4 run ten steps against the oracle.  c3 meets the nominal 2e-2.  The
bounds of c2 and c4 follow, step by step, what two correct evaluations of those workloads differ by
(tests/golden/c2_conditioning.json, c4_conditioning.json, made by the CPU oracle alone): the nominal tolerance
while twice that gap stays below it, twice the oracle-against-oracle gap afterwards.  c5
(55 TFLOP per step) is checked on what the oracle can compute one by one.  A chunk's update depends on the
chunks below it only through the activation it receives (Sec. 3), so (a) for chunks 0, 1, 12 and 23 the oracle
forms the input by a forward pass through the blocks below and one local update of that chunk alone, and (b) a
three-chunk oracle with the same seeded weights reproduces chunks 0-2 of the 24 over three pipelined steps
(both halves of the boundary buffers, labels carried with the activations); plus properties that hold at any
size (initial losses near ln V for every chunk, first Adam step bounded by the learning rate).
"""
import json
import math
import os

import numpy as np
import pytest

import lp_synth
from oracle.local_step import LocalUpdateOracle
from paper_2012_03837_b200 import binding as lp
from tests import lp_testlib as T
from tests.test_gpu_parity import check

pytestmark = pytest.mark.gpu

def golden(name):
    return json.load(open(os.path.join(os.path.dirname(os.path.abspath(__file__)), "golden", f"{name}_conditioning.json")))["steps"]


def gaps(gm, orc, init):
    """Per chunk: the largest ||a-b||_2 / ||b||_2 over its weight matrices, and the largest ||a-b||_2 / ||b-init||_2
    over its vectors (they start at 0 or 1: the error of the accumulated update itself)."""
    got = gm.get(lp.LP_MASTER)
    mats, vecs = [0.0] * gm.K, [0.0] * gm.K
    for n, a in got.items():
        if n in orc.buffers:
            continue
        k = gm.index[n][1]["chunk"]
        a = T.strip_key_bias(n, a.astype(np.float64))
        b = T.strip_key_bias(n, orc.p[n].astype(np.float64))
        e = float(np.linalg.norm(a - b))
        if got[n].ndim >= 2:
            mats[k] = max(mats[k], e / float(np.linalg.norm(b)))
        else:
            i0 = T.strip_key_bias(n, np.asarray(init[n], dtype=np.float64))
            vecs[k] = max(vecs[k], e / max(float(np.linalg.norm(b - i0)), 1e-30))
    return mats, vecs


def run_against_witness(cfg, witnesses, base_w, base_loss, base_v):
    """Ten steps, compared after every step.  The bound at step t is max(nominal tolerance, 2 x the gap between two
    correct evaluations of this workload at step t), the gap taken from tests/golden/<workload>_conditioning.json
    (CPU oracle alone) as the largest over the chunks, over the listed witnesses and over steps t and t+1: which
    chunk a rounding event hits, and at which step the first one falls, is chance.  Losses: the gap is a series of isolated transients that move down the pipeline with the
    minibatch that caused them, and their size differs between two realisations of the same kind of perturbation
    by more than a factor of two (5.6e-3 and 1.3e-2 in the two bf16 witnesses of c2; the library's largest: 3.0e-2
    in bf16, 5.3e-3 with fp32 storage against 1.5e-3 of the fp32 witness), so the bound is
    max(nominal, 4 x the largest gap of any witness at any of the ten steps)."""
    gold = golden(cfg["name"])
    loss_tol = max(base_loss, 4 * max(max(s[w]["loss"]) for s in gold for w in witnesses))
    params = lp_synth.init_params(cfg)
    gm = T.GpuModel(cfg, params)
    orc = LocalUpdateOracle(cfg, params, dtype=np.float32)
    for t in range(10):
        x, y = lp_synth.minibatch(cfg, t)
        gl, ol = gm.step(x, y), orc.step(x, y)
        lerr = np.abs(gl - ol) / np.abs(ol)
        w, v = gaps(gm, orc, params)
        near = (t, min(t + 1, 9))                            # when the first rounding event falls is chance: one step of slack
        w_tol = max(base_w, 2 * max(max(gold[u][wn]["weights"]) for wn in witnesses for u in near))
        v_tol = max(base_v, 2 * max(max(gold[u][wn]["vectors"]) for wn in witnesses for u in near))
        print(f"{cfg['name']} {cfg['dtype']} step {t + 1}: loss err {lerr.max():.2e} (tol {loss_tol:.2e}); matrices "
              f"{max(w):.2e} (tol {w_tol:.2e}) per chunk {[f'{a:.1e}' for a in w]}; vectors {max(v):.2e} (tol {v_tol:.2e})")
        assert lerr.max() <= loss_tol, (t, lerr)
        assert max(w) <= w_tol, (t, w, w_tol)
        assert max(v) <= v_tol, (t, v, v_tol)
    gm.close()


def test_c2_wide_mlp_full_size_fp32_storage():
    """The c2 network and schedule with fp32 storage (FP32-ALU kernels) against the fp32 oracle: two fp32
    evaluations that differ in summation order only.  The witness is the oracle in fp32 against itself in fp64,
    which reaches 2.2e-2 of a weight matrix's norm after ten steps on the CPU alone."""
    run_against_witness(lp_synth.config("c2", dtype="fp32"), ["fp32_vs_fp64"], 1e-3, 1e-4, 1e-3)


def test_c2_wide_mlp_bf16_full_size():
    """bf16 storage.  The witnesses are the fp32 oracle with its weight matrices (as the passes read them) and every
    layer's stored output rounded to bf16, and the fp32 oracle with only its chunk outputs rounded, each against the
    plain fp32 oracle: 2e-2 of a weight matrix's norm is crossed within four steps on the CPU alone."""
    run_against_witness(lp_synth.config("c2"), ["bf16io_vs_fp32", "bf16out_vs_fp32"], 2e-2, 2e-2, 2e-1)


def test_c3_transformer_bf16_full_size():
    check(lp_synth.config("c3"), steps=10, grads_first=False)


def test_c4_resnet_bf16_full_size():
    """Ten steps of SGD with lr 0.1 and momentum 0.9 move the small head matrices by a multiple of their initial
    norm, so they carry the gradient's bf16 error like the vectors do; same witness as for c2."""
    run_against_witness(lp_synth.config("c4"), ["bf16io_vs_fp32"], 2e-2, 2e-2, 2e-1)


def l2_rel(a, b):
    a, b = a.astype(np.float64), b.astype(np.float64)
    return float(np.linalg.norm(a - b) / max(np.linalg.norm(b), 1e-30))


def test_c5_large_transformer_sampled_chunks_and_pipelined_steps():
    cfg = lp_synth.config("c5")
    K = lp_synth.num_chunks(cfg)
    params = lp_synth.init_params(cfg)
    gm = T.GpuModel(cfg, params)
    lr = cfg["optim"]["lr"]
    # logits of a fresh head are N(0, s^2) with s^2 = 0.02^2 * d_model (LayerNorm output has unit variance), so
    # the expected loss is ln V + s^2 / 2 (log-normal mean of the partition function)
    expect0 = math.log(cfg["vocab"]) + 0.5 * 0.02 ** 2 * cfg["d_model"]

    # ---- (a) step 0 (pipelined, primed: every chunk trains on minibatch 0), chunks 0, 1, 12, 23
    x0, y0 = lp_synth.minibatch(cfg, 0)
    losses0 = gm.step(x0, y0)
    assert np.all(np.abs(losses0 - expect0) < 0.05), losses0
    full = LocalUpdateOracle(cfg, params, dtype=np.float32)
    sampled = (0, 1, 12, 23)
    inputs, h = {}, full._cast_input(x0)
    for k in range(K):
        if k in sampled:
            inputs[k] = h
        if k < K - 1:
            h, _ = full.chunk_forward(k, h)          # initial weights: the priming pass of the first pipelined step
    worst_g, worst_w = 0.0, 0.0
    for k in sampled:
        loss, _, grads = full.local_grads(k, inputs[k], y0)
        full.apply_update(k, grads)
        assert abs(losses0[k] - loss) / abs(loss) <= 2e-2, (k, losses0[k], loss)
        for n, g_ref in grads.items():
            i, info = gm.index[n]
            g = np.empty(info["shape"], np.float32)
            w = np.empty(info["shape"], np.float32)
            lp.lp_get_tensor(gm.h, i, lp.LP_GRAD, g, gm.stream)
            lp.lp_get_tensor(gm.h, i, lp.LP_MASTER, w, gm.stream)
            if g.ndim == 2:
                ge = l2_rel(g, g_ref)
                worst_g = max(worst_g, ge)
                assert ge <= 0.1, (n, ge)            # bf16 rounding of the activations: a few percent in l2
                we = l2_rel(w, full.p[n])
                worst_w = max(worst_w, we)
                assert we <= 2e-2, (n, we)
            # first Adam step: |dw| = lr |g| / (|g| + eps) <= lr
            dw = np.abs(w.astype(np.float64) - params[n].astype(np.float64)).max()
            assert dw <= lr * (1 + 1e-3), (n, dw)
        print(f"c5 step 0 chunk {k}: loss gpu {losses0[k]:.5f} oracle {loss:.5f}")
    print("c5 sampled chunks: worst first-step matrix gradient error (l2)", worst_g, "worst matrix error after the update", worst_w)
    del full, inputs

    # ---- (b) three pipelined steps, chunks 0-2 against a three-chunk oracle (same seeded tensors)
    small = lp_synth.config("c5", blocks_per_chunk=[1, 1, 1])
    p_small = lp_synth.init_params(small)
    for n, a in p_small.items():                     # same seeded stream per tensor
        assert np.array_equal(a, params[n]), n
    del params
    orc = LocalUpdateOracle(small, p_small, dtype=np.float32)
    ol = orc.step(x0, y0, "pipelined")
    assert np.all(np.abs(losses0[:3] - ol) / np.abs(ol) <= 2e-2), (losses0[:3], ol)
    for t in (1, 2):
        x, y = lp_synth.minibatch(cfg, t)
        gl = gm.step(x, y)
        ol = orc.step(x, y, "pipelined")
        print(f"c5 pipelined step {t}: losses chunk 0-2 gpu", gl[:3], "oracle", ol)
        assert np.all(np.abs(gl[:3] - ol) / np.abs(ol) <= 2e-2), (t, gl[:3], ol)
        # chunks k > 0 see an older minibatch again with the labels they have just trained on: every loss stays
        # finite and in the neighbourhood of its initial value
        assert np.all(np.isfinite(gl)) and np.all(np.abs(gl - expect0) < 1.5), gl
    worst = 0.0
    for n in p_small:
        i, info = gm.index[n]
        if len(info["shape"]) == 2:
            w = np.empty(info["shape"], np.float32)
            lp.lp_get_tensor(gm.h, i, lp.LP_MASTER, w, gm.stream)
            e = l2_rel(w, orc.p[n])
            worst = max(worst, e)
            assert e <= 2e-2, (n, e)
    print("c5 chunks 0-2 after three pipelined steps: worst matrix error", worst)
    gm.close()
