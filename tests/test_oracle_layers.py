"""Pins for the oracle's layers: closed forms, brute force, invariants, finite differences.
None of these re-types the oracle's own formula; each fixes a value by another route."""
import math
import os

import numpy as np
import pytest

from oracle import flops
from oracle import layers as L
from oracle import optim as O

RNG = np.random.default_rng(1234)


def fd_grad(f, x, eps=1e-6):
    """Central finite differences of scalar f with respect to array x (fp64)."""
    g = np.zeros_like(x)
    it = np.nditer(x, flags=["multi_index"])
    for _ in it:
        i = it.multi_index
        old = x[i]
        x[i] = old + eps
        fp = f()
        x[i] = old - eps
        fm = f()
        x[i] = old
        g[i] = (fp - fm) / (2 * eps)
    return g


def rel(a, b):
    return np.abs(a - b).max() / max(np.abs(b).max(), 1e-30)


# ---------------------------------------------------------------- App. A.1 worked example

def test_flops_worked_example_matches_paper():
    vals = {}
    with open(os.path.join(os.path.dirname(__file__), "golden", "mlp_flops.txt")) as f:
        for line in f:
            if line.startswith("#") or not line.strip():
                continue
            k, v = line.split()
            vals[k] = float(v)
    assert flops.mlp_mean_forward_flops(int(vals["input_size"]), int(vals["hidden"]), int(vals["layers"])) == vals["mean_forward_flops"]
    assert flops.mlp_aux_flops(int(vals["hidden"])) == vals["aux_flops"]


def test_cost_model_backprop_is_one_chunk_and_greedy_is_L_chunks():
    f, a, bm, layers = 100.0, 7.0, 1.5, 8
    assert flops.cost_per_example("chunked", f, a, bm, layers, chunks=1) == flops.cost_per_example("backprop", f, a, bm, layers)
    assert flops.cost_per_example("chunked", f, a, bm, layers, chunks=layers) == flops.cost_per_example("greedy", f, a, bm, layers)
    assert flops.cost_per_example("overlapping", f, a, bm, layers) > flops.cost_per_example("greedy", f, a, bm, layers)


# ---------------------------------------------------------------- softmax cross-entropy

def test_xent_equal_logits_is_log_classes():
    for c in (10, 1000):
        z = np.full((7, c), 3.25)
        y = RNG.integers(0, c, 7).astype(np.int32)
        loss, dz = L.softmax_xent(z, y)
        assert abs(loss - math.log(c)) < 1e-12
        assert np.allclose(dz.sum(axis=1), 0, atol=1e-15)


def test_xent_ignore_rows_and_row_sums():
    z = RNG.standard_normal((9, 6))
    y = np.array([0, 5, -1, 2, -1, 3, 3, 1, -1], dtype=np.int32)
    loss, dz = L.softmax_xent(z, y)
    assert np.all(dz[y < 0] == 0)
    assert np.allclose(dz.sum(axis=1), 0, atol=1e-15)
    # brute force with python floats over the 6 valid rows
    tot = 0.0
    for r in range(9):
        if y[r] >= 0:
            tot += math.log(sum(math.exp(v) for v in z[r])) - z[r, y[r]]
    assert abs(loss - tot / 6) < 1e-12
    assert loss >= 0


def test_xent_gradient_fd():
    z = RNG.standard_normal((5, 4))
    y = np.array([1, -1, 3, 0, 2], dtype=np.int32)
    _, dz = L.softmax_xent(z, y)
    g = fd_grad(lambda: float(L.softmax_xent(z, y)[0]), z)
    assert rel(dz, g) < 1e-7


def test_xent_large_logits_stable():
    z = np.array([[1000.0, 0.0], [-1000.0, 0.0]])
    loss, dz = L.softmax_xent(z, np.array([0, 1], dtype=np.int32))
    assert np.isfinite(loss) and abs(loss) < 1e-12 and np.all(np.isfinite(dz))


# ---------------------------------------------------------------- dense layers, activations

def test_linear_brute_force_and_fd():
    x = RNG.standard_normal((3, 4)); W = RNG.standard_normal((5, 4)); b = RNG.standard_normal(5)
    y, c = L.linear_fwd(x, W, b)
    for r in range(3):
        for o in range(5):
            assert abs(y[r, o] - (sum(x[r, i] * W[o, i] for i in range(4)) + b[o])) < 1e-12
    dy = RNG.standard_normal(y.shape)
    dx, dW, db = L.linear_bwd(dy, c)
    f = lambda: float((L.linear_fwd(x, W, b)[0] * dy).sum())
    assert rel(dx, fd_grad(f, x)) < 1e-7
    assert rel(dW, fd_grad(f, W)) < 1e-7
    assert rel(db, fd_grad(f, b)) < 1e-7


def test_gelu_values_and_fd():
    # closed forms: gelu(0)=0, gelu(x) -> x for large x, gelu(-x) = gelu(x) - x
    x = np.array([0.0, 10.0, -10.0, 0.7, -0.7, 1.0])
    y, c = L.gelu_fwd(x)
    assert y[0] == 0 and abs(y[1] - 10) < 1e-12 and abs(y[2]) < 1e-12
    assert abs((y[3] - y[4]) - 0.7) < 1e-12
    assert abs(y[5] - 0.5 * (1 + math.erf(1 / math.sqrt(2)))) < 1e-15
    assert abs(y[5] - 0.8413447460685429) < 1e-12        # Phi(1), tabulated
    xs = RNG.standard_normal((4, 3))
    dy = RNG.standard_normal((4, 3))
    g = fd_grad(lambda: float((L.gelu_fwd(xs)[0] * dy).sum()), xs)
    assert rel(L.gelu_bwd(dy, (xs,)), g) < 1e-7


def test_relu_mask():
    x = np.array([[-1.0, 2.0, 0.0, 3.0]])
    y, c = L.relu_fwd(x)
    assert np.array_equal(y, [[0, 2, 0, 3]])
    assert np.array_equal(L.relu_bwd(np.ones_like(x), c), [[0, 1, 0, 1]])


# ---------------------------------------------------------------- normalisation

def test_layernorm_invariants_and_fd():
    x = RNG.standard_normal((2, 3, 8)) * 3 + 1
    g = RNG.standard_normal(8); b = RNG.standard_normal(8)
    y, c = L.layernorm_fwd(x, np.ones(8), np.zeros(8), eps=0.0)
    assert np.allclose(y.mean(-1), 0, atol=1e-12) and np.allclose((y ** 2).mean(-1), 1, atol=1e-12)
    dy = RNG.standard_normal(y.shape)
    y0, c0 = L.layernorm_fwd(x, g, b, eps=0.0)      # orthogonality to xhat is exact only at eps=0
    dx0 = L.layernorm_bwd(dy, c0)[0]
    assert np.allclose(dx0.sum(-1), 0, atol=1e-12)
    assert np.allclose((dx0 * c0[0]).sum(-1), 0, atol=1e-12)
    y, c = L.layernorm_fwd(x, g, b)
    dx, dg, db = L.layernorm_bwd(dy, c)
    f = lambda: float((L.layernorm_fwd(x, g, b)[0] * dy).sum())
    assert rel(dx, fd_grad(f, x)) < 1e-6
    assert rel(dg, fd_grad(f, g)) < 1e-7
    assert rel(db, fd_grad(f, b)) < 1e-7


def test_batchnorm_invariants_and_fd():
    x = RNG.standard_normal((3, 4, 2, 2)) * 2 - 1
    g = RNG.standard_normal(4); b = RNG.standard_normal(4)
    y, c = L.batchnorm_fwd(x, np.ones(4), np.zeros(4), eps=0.0)
    assert np.allclose(y.mean((0, 2, 3)), 0, atol=1e-12) and np.allclose((y ** 2).mean((0, 2, 3)), 1, atol=1e-12)
    dy = RNG.standard_normal(y.shape)
    y0, c0 = L.batchnorm_fwd(x, g, b, eps=0.0)
    dx0 = L.batchnorm_bwd(dy, c0)[0]
    assert np.allclose(dx0.sum((0, 2, 3)), 0, atol=1e-12)
    assert np.allclose((dx0 * c0[0]).sum((0, 2, 3)), 0, atol=1e-12)
    y, c = L.batchnorm_fwd(x, g, b)
    dx, dg, db = L.batchnorm_bwd(dy, c)
    f = lambda: float((L.batchnorm_fwd(x, g, b)[0] * dy).sum())
    assert rel(dx, fd_grad(f, x)) < 1e-6
    assert rel(dg, fd_grad(f, g)) < 1e-7
    assert rel(db, fd_grad(f, b)) < 1e-7


# ---------------------------------------------------------------- convolution

def conv_direct(x, W, stride, pad):
    n, c, h, w = x.shape
    o, _, kh, kw = W.shape
    ho = (h + 2 * pad - kh) // stride + 1
    wo = (w + 2 * pad - kw) // stride + 1
    y = np.zeros((n, o, ho, wo))
    for a in range(n):
        for oo in range(o):
            for p in range(ho):
                for q in range(wo):
                    s = 0.0
                    for cc in range(c):
                        for i in range(kh):
                            for j in range(kw):
                                hi, wi = p * stride + i - pad, q * stride + j - pad
                                if 0 <= hi < h and 0 <= wi < w:
                                    s += x[a, cc, hi, wi] * W[oo, cc, i, j]
                    y[a, oo, p, q] = s
    return y


@pytest.mark.parametrize("k,stride,pad,h", [(3, 1, 1, 5), (3, 2, 1, 6), (3, 2, 1, 5), (1, 2, 0, 6)])
def test_conv_matches_direct_loops_and_fd(k, stride, pad, h):
    x = RNG.standard_normal((2, 3, h, h)); W = RNG.standard_normal((4, 3, k, k))
    y, c = L.conv2d_fwd(x, W, stride, pad)
    assert np.allclose(y, conv_direct(x, W, stride, pad), atol=1e-12)
    dy = RNG.standard_normal(y.shape)
    dx, dW = L.conv2d_bwd(dy, c)
    f = lambda: float((L.conv2d_fwd(x, W, stride, pad)[0] * dy).sum())
    assert rel(dx, fd_grad(f, x)) < 1e-7
    assert rel(dW, fd_grad(f, W)) < 1e-7


def test_conv1x1_is_linear_over_channels():
    x = RNG.standard_normal((2, 3, 4, 4)); W = RNG.standard_normal((5, 3, 1, 1))
    y, _ = L.conv2d_fwd(x, W, 1, 0)
    ref = np.einsum("nchw,oc->nohw", x, W[:, :, 0, 0])
    assert np.allclose(y, ref, atol=1e-12)


def test_gap_fwd_bwd():
    x = RNG.standard_normal((2, 3, 4, 4))
    y, c = L.gap_fwd(x)
    assert abs(y[1, 2] - sum(x[1, 2].ravel()) / 16) < 1e-12
    dy = RNG.standard_normal((2, 3))
    assert rel(L.gap_bwd(dy, c), fd_grad(lambda: float((L.gap_fwd(x)[0] * dy).sum()), x)) < 1e-7


# ---------------------------------------------------------------- attention, embedding

def attn_naive(qkv, h):
    b, t, d3 = qkv.shape
    d = d3 // 3; dh = d // h
    out = np.zeros((b, t, d))
    for bb in range(b):
        for hh in range(h):
            q = qkv[bb, :, hh * dh:(hh + 1) * dh]
            k = qkv[bb, :, d + hh * dh:d + (hh + 1) * dh]
            v = qkv[bb, :, 2 * d + hh * dh:2 * d + (hh + 1) * dh]
            for i in range(t):
                s = [float(q[i] @ k[j]) / math.sqrt(dh) for j in range(i + 1)]
                m = max(s)
                e = [math.exp(v_ - m) for v_ in s]
                z = sum(e)
                out[bb, i, hh * dh:(hh + 1) * dh] = sum((e[j] / z) * v[j] for j in range(i + 1))
    return out


def test_attention_matches_naive_causal_and_fd():
    qkv = RNG.standard_normal((2, 5, 3 * 8))
    out, c = L.attention_fwd(qkv, 2)
    assert np.allclose(out, attn_naive(qkv, 2), atol=1e-12)
    assert np.allclose(c[3].sum(-1), 1, atol=1e-12)
    # causality: changing the last token leaves earlier outputs bit-identical
    q2 = qkv.copy(); q2[:, 4, :] += 1.0
    out2, _ = L.attention_fwd(q2, 2)
    assert np.array_equal(out[:, :4], out2[:, :4])
    dout = RNG.standard_normal(out.shape)
    g = fd_grad(lambda: float((L.attention_fwd(qkv, 2)[0] * dout).sum()), qkv)
    assert rel(L.attention_bwd(dout, c), g) < 1e-6


def test_attention_single_token_returns_value():
    qkv = RNG.standard_normal((3, 1, 12))
    out, _ = L.attention_fwd(qkv, 2)
    assert np.allclose(out[:, 0], qkv[:, 0, 8:12], atol=1e-15)


def test_embedding_gradient_brute_force():
    ids = np.array([[1, 3, 1], [3, 3, 0]], dtype=np.int32)
    tok = RNG.standard_normal((6, 4)); pos = RNG.standard_normal((3, 4))
    h, c = L.embedding_fwd(ids, tok, pos)
    assert np.array_equal(h[1, 2], tok[0] + pos[2])
    dh = RNG.standard_normal(h.shape)
    dtok, dpos = L.embedding_bwd(dh, c)
    for r in range(6):
        exp = sum((dh[b, t] for b in range(2) for t in range(3) if ids[b, t] == r), np.zeros(4))
        assert np.allclose(dtok[r], exp, atol=1e-15)
    assert np.all(dtok[[2, 4, 5]] == 0)
    assert np.allclose(dpos, dh[0] + dh[1], atol=1e-15)


# ---------------------------------------------------------------- optimizers

def test_adam_first_step_and_zero_grad():
    w = RNG.standard_normal(6); g = RNG.standard_normal(6)
    st = {}
    w1 = O.adam_update(w, g, st, 1e-3, 0.9, 0.999, 1e-8)
    assert np.allclose(w1 - w, -1e-3 * g / (np.abs(g) + 1e-8), rtol=1e-9)
    st = {}
    assert np.array_equal(O.adam_update(w, np.zeros(6), st, 1e-3, 0.9, 0.999, 1e-8), w)


def test_adam_constant_gradient_n_steps():
    # constant gradient: bias-corrected m = g and v = g^2 at every step, so each step moves -lr*sign(g)
    w = np.zeros(3); g = np.array([0.5, -2.0, 1e-3]); st = {}
    for _ in range(7):
        w = O.adam_update(w, g, st, 1e-2, 0.9, 0.999, 0.0)
    assert np.allclose(w, -7e-2 * np.sign(g), rtol=1e-9)


def test_sgdm_closed_forms():
    w = RNG.standard_normal(5); g = RNG.standard_normal(5); st = {}
    w1 = O.sgdm_update(w, g, st, 0.1, 0.9, 5e-4, True)
    assert np.allclose(w1 - w, -0.1 * (g + 5e-4 * w), rtol=1e-12)
    st = {}
    w1 = O.sgdm_update(w, g, st, 0.1, 0.9, 5e-4, False)
    assert np.allclose(w1 - w, -0.1 * g, rtol=1e-12)
    # constant gradient, no decay: displacement after n steps = -lr*g*sum_{j<n} (1-mu^(j+1))/(1-mu)
    w = np.zeros(2); g = np.array([1.0, -3.0]); st = {}; n = 6; mu = 0.9
    for _ in range(n):
        w = O.sgdm_update(w, g, st, 0.01, mu, 0.0, True)
    geo = sum((1 - mu ** (j + 1)) / (1 - mu) for j in range(n))
    assert np.allclose(w, -0.01 * g * geo, rtol=1e-12)
