"""CPU oracle, layer definitions: forward and hand-derived backward of every layer the local
update step needs.  TEST INFRASTRUCTURE ONLY: slow, plain NumPy, no blocking or fusion; it shares
no code with the CUDA path and must never be imported by the product.

The paper fixes the architectures only by size (App. A.1: an MLP layer is a matrix-vector
product, a bias add and a ReLU, and its auxiliary classifier a matrix-vector product, a bias add
and a softmax cross-entropy; App. B.2: transformer layers with an auxiliary LayerNorm + vocabulary
projection; App. B.3: ResNet blocks with BatchNorm), so every function below is the textbook
definition of that layer.  Each backward is checked against central finite differences and against
an independent reverse-mode differentiation in the CPU tests.

Every forward returns (output, cache); every backward takes (upstream gradient, cache) and returns
the gradients in the order (input, parameters...).
"""
from __future__ import annotations

import numpy as np
from scipy.special import erf


# ------------------------------------------------------------------ dense layers (App. A.1)

def linear_fwd(x, W, b):
    """y[r, o] = sum_i x[r, i] W[o, i] + b[o]."""
    return x @ W.T + b, (x, W)


def linear_bwd(dy, cache):
    x, W = cache
    dx = dy @ W
    dW = dy.T @ x
    db = dy.sum(axis=0)
    return dx, dW, db


def relu_fwd(x):
    y = np.maximum(x, 0)
    return y, (y,)


def relu_bwd(dy, cache):
    (y,) = cache
    return dy * (y > 0)


def gelu_fwd(x):
    """Exact GELU: x * Phi(x) with Phi the standard normal CDF."""
    y = 0.5 * x * (1.0 + erf(x / np.sqrt(2.0)))
    return y.astype(x.dtype), (x,)


def gelu_bwd(dy, cache):
    (x,) = cache
    cdf = 0.5 * (1.0 + erf(x / np.sqrt(2.0)))
    pdf = np.exp(-0.5 * x * x) / np.sqrt(2.0 * np.pi)
    return (dy * (cdf + x * pdf)).astype(x.dtype)


# ------------------------------------------------------------------ normalisation

def layernorm_fwd(x, g, b, eps=1e-5):
    """Normalise each row over its last axis (biased variance), then scale and shift."""
    mu = x.mean(axis=-1, keepdims=True)
    var = ((x - mu) ** 2).mean(axis=-1, keepdims=True)
    rstd = 1.0 / np.sqrt(var + eps)
    xhat = (x - mu) * rstd
    return xhat * g + b, (xhat, rstd, g)


def layernorm_bwd(dy, cache):
    xhat, rstd, g = cache
    dxhat = dy * g
    m1 = dxhat.mean(axis=-1, keepdims=True)
    m2 = (dxhat * xhat).mean(axis=-1, keepdims=True)
    dx = rstd * (dxhat - m1 - xhat * m2)
    red = tuple(range(dy.ndim - 1))
    dg = (dy * xhat).sum(axis=red)
    db = dy.sum(axis=red)
    return dx, dg, db


def batchnorm_fwd(x, g, b, eps=1e-5):
    """Train-mode BatchNorm over [N, C, H, W]: per-channel batch mean and biased variance."""
    mu = x.mean(axis=(0, 2, 3), keepdims=True)
    var = ((x - mu) ** 2).mean(axis=(0, 2, 3), keepdims=True)
    rstd = 1.0 / np.sqrt(var + eps)
    xhat = (x - mu) * rstd
    y = xhat * g.reshape(1, -1, 1, 1) + b.reshape(1, -1, 1, 1)
    return y, (xhat, rstd, g, mu.reshape(-1), var.reshape(-1))


def batchnorm_running_update(run_mean, run_var, cache, n, momentum=0.1):
    """Running statistics after a train-mode pass over n values per channel: exponential averages of the
    batch mean and of the unbiased batch variance (n / (n - 1) times the biased one)."""
    mu, var = cache[3], cache[4]
    unbiased = var * (n / max(n - 1, 1))
    return (1 - momentum) * run_mean + momentum * mu, (1 - momentum) * run_var + momentum * unbiased


def batchnorm_eval(x, g, b, run_mean, run_var, eps=1e-5):
    """Evaluation-mode BatchNorm over [N, C, H, W]: normalises with the running statistics."""
    sh = (1, -1, 1, 1)
    return (x - run_mean.reshape(sh)) / np.sqrt(run_var.reshape(sh) + eps) * g.reshape(sh) + b.reshape(sh)


def batchnorm_bwd(dy, cache):
    xhat, rstd, g = cache[:3]
    dxhat = dy * g.reshape(1, -1, 1, 1)
    m1 = dxhat.mean(axis=(0, 2, 3), keepdims=True)
    m2 = (dxhat * xhat).mean(axis=(0, 2, 3), keepdims=True)
    dx = rstd * (dxhat - m1 - xhat * m2)
    dg = (dy * xhat).sum(axis=(0, 2, 3))
    db = dy.sum(axis=(0, 2, 3))
    return dx, dg, db


# ------------------------------------------------------------------ convolution

def _im2col(x, kh, kw, stride, pad):
    n, c, h, w = x.shape
    ho = (h + 2 * pad - kh) // stride + 1
    wo = (w + 2 * pad - kw) // stride + 1
    xp = np.pad(x, ((0, 0), (0, 0), (pad, pad), (pad, pad)))
    cols = np.empty((n, ho, wo, c, kh, kw), dtype=x.dtype)
    for i in range(kh):
        for j in range(kw):
            cols[:, :, :, :, i, j] = xp[:, :, i:i + stride * ho:stride, j:j + stride * wo:stride].transpose(0, 2, 3, 1)
    return cols.reshape(n * ho * wo, c * kh * kw), ho, wo


def conv2d_fwd(x, W, stride, pad):
    """Cross-correlation without bias: y[n,o,p,q] = sum_{c,i,j} x[n,c,p*s+i-pad,q*s+j-pad] W[o,c,i,j]."""
    o, c, kh, kw = W.shape
    cols, ho, wo = _im2col(x, kh, kw, stride, pad)
    y = cols @ W.reshape(o, -1).T
    y = y.reshape(x.shape[0], ho, wo, o).transpose(0, 3, 1, 2)
    return np.ascontiguousarray(y), (cols, x.shape, W, stride, pad, ho, wo)


def conv2d_bwd(dy, cache):
    cols, xshape, W, stride, pad, ho, wo = cache
    o, c, kh, kw = W.shape
    n, _, h, w = xshape
    dy2 = dy.transpose(0, 2, 3, 1).reshape(-1, o)
    dW = (dy2.T @ cols).reshape(W.shape)
    dcols = (dy2 @ W.reshape(o, -1)).reshape(n, ho, wo, c, kh, kw)
    dxp = np.zeros((n, c, h + 2 * pad, w + 2 * pad), dtype=dy.dtype)
    for i in range(kh):
        for j in range(kw):
            dxp[:, :, i:i + stride * ho:stride, j:j + stride * wo:stride] += dcols[:, :, :, :, i, j].transpose(0, 3, 1, 2)
    dx = dxp[:, :, pad:pad + h, pad:pad + w]
    return np.ascontiguousarray(dx), dW


def gap_fwd(x):
    """Global average pool over H and W: [N, C, H, W] -> [N, C]."""
    return x.mean(axis=(2, 3)), (x.shape,)


def gap_bwd(dy, cache):
    (shape,) = cache
    n, c, h, w = shape
    return np.broadcast_to(dy.reshape(n, c, 1, 1) / (h * w), shape).astype(dy.dtype)


# ------------------------------------------------------------------ attention and embeddings

def attention_fwd(qkv, n_heads):
    """Causal multi-head softmax attention.  qkv is [B, T, 3d]: columns [0,d) are the queries,
    [d,2d) the keys, [2d,3d) the values, each split into n_heads consecutive groups of d/n_heads.
    Position t attends to positions <= t; scores are scaled by 1/sqrt(d/n_heads)."""
    b, t, d3 = qkv.shape
    d = d3 // 3
    dh = d // n_heads
    q, k, v = (qkv[:, :, i * d:(i + 1) * d].reshape(b, t, n_heads, dh).transpose(0, 2, 1, 3) for i in range(3))
    scale = 1.0 / np.sqrt(dh)
    s = (q @ k.transpose(0, 1, 3, 2)) * scale
    mask = np.triu(np.ones((t, t), dtype=bool), 1)
    s = np.where(mask, -np.inf, s)
    s = s - s.max(axis=-1, keepdims=True)
    p = np.exp(s)
    p = p / p.sum(axis=-1, keepdims=True)
    o = p @ v
    out = o.transpose(0, 2, 1, 3).reshape(b, t, d)
    return out.astype(qkv.dtype), (q, k, v, p.astype(qkv.dtype), scale)


def attention_bwd(dout, cache):
    q, k, v, p, scale = cache
    b, h, t, dh = q.shape
    do = dout.reshape(b, t, h, dh).transpose(0, 2, 1, 3)
    dv = p.transpose(0, 1, 3, 2) @ do
    dp = do @ v.transpose(0, 1, 3, 2)
    ds = p * (dp - (dp * p).sum(axis=-1, keepdims=True))
    dq = (ds @ k) * scale
    dk = (ds.transpose(0, 1, 3, 2) @ q) * scale
    parts = [g.transpose(0, 2, 1, 3).reshape(b, t, h * dh) for g in (dq, dk, dv)]
    return np.concatenate(parts, axis=-1).astype(dout.dtype)


def embedding_fwd(ids, tok, pos):
    """h[b, t] = tok[ids[b, t]] + pos[t]."""
    return tok[ids] + pos[None, :ids.shape[1], :], (ids, tok.shape, pos.shape)


def embedding_bwd(dh, cache):
    ids, tshape, pshape = cache
    dtok = np.zeros(tshape, dtype=dh.dtype)
    np.add.at(dtok, ids.reshape(-1), dh.reshape(-1, dh.shape[-1]))
    dpos = np.zeros(pshape, dtype=dh.dtype)
    dpos[:ids.shape[1]] = dh.sum(axis=0)
    return dtok, dpos


# ------------------------------------------------------------------ loss (App. A.1, App. B.2)

def softmax_xent(z, y):
    """Mean softmax cross-entropy over the rows whose label is >= 0, and its gradient.

    z: [R, C] logits; y: [R] integer labels, -1 = ignore.  Returns (loss, dz) with
    loss = (1/R_valid) sum_r (logsumexp(z_r) - z_r[y_r]) and dz_r = (softmax(z_r) - onehot(y_r)) / R_valid
    on valid rows, zero on ignored rows.
    """
    valid = y >= 0
    n_valid = int(valid.sum())
    m = z.max(axis=1, keepdims=True)
    e = np.exp(z - m)
    se = e.sum(axis=1, keepdims=True)
    lse = (m + np.log(se)).reshape(-1)
    rows = np.arange(z.shape[0])
    ysafe = np.where(valid, y, 0)
    row_loss = np.where(valid, lse - z[rows, ysafe], 0)
    loss = row_loss.sum(dtype=np.float64) / n_valid
    dz = e / se
    dz[rows, ysafe] -= 1
    dz = dz * (valid.reshape(-1, 1) / z.dtype.type(n_valid))
    return z.dtype.type(loss), dz.astype(z.dtype)
