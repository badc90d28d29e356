"""CPU oracle, optimizers.  TEST INFRASTRUCTURE ONLY (see oracle/layers.py).

Each chunk's parameters are updated from that chunk's own gradients (Sec. 1: with local updates a
layer is updated before the forward pass through the rest of the network completes; Sec. 6: the
updates can be applied asynchronously).  The paper trains with Adam and with SGD with momentum
(App. B.1-B.3) and gives no formula, so these are the standard definitions.
"""
from __future__ import annotations

import numpy as np


def sgdm_update(w, g, state, lr, momentum, weight_decay, decay):
    """g' = g + wd*w (only where `decay`), v <- mu*v + g', w <- w - lr*v.  No Nesterov, no dampening."""
    if decay and weight_decay != 0.0:
        g = g + w.dtype.type(weight_decay) * w
    v = state.get("v")
    v = g.copy() if v is None else w.dtype.type(momentum) * v + g
    state["v"] = v
    return w - w.dtype.type(lr) * v


def adam_update(w, g, state, lr, beta1, beta2, eps):
    """m <- b1 m + (1-b1) g; v <- b2 v + (1-b2) g^2; w <- w - lr * (m/(1-b1^t)) / (sqrt(v/(1-b2^t)) + eps), t from 1."""
    T = w.dtype.type
    t = state.get("t", 0) + 1
    m = state.get("m", np.zeros_like(w))
    v = state.get("v", np.zeros_like(w))
    m = T(beta1) * m + T(1.0 - beta1) * g
    v = T(beta2) * v + T(1.0 - beta2) * g * g
    state.update(t=t, m=m, v=v)
    mhat = m / T(1.0 - beta1 ** t)
    vhat = v / T(1.0 - beta2 ** t)
    return w - T(lr) * mhat / (np.sqrt(vhat) + T(eps))
