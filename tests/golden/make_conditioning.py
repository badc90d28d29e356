"""Writes tests/golden/c2_conditioning.json and c4_conditioning.json: how far apart two correct evaluations
of a workload drift over its first ten steps.

The wide-MLP workload c2 (K = 8 chunks of two 2048-wide Linear+ReLU layers, pipelined schedule, Adam with
lr 1e-3) amplifies rounding: Adam's normalised step moves a weight by about +-lr whatever the size of its
gradient, so a gradient element whose sign depends on the last bits turns a 1e-7 difference into a 2e-3 one,
and the difference is handed down the pipeline (Sec. 6) to every later chunk.  The ResNet workload c4 (SGD with
lr 0.1 and momentum 0.9, BatchNorm centring every ReLU input at zero) moves its small head matrices by a
multiple of their initial norm within ten steps, so a few percent of gradient error show up in them directly.
This script measures both with the CPU oracle alone, per step t = 1..10 and per chunk:

  fp32_vs_fp64     (c2) the oracle in fp32 against the oracle in fp64 (same inputs, same algorithm);
  bf16io_vs_fp32   the fp32 oracle that keeps fp32 master weights but uses weight matrices rounded to bf16 in
                   its forward and backward passes and rounds every layer's stored output (activations forward,
                   input gradients backward) to bf16 -- the storage formats of the bf16 workloads, with fp32
                   arithmetic inside every layer and nothing else changed -- against the plain fp32 oracle;
  bf16out_vs_fp32  (c2) the fp32 oracle with only its chunk outputs rounded to bf16, against the plain fp32 oracle:
                   a second realisation of such a perturbation (the size of a loss transient differs between
                   realisations by more than a factor of two).

Each entry holds the relative loss gap |a-b|/|b|, the largest relative l2 gap over the chunk's weight matrices
and the largest gap of its vectors relative to their accumulated update.  The GPU parity tests of the full-size
workloads take their bounds from these files.  Only oracle/ and the seeded generators are used; run from the
repository root:  python tests/golden/make_conditioning.py [c2|c4]
"""
import json
import os
import sys

import numpy as np

ROOT = os.path.dirname(os.path.dirname(os.path.dirname(os.path.abspath(__file__))))
sys.path.insert(0, ROOT)
import lp_synth  # noqa: E402
from oracle.local_step import LocalUpdateOracle  # noqa: E402


import oracle.layers as L  # noqa: E402

# Layers whose output the bf16 workloads store in bf16 (R10 of the design notes: bf16 activations between kernels,
# fp32 accumulation inside a layer, fp32 statistics and loss).  While ROUNDING is set, the first result of each of
# these functions -- a forward output, or the gradient with respect to the layer input -- is rounded to bf16 (ties
# to even) as the witness stores it; parameter gradients, caches and everything else stay fp32.  The oracle
# itself is not changed: the wrappers are installed by this script only, and do nothing for the plain oracles.
ROUNDING = False
_STORED = ("linear_fwd", "linear_bwd", "relu_fwd", "relu_bwd", "gelu_fwd", "gelu_bwd", "layernorm_fwd", "layernorm_bwd",
           "batchnorm_fwd", "batchnorm_eval", "batchnorm_bwd", "conv2d_fwd", "conv2d_bwd", "gap_fwd", "gap_bwd",
           "attention_fwd", "attention_bwd", "embedding_fwd")


def _stored_in_bf16(fn):
    def wrapped(*a, **k):
        out = fn(*a, **k)
        if not ROUNDING:
            return out
        if isinstance(out, tuple):
            return (lp_synth.bf16_round(out[0]),) + out[1:]
        return lp_synth.bf16_round(out)
    return wrapped


for _name in _STORED:
    setattr(L, _name, _stored_in_bf16(getattr(L, _name)))


class Bf16OutputOracle(LocalUpdateOracle):
    """The fp32 oracle with nothing but its chunk outputs rounded to bf16 (head and next chunk read the rounded
    value): a second realisation of a storage-format perturbation, for the spread between realisations."""

    def chunk_forward(self, k, inp):
        h, cache = super().chunk_forward(k, inp)
        return lp_synth.bf16_round(h), cache


class Bf16StorageOracle(LocalUpdateOracle):
    """The fp32 oracle with bf16 storage of what the bf16 workloads store in bf16: the weight matrices as the
    forward and backward passes read them (the fp32 masters are what the optimizer updates) and every layer's
    output activation and input gradient."""

    def _as_stored(self, k, fn):
        global ROUNDING
        saved = {n: self.p[n] for n in self.names_of_chunk[k] if self.p[n].ndim >= 2}
        for n, a in saved.items():
            self.p[n] = lp_synth.bf16_round(a)
        ROUNDING = True
        try:
            return fn()
        finally:
            ROUNDING = False
            self.p.update(saved)

    def chunk_forward(self, k, inp):
        if ROUNDING:                                         # called from within local_grads
            return super().chunk_forward(k, inp)
        return self._as_stored(k, lambda: super(Bf16StorageOracle, self).chunk_forward(k, inp))

    def local_grads(self, k, inp, y):
        return self._as_stored(k, lambda: super(Bf16StorageOracle, self).local_grads(k, inp, y))


def gaps(a, b, init):
    mats, vecs = [], []
    for k in range(a.K):
        wm = wv = 0.0
        for n in a.names_of_chunk[k]:
            if n in a.buffers:
                continue
            x, y = a.p[n].astype(np.float64), b.p[n].astype(np.float64)
            e = float(np.linalg.norm(x - y))
            if x.ndim >= 2:
                wm = max(wm, e / float(np.linalg.norm(y)))
            else:
                wv = max(wv, e / max(float(np.linalg.norm(y - init[n])), 1e-30))
        mats.append(wm)
        vecs.append(wv)
    return mats, vecs


def run(name, steps=10):
    cfg = lp_synth.config(name)
    params = lp_synth.init_params(cfg)
    o32 = LocalUpdateOracle(cfg, params, dtype=np.float32)
    ob = Bf16StorageOracle(cfg, params, dtype=np.float32)
    o64 = LocalUpdateOracle(cfg, params, dtype=np.float64) if name == "c2" else None
    oo = Bf16OutputOracle(cfg, params, dtype=np.float32) if name == "c2" else None
    rec = []
    for t in range(steps):
        x, y = lp_synth.minibatch(cfg, t)
        l32, lb = o32.step(x, y), ob.step(x, y)
        m, v = gaps(ob, o32, params)
        r = dict(step=t + 1, bf16io_vs_fp32=dict(loss=[float(abs(a - b) / abs(b)) for a, b in zip(lb, l32)], weights=m, vectors=v))
        if o64 is not None:
            l64, lo = o64.step(x, y), oo.step(x, y)
            m, v = gaps(o32, o64, params)
            r["fp32_vs_fp64"] = dict(loss=[float(abs(a - b) / abs(b)) for a, b in zip(l32, l64)], weights=m, vectors=v)
            m, v = gaps(oo, o32, params)
            r["bf16out_vs_fp32"] = dict(loss=[float(abs(a - b) / abs(b)) for a, b in zip(lo, l32)], weights=m, vectors=v)
        rec.append(r)
        print(name, json.dumps(r), flush=True)
    return rec


if __name__ == "__main__":
    for name in (sys.argv[1:] or ["c2", "c4"]):
        rec = run(name)
        with open(os.path.join(os.path.dirname(os.path.abspath(__file__)), f"{name}_conditioning.json"), "w") as f:
            json.dump(dict(workload=name, steps=rec), f, indent=1)
