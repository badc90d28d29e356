"""Helpers of the GPU parity tests: drive the C-ABI library and the oracle on the same seeded
inputs and compare them tensor by tensor."""
from __future__ import annotations

import numpy as np
import torch

import lp_synth
from oracle.local_step import LocalUpdateOracle
from paper_2012_03837_b200 import binding as lp


def to_abi_layout(name: str, a: np.ndarray) -> np.ndarray:
    """Oracle layout -> library layout: convolution filters are [C_out, kh, kw, C_in] at the ABI."""
    if a.ndim == 4:
        return np.ascontiguousarray(a.transpose(0, 2, 3, 1))
    return np.ascontiguousarray(a)


class GpuModel:
    def __init__(self, cfg: dict, params: dict | None = None, gemm_backend: int = 0, ramp: str = "prime",
                 overlap: bool = False, fused: bool | None = None):
        self.cfg = cfg
        m, K, hd, op = lp.specs_from_config(cfg, gemm_backend)
        self._specs = (m, hd, op)
        self.K = K
        self.h = lp.lp_create(m, K, hd, op)
        self.index = {}
        for i in range(lp.lp_num_tensors(self.h)):
            info = lp.lp_tensor_info_get(self.h, i)
            self.index[info["name"]] = (i, info)
        self.dev = torch.device("cuda:0")
        self.losses = torch.zeros(K, dtype=torch.float32, device=self.dev)
        self.stream = torch.cuda.current_stream().cuda_stream
        self.set_params(params if params is not None else lp_synth.init_params(cfg))
        if ramp == "idle":
            lp.lp_set_ramp(self.h, lp.LP_RAMP_IDLE)
        if overlap:
            lp.lp_set_overlap(self.h, True)
        if fused is not None:                       # None: the library's default (single launch where available)
            lp.lp_set_fused_step(self.h, fused)

    def close(self):
        if self.h:
            lp.lp_destroy(self.h)
            self.h = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def set_params(self, params: dict):
        assert set(params) == set(self.index), (set(params) ^ set(self.index))
        for n, a in params.items():
            i, info = self.index[n]
            arr = to_abi_layout(n, np.asarray(a, dtype=np.float32))
            assert tuple(arr.shape) == tuple(info["shape"]), (n, arr.shape, info["shape"])
            lp.lp_set_tensor(self.h, i, lp.LP_MASTER, arr, self.stream)

    def get(self, which=lp.LP_MASTER) -> dict:
        out = {}
        for n, (i, info) in self.index.items():
            arr = np.empty(info["shape"], dtype=np.float32)
            lp.lp_get_tensor(self.h, i, which, arr, self.stream)
            if arr.ndim == 4:
                arr = np.ascontiguousarray(arr.transpose(0, 3, 1, 2))
            out[n] = arr
        return out

    def device_batch(self, x: np.ndarray, y: np.ndarray):
        if self.cfg["family"] == "lm":
            xt = torch.from_numpy(x).to(self.dev)
        else:
            xt = torch.from_numpy(x).to(self.dev)
            if self.cfg["dtype"] == "bf16":
                xt = xt.to(torch.bfloat16)
        return xt.contiguous(), torch.from_numpy(y).to(self.dev).contiguous()

    def step(self, x: np.ndarray, y: np.ndarray, schedule: str | None = None) -> np.ndarray:
        schedule = schedule or self.cfg["schedule"]
        xt, yt = self.device_batch(x, y)
        lp.lp_step(self.h, xt, yt, lp.LP_SYNC if schedule == "sync" else lp.LP_PIPELINED, self.stream, self.losses)
        torch.cuda.synchronize()
        lp.lp_status_poll(self.h, self.stream)
        return self.losses.cpu().numpy().astype(np.float64)

    def forward(self, x, y):
        xt, yt = self.device_batch(x, y)
        rows = lp_synth.units_per_step(self.cfg)
        classes = self.cfg["vocab"] if self.cfg["family"] == "lm" else self.cfg["classes"]
        dt = torch.bfloat16 if self.cfg["dtype"] == "bf16" else torch.float32
        logits = torch.empty(rows, classes, dtype=dt, device=self.dev)
        lp.lp_forward(self.h, xt, yt, self.stream, logits, self.losses)
        torch.cuda.synchronize()
        return logits.float().cpu().numpy(), self.losses.cpu().numpy().astype(np.float64)


def gpu_evaluate(gm: GpuModel, x, y, bn: str = "batch"):
    """lp_evaluate on (x, y): (losses [K], correct [K], predictions [K, rows])."""
    xt, yt = gm.device_batch(x, y)
    rows = lp_synth.units_per_step(gm.cfg)
    correct = torch.full((gm.K,), -1, dtype=torch.int32, device=gm.dev)
    pred = torch.full((gm.K, rows), -1, dtype=torch.int32, device=gm.dev)
    lp.lp_evaluate(gm.h, xt, yt, gm.stream, gm.losses, correct, pred,
                   lp.LP_BN_RUNNING if bn == "running" else lp.LP_BN_BATCH)
    torch.cuda.synchronize()
    lp.lp_status_poll(gm.h, gm.stream)
    return gm.losses.cpu().numpy().astype(np.float64), correct.cpu().numpy(), pred.cpu().numpy()


def tensor_rel_err(a: np.ndarray, b: np.ndarray) -> float:
    """max |a - b| / max |b| over one tensor (the oracle's tensor is b)."""
    return float(np.abs(a.astype(np.float64) - b.astype(np.float64)).max() / max(np.abs(b).max(), 1e-30))


def run_both(cfg: dict, steps: int, gemm_backend: int = 0, params: dict | None = None, ramp: str = "prime",
             overlap: bool = False, fused: bool | None = None):
    """Run `steps` steps on both sides.  Returns (gpu_losses [steps,K], oracle_losses, gpu model, oracle)."""
    params = params if params is not None else lp_synth.init_params(cfg)
    gm = GpuModel(cfg, params, gemm_backend, ramp, overlap, fused)
    orc = LocalUpdateOracle(cfg, params, dtype=np.float32, ramp=ramp, overlap=overlap)
    gl, ol = [], []
    for t in range(steps):
        x, y = lp_synth.minibatch(cfg, t)
        gl.append(gm.step(x, y))
        ol.append(orc.step(x, y))
    return np.array(gl), np.array(ol), gm, orc


def strip_key_bias(name: str, a: np.ndarray) -> np.ndarray:
    """Drop the key third of a fused q/k/v bias.  Adding a constant to every key of a head shifts
    all scores of a query row equally and softmax ignores it, so that gradient is identically zero;
    what either implementation stores there is rounding noise, which Adam turns into +-lr steps."""
    if name.endswith(".bqkv"):
        d = a.shape[0] // 3
        return np.concatenate([a[:d], a[2 * d:]])
    return a


def compare_weights(gm: GpuModel, orc: LocalUpdateOracle, init: dict) -> dict:
    """Per tensor: (kind, error).  Matrices: ||a-b||_2 / ||b||_2.  Vectors (biases, norm scales and
    shifts: they start at 0 or 1, so their value after a few steps IS the accumulated update):
    ||a-b||_2 / ||b - init||_2.  Also "chunk<k>": the relative l2 error of all of chunk k's parameters."""
    got = gm.get(lp.LP_MASTER)
    out = {}
    per_chunk = {}
    for n in got:
        a = strip_key_bias(n, got[n].astype(np.float64))
        b = strip_key_bias(n, orc.p[n].astype(np.float64))
        i0 = strip_key_bias(n, np.asarray(init[n], dtype=np.float64))
        e = np.linalg.norm(a - b)
        if got[n].ndim >= 2:
            out[n] = ("matrix", e / max(np.linalg.norm(b), 1e-30))
        else:
            out[n] = ("vector", e / max(np.linalg.norm(b - i0), 1e-30))
        k = gm.index[n][1]["chunk"]
        se, sb = per_chunk.get(k, (0.0, 0.0))
        per_chunk[k] = (se + e * e, sb + float((b * b).sum()))
    for k, (se, sb) in per_chunk.items():
        out[f"chunk{k}"] = ("chunk", float(np.sqrt(se / sb)))
    return out
