"""Seeded synthetic workloads for the local-update step (shared by the CPU oracle's tests
and by the CUDA path's tests and benchmark).

This module holds no arithmetic of the method: it names the five workloads, enumerates the
parameter tensors of a model (name, shape, initialiser), and draws inputs, labels and initial
weights from counter-based NumPy streams.  Nothing here computes a forward pass, a loss, a
gradient or an update.

The inputs stand in for the data sets the paper trains on (Sec. 4.1: CIFAR-10 vectors for the
MLPs; Sec. 4.2 / App. B.2: LM1B sub-word ids with 8k and 32k vocabularies; Sec. 4.3 / App. B.3:
image batches for ResNets): they take the shapes, class counts and value ranges of those
workloads and nothing else.
"""
from __future__ import annotations

import copy
import zlib

import numpy as np

# ----------------------------------------------------------------------------- workloads

_BASE = {
    # MLP, fp32, K=4, synchronous, SGD-momentum.
    "c1": dict(
        family="mlp", dtype="fp32", batch=64, d_in=256, chunks=[[256], [256], [256], [256]],
        classes=10, schedule="sync",
        optim=dict(kind="sgdm", lr=0.01, momentum=0.9, weight_decay=0.0), steps=10, seed=0,
    ),
    # Wide MLP, bf16 with fp32 master weights, K=8, pipelined, Adam.
    "c2": dict(
        family="mlp", dtype="bf16", batch=1024, d_in=1024, chunks=[[2048, 2048]] * 8,
        classes=1000, schedule="pipelined",
        optim=dict(kind="adam", lr=1e-3, beta1=0.9, beta2=0.999, eps=1e-8), steps=20, seed=0,
    ),
    # Decoder-only transformer LM, bf16, K=8 (one block per chunk), synchronous, Adam.
    "c3": dict(
        family="lm", dtype="bf16", batch=32, seq_len=256, vocab=8192, d_model=512, n_heads=8,
        d_ffn=2048, blocks_per_chunk=[1] * 8, schedule="sync",
        optim=dict(kind="adam", lr=3e-4, beta1=0.9, beta2=0.999, eps=1e-8), steps=10, seed=0,
    ),
    # ResNet-18-shaped convnet, bf16, K=4 stages, SGD-momentum with weight decay.
    "c4": dict(
        family="resnet", dtype="bf16", batch=256, in_channels=3, height=32, width=32,
        stem_channels=64, stage_channels=[64, 128, 256, 512], blocks_per_stage=2, classes=10,
        schedule="sync",
        optim=dict(kind="sgdm", lr=0.1, momentum=0.9, weight_decay=5e-4), steps=10, seed=0,
    ),
    # Large decoder-only transformer LM, bf16, K=24, pipelined, Adam.
    "c5": dict(
        family="lm", dtype="bf16", batch=16, seq_len=512, vocab=32768, d_model=1024,
        n_heads=16, d_ffn=4096, blocks_per_chunk=[1] * 24, schedule="pipelined",
        optim=dict(kind="adam", lr=2e-4, beta1=0.9, beta2=0.999, eps=1e-8), steps=50, seed=0,
    ),
}


def config(name: str, **overrides) -> dict:
    """Return a deep copy of workload `name` ("c1".."c5") with top-level keys overridden."""
    cfg = copy.deepcopy(_BASE[name])
    cfg["name"] = name
    for k, v in overrides.items():
        if k == "optim":
            cfg["optim"].update(v)
        else:
            cfg[k] = copy.deepcopy(v)
    return cfg


def num_chunks(cfg: dict) -> int:
    if cfg["family"] == "mlp":
        return len(cfg["chunks"])
    if cfg["family"] == "lm":
        return len(cfg["blocks_per_chunk"])
    return len(cfg["stage_channels"])


def units_per_step(cfg: dict) -> int:
    """Samples (MLP, ResNet) or tokens (LM) one step consumes."""
    if cfg["family"] == "lm":
        return cfg["batch"] * cfg["seq_len"]
    return cfg["batch"]


# ----------------------------------------------------------------------------- bf16 helper

def bf16_round(a: np.ndarray) -> np.ndarray:
    """Round fp32 values to the nearest bfloat16 (ties to even), returned as fp32."""
    a = np.ascontiguousarray(a, dtype=np.float32)
    u = a.view(np.uint32).astype(np.uint64)
    u = (u + 0x7FFF + ((u >> 16) & 1)) & 0xFFFF0000
    return u.astype(np.uint32).view(np.float32).reshape(a.shape)


def to_bf16_bits(a: np.ndarray) -> np.ndarray:
    """fp32 -> uint16 bfloat16 bit patterns (round to nearest even)."""
    return (bf16_round(a).view(np.uint32) >> 16).astype(np.uint16)


def from_bf16_bits(b: np.ndarray) -> np.ndarray:
    """uint16 bfloat16 bit patterns -> fp32."""
    return (np.asarray(b, dtype=np.uint16).astype(np.uint32) << 16).view(np.float32)


# ----------------------------------------------------------------------------- parameter table

def param_table(cfg: dict) -> list[dict]:
    """Ordered list of parameter tensors: name, chunk, shape, init ("normal" std / "zeros" /
    "ones"), and whether weight decay applies (matrices and filters only).

    Layouts: Linear weights are [out, in]; convolution filters are [C_out, C_in, kh, kw];
    embedding tables are [rows, d_model].  Entries marked buffer=True are state that no gradient
    reaches (BatchNorm running mean ".rm" and variance ".rv"); they come last so that the other
    tensors keep their random streams.
    """
    fam = cfg["family"]
    out: list[dict] = []

    def add(name, chunk, shape, init, std=0.0, decay=False, buffer=False):
        out.append(dict(name=name, chunk=chunk, shape=tuple(int(s) for s in shape), init=init,
                        std=float(std), decay=bool(decay), buffer=bool(buffer)))

    if fam == "mlp":
        d_prev = cfg["d_in"]
        for k, widths in enumerate(cfg["chunks"]):
            for i, w in enumerate(widths):
                add(f"c{k}.l{i}.W", k, (w, d_prev), "normal", np.sqrt(2.0 / d_prev), True)
                add(f"c{k}.l{i}.b", k, (w,), "zeros")
                d_prev = w
            add(f"c{k}.head.W", k, (cfg["classes"], d_prev), "normal", np.sqrt(1.0 / d_prev), True)
            add(f"c{k}.head.b", k, (cfg["classes"],), "zeros")
    elif fam == "lm":
        d, f, v, t = cfg["d_model"], cfg["d_ffn"], cfg["vocab"], cfg["seq_len"]
        s = 0.02
        blk = 0
        for k, nb in enumerate(cfg["blocks_per_chunk"]):
            if k == 0 and not cfg.get("input_is_activation"):
                add("c0.tok", 0, (v, d), "normal", s, True)
                add("c0.pos", 0, (t, d), "normal", s, True)
            for _ in range(nb):
                p = f"c{k}.b{blk}"
                add(p + ".ln1.g", k, (d,), "ones")
                add(p + ".ln1.b", k, (d,), "zeros")
                add(p + ".Wqkv", k, (3 * d, d), "normal", s, True)
                add(p + ".bqkv", k, (3 * d,), "zeros")
                add(p + ".Wo", k, (d, d), "normal", s, True)
                add(p + ".bo", k, (d,), "zeros")
                add(p + ".ln2.g", k, (d,), "ones")
                add(p + ".ln2.b", k, (d,), "zeros")
                add(p + ".W1", k, (f, d), "normal", s, True)
                add(p + ".b1", k, (f,), "zeros")
                add(p + ".W2", k, (d, f), "normal", s, True)
                add(p + ".b2", k, (d,), "zeros")
                blk += 1
            add(f"c{k}.head.ln.g", k, (d,), "ones")
            add(f"c{k}.head.ln.b", k, (d,), "zeros")
            add(f"c{k}.head.W", k, (v, d), "normal", s, True)
            add(f"c{k}.head.b", k, (v,), "zeros")
    elif fam == "resnet":
        cin = cfg["in_channels"]
        inner = bool(cfg.get("input_is_activation"))     # a later stage on its own: no stem, input = activation
        c_prev = cin if inner else cfg["stem_channels"]
        for k, c in enumerate(cfg["stage_channels"]):
            if k == 0 and not inner:
                add("c0.stem.conv", 0, (c_prev, cin, 3, 3), "normal", np.sqrt(2.0 / (cin * 9)), True)
                add("c0.stem.bn.g", 0, (c_prev,), "ones")
                add("c0.stem.bn.b", 0, (c_prev,), "zeros")
            bottleneck = cfg.get("block") == "bottleneck"
            c_out = 4 * c if bottleneck else c           # a bottleneck block leaves four times its inner width
            for j in range(resnet_stage_blocks(cfg, k)):
                p = f"c{k}.r{j}"
                c_in_blk = c_prev if j == 0 else c_out
                if bottleneck:
                    add(p + ".conv1", k, (c, c_in_blk, 1, 1), "normal", np.sqrt(2.0 / c_in_blk), True)
                    add(p + ".bn1.g", k, (c,), "ones")
                    add(p + ".bn1.b", k, (c,), "zeros")
                    add(p + ".conv2", k, (c, c, 3, 3), "normal", np.sqrt(2.0 / (c * 9)), True)
                    add(p + ".bn2.g", k, (c,), "ones")
                    add(p + ".bn2.b", k, (c,), "zeros")
                    add(p + ".conv3", k, (c_out, c, 1, 1), "normal", np.sqrt(2.0 / c), True)
                    add(p + ".bn3.g", k, (c_out,), "ones")
                    add(p + ".bn3.b", k, (c_out,), "zeros")
                else:
                    add(p + ".conv1", k, (c, c_in_blk, 3, 3), "normal", np.sqrt(2.0 / (c_in_blk * 9)), True)
                    add(p + ".bn1.g", k, (c,), "ones")
                    add(p + ".bn1.b", k, (c,), "zeros")
                    add(p + ".conv2", k, (c, c, 3, 3), "normal", np.sqrt(2.0 / (c * 9)), True)
                    add(p + ".bn2.g", k, (c,), "ones")
                    add(p + ".bn2.b", k, (c,), "zeros")
                if j == 0 and (resnet_stage_stride(cfg, k) != 1 or c_in_blk != c_out):
                    add(p + ".sc.conv", k, (c_out, c_in_blk, 1, 1), "normal", np.sqrt(2.0 / c_in_blk), True)
                    add(p + ".sc.bn.g", k, (c_out,), "ones")
                    add(p + ".sc.bn.b", k, (c_out,), "zeros")
            c = c_out
            c_prev = c
            add(f"c{k}.head.W", k, (cfg["classes"], c), "normal", np.sqrt(1.0 / c), True)
            add(f"c{k}.head.b", k, (cfg["classes"],), "zeros")
            if cfg.get("head") == "bn_relu_gap":
                add(f"c{k}.head.bn.g", k, (c,), "ones")
                add(f"c{k}.head.bn.b", k, (c,), "zeros")
        for t in [t for t in out if t["name"].endswith(".g") and ".bn" in t["name"]]:
            stem = t["name"][:-2]
            add(stem + ".rm", t["chunk"], t["shape"], "zeros", buffer=True)
            add(stem + ".rv", t["chunk"], t["shape"], "ones", buffer=True)
    else:
        raise ValueError(fam)
    return out


def resnet_stage_blocks(cfg: dict, k: int) -> int:
    """Residual blocks in stage k: cfg["blocks_per_stage"] is one count for all stages or a list per stage
    (a ResNet-50 has 3, 4, 6, 3)."""
    n = cfg["blocks_per_stage"]
    return int(n[k]) if isinstance(n, (list, tuple)) else int(n)


def resnet_stage_stride(cfg: dict, k: int) -> int:
    """Stride of the first convolution of stage k: 1 for the network's first stage, 2 afterwards."""
    return 1 if (k == 0 and not cfg.get("input_is_activation")) else 2


# ----------------------------------------------------------------------------- random streams

def _rng(seed: int, *key) -> np.random.Generator:
    """Independent PCG64 stream for (seed, key...); string keys are hashed with CRC-32."""
    ints = [int(seed)]
    for k in key:
        ints.append(zlib.crc32(k.encode()) if isinstance(k, str) else int(k))
    return np.random.Generator(np.random.PCG64(np.random.SeedSequence(ints)))


def init_params(cfg: dict) -> dict[str, np.ndarray]:
    """Initial parameters as fp32 arrays keyed by name.  For bf16 workloads the values are
    already rounded to bfloat16, so both implementations start from the same bits."""
    params = {}
    for i, t in enumerate(param_table(cfg)):
        if t["init"] == "normal":
            a = _rng(cfg["seed"], "w", i).standard_normal(t["shape"], dtype=np.float32) * np.float32(t["std"])
        elif t["init"] == "ones":
            a = np.ones(t["shape"], np.float32)
        else:
            a = np.zeros(t["shape"], np.float32)
        if cfg["dtype"] == "bf16":
            a = bf16_round(a)
        params[t["name"]] = a.astype(np.float32)
    return params


def minibatch(cfg: dict, t: int) -> tuple[np.ndarray, np.ndarray]:
    """Minibatch of step t: (x, y).

    MLP: x fp32 [B, d_in] ~ N(0,1) (bf16-rounded for bf16 workloads), y int32 [B] uniform classes.
    LM: x int32 ids [B, T] uniform over the vocabulary; y int32 [B, T] = ids shifted left by one,
        last position -1 (ignored by the loss).
    ResNet: x fp32 [B, C, H, W] ~ N(0,1) (bf16-rounded), y int32 [B].
    """
    g = _rng(cfg["seed"], "batch", t)
    fam = cfg["family"]
    if fam == "mlp":
        x = g.standard_normal((cfg["batch"], cfg["d_in"]), dtype=np.float32)
        y = g.integers(0, cfg["classes"], size=(cfg["batch"],), dtype=np.int32)
    elif fam == "lm":
        x = g.integers(0, cfg["vocab"], size=(cfg["batch"], cfg["seq_len"]), dtype=np.int32)
        y = np.full_like(x, -1)
        y[:, :-1] = x[:, 1:]
        return x, y
    else:
        x = g.standard_normal((cfg["batch"], cfg["in_channels"], cfg["height"], cfg["width"]),
                              dtype=np.float32)
        y = g.integers(0, cfg["classes"], size=(cfg["batch"],), dtype=np.int32)
    if cfg["dtype"] == "bf16":
        x = bf16_round(x)
    return x, y
