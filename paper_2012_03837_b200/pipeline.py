"""Chunks spread over GPUs (Sec. 6): every rank owns one chunk of the chain, or several consecutive ones, trains
them with their own local updates, and hands the output activation of its last chunk, together with the labels
of the minibatch it came from, to the next rank.  No gradient ever travels between ranks (Sec. 3), so the only
traffic is one activation tensor and one label tensor per step and direction, sent point to point (NCCL over
NVLink for device tensors).

At iteration t chunk k trains on the activation chunk k-1 produced at iteration t-1, i.e. on minibatch t-k: the
pipelined schedule of the single-GPU step, with every chunk idle until its first input arrives and again once
its last minibatch has passed (the pipeline drains from the front).  Inside a rank that holds several chunks this
is the library's own pipelined schedule with the idle ramp-up and ``lp_set_drain``.

Host-side plumbing only: the chunks themselves run inside the library (``ChunkStage`` wraps one handle whose model
is that rank's chunks alone; pieces after the first are built with ``input_is_activation``).
"""
from __future__ import annotations

import numpy as np

from . import binding as B


# ----------------------------------------------------------------------------- one chunk as a model of its own

def _conv_out(n: int, stride: int) -> int:
    return (n + 2 - 3) // stride + 1


def stage_config(cfg: dict, r: int, count: int = 1) -> dict:
    """Workload dictionary of chunks r .. r+count-1 of `cfg` as a stand-alone model of `count` chunks."""
    c = {k: v for k, v in cfg.items()}
    c["schedule"] = "sync" if count == 1 else "pipelined"
    fam = cfg["family"]
    if fam == "mlp":
        c["chunks"] = [list(ch) for ch in cfg["chunks"][r:r + count]]
        if r > 0:
            c["d_in"] = cfg["chunks"][r - 1][-1]
    elif fam == "lm":
        c["blocks_per_chunk"] = list(cfg["blocks_per_chunk"][r:r + count])
    else:
        c["stage_channels"] = list(cfg["stage_channels"][r:r + count])
        if isinstance(cfg["blocks_per_stage"], (list, tuple)):
            c["blocks_per_stage"] = list(cfg["blocks_per_stage"][r:r + count])
        if r > 0:
            h, w = cfg["height"], cfg["width"]
            for k in range(1, r):                       # stage 0 keeps the size, every later stage halves it
                h, w = _conv_out(h, 2), _conv_out(w, 2)
            c["height"], c["width"] = h, w
            c["in_channels"] = cfg["stage_channels"][r - 1] * (4 if cfg.get("block") == "bottleneck" else 1)
            c["stem_channels"] = c["in_channels"]
    c["input_is_activation"] = r > 0
    return c


def global_name(cfg: dict, r: int, local: str) -> str:
    """Name, in the whole model, of the tensor that the stand-alone piece starting at chunk r calls `local`
    ("c<j>...." with j counted inside the piece)."""
    head, rest = local.split(".", 1)
    j = int(head[1:])
    if cfg["family"] == "lm" and rest.startswith("b"):
        i, tail = rest[1:].split(".", 1)
        off = sum(cfg["blocks_per_chunk"][:r])
        rest = f"b{off + int(i)}.{tail}"
    return f"c{r + j}.{rest}"


def chunk_flops(cfg: dict, k: int) -> float:
    """Multiply-add work of one local update of chunk k (trunk and head, forward plus the two gradient products of
    every layer): what the chunks are balanced by when several of them share a GPU."""
    fam = cfg["family"]
    if fam == "mlp":
        d_prev = cfg["d_in"] if k == 0 else cfg["chunks"][k - 1][-1]
        f = 0.0
        for w in cfg["chunks"][k]:
            f += d_prev * w
            d_prev = w
        return 6.0 * cfg["batch"] * (f + d_prev * cfg["classes"])
    if fam == "lm":
        d, ffn, t = cfg["d_model"], cfg["d_ffn"], cfg["seq_len"]
        per_token = cfg["blocks_per_chunk"][k] * (4 * d * d + 2 * d * ffn + 2 * d * (t + 1) / 2 * 5 / 3) + d * cfg["vocab"]
        return 6.0 * cfg["batch"] * t * per_token
    bott = cfg.get("block") == "bottleneck"
    h, w = cfg["height"], cfg["width"]
    c_prev = cfg["in_channels"] if cfg.get("input_is_activation") else cfg["stem_channels"]
    f = 0.0
    for j, c in enumerate(cfg["stage_channels"][:k + 1]):
        stride = 1 if (j == 0 and not cfg.get("input_is_activation")) else 2
        h, w = _conv_out(h, stride), _conv_out(w, stride)
        blocks = cfg["blocks_per_stage"][j] if isinstance(cfg["blocks_per_stage"], (list, tuple)) else cfg["blocks_per_stage"]
        c_out = 4 * c if bott else c
        if j == k:
            for i in range(blocks):
                c_in = c_prev if i == 0 else c_out
                f += h * w * ((c_in * c + 9 * c * c + c * c_out) if bott else (9 * c_in * c + 9 * c * c))
                if i == 0 and (stride != 1 or c_in != c_out):
                    f += h * w * c_in * c_out
            f += c_out * cfg["classes"]
        c_prev = c_out
    return 6.0 * cfg["batch"] * f


def partition_chunks(costs, world: int) -> list:
    """Split chunks 0 .. K-1 into `world` contiguous, non-empty ranges so that the largest range sum is as small as
    possible (the slowest rank sets the pipeline's pace); returns [(first, count)] per rank."""
    K = len(costs)
    if not 1 <= world <= K:
        raise ValueError("need 1 <= ranks <= chunks")
    pre = [0.0]
    for c in costs:
        pre.append(pre[-1] + float(c))
    INF = float("inf")
    best = [[INF] * (K + 1) for _ in range(world + 1)]     # best[w][i]: chunks 0..i-1 on w ranks
    cut = [[0] * (K + 1) for _ in range(world + 1)]
    best[0][0] = 0.0
    for w in range(1, world + 1):
        for i in range(w, K - (world - w) + 1):
            for j in range(w - 1, i):
                v = max(best[w - 1][j], pre[i] - pre[j])
                if v < best[w][i]:
                    best[w][i], cut[w][i] = v, j
    out, i = [], K
    for w in range(world, 0, -1):
        j = cut[w][i]
        out.append((j, i - j))
        i = j
    return out[::-1]


class ChunkStage:
    """Chunks r .. r+count-1 of `cfg` on the current CUDA device: one library handle, device buffers for what it
    receives and what it hands on.  With several chunks the handle runs the pipelined schedule with the idle
    ramp-up among them."""

    def __init__(self, cfg: dict, r: int, params: dict | None = None, count: int = 1):
        import torch
        self.torch = torch
        self.cfg, self.r, self.count = cfg, r, count
        self.scfg = stage_config(cfg, r, count)
        m, K, hd, op = B.specs_from_config(self.scfg)
        assert K == count
        self.h = B.lp_create(m, K, hd, op)
        if count > 1:
            B.lp_set_ramp(self.h, B.LP_RAMP_IDLE)
        self.names = {}
        for i in range(B.lp_num_tensors(self.h)):
            info = B.lp_tensor_info_get(self.h, i)
            self.names[global_name(cfg, r, info["name"])] = (i, info)
        if params is not None:
            self.set_params(params)
        dev = torch.device("cuda", torch.cuda.current_device())
        bf = cfg["dtype"] == "bf16"
        self.act_dtype = torch.bfloat16 if bf else torch.float32
        esize = 2 if bf else 4
        self.out = [torch.empty(B.lp_chunk_output_bytes(self.h, count - 1) // esize, dtype=self.act_dtype, device=dev)
                    for _ in range(2)]
        self.loss = torch.zeros(count, dtype=torch.float32, device=dev)
        self.steps = 0

    # what arrives from the previous rank: (activation, labels) buffers of the right size
    def input_buffers(self):
        torch = self.torch
        dev = self.out[0].device
        c = self.scfg
        if c["family"] == "mlp":
            n, rows = c["batch"] * c["d_in"], c["batch"]
        elif c["family"] == "lm":
            n, rows = c["batch"] * c["seq_len"] * c["d_model"], c["batch"] * c["seq_len"]
        else:
            n, rows = c["batch"] * c["height"] * c["width"] * c["in_channels"], c["batch"]
        return (torch.empty(n, dtype=self.act_dtype, device=dev), torch.empty(rows, dtype=torch.int32, device=dev))

    def set_params(self, params: dict):
        """Install master values by their names in the whole model; convolution filters are given as
        [C_out, C_in, kh, kw] and stored as [C_out, kh, kw, C_in]."""
        for g, (i, info) in self.names.items():
            a = np.asarray(params[g], dtype=np.float32)
            if a.ndim == 4:
                a = a.transpose(0, 2, 3, 1)
            a = np.ascontiguousarray(a)
            assert tuple(a.shape) == tuple(info["shape"]), (g, a.shape, info["shape"])
            B.lp_set_tensor(self.h, i, B.LP_MASTER, a)

    def get_params(self) -> dict:
        out = {}
        for g, (i, info) in self.names.items():
            a = np.empty(info["shape"], dtype=np.float32)
            B.lp_get_tensor(self.h, i, B.LP_MASTER, a)
            out[g] = np.ascontiguousarray(a.transpose(0, 3, 1, 2)) if a.ndim == 4 else a
        return out

    def step(self, x, y, idle_first: int = 0):
        """One step of this rank's chunks on (x, y), device tensors: the first chunk trains on (x, y), every later one
        on what its predecessor produced a step earlier; the first `idle_first` chunks idle (the pipeline is draining).
        Returns (loss tensor with one entry per chunk, NaN where a chunk idled; output activation of the last chunk)."""
        stream = self.torch.cuda.current_stream().cuda_stream
        out = self.out[self.steps & 1]
        if self.count == 1:
            B.lp_step(self.h, x, y, B.LP_SYNC, stream, self.loss)
        else:
            B.lp_set_drain(self.h, idle_first)
            B.lp_step(self.h, x, y, B.LP_PIPELINED, stream, self.loss)
        B.lp_chunk_output(self.h, self.count - 1, out, out.numel() * out.element_size(), stream)
        self.steps += 1
        return self.loss, out

    def close(self):
        if self.h:
            B.lp_destroy(self.h)
            self.h = None


# ----------------------------------------------------------------------------- the exchange between ranks

class ChunkPerGpuPipeline:
    """Rank `rank` of `world` ranks holding chunks first .. first+count-1 of K (one chunk each by default).
    `stage` needs step(x, y, idle_first) -> (losses, out) and input_buffers() -> (activation, labels); `dist` is
    torch.distributed (or an object with isend / irecv of the same meaning), so the exchange can be exercised on
    CPU tensors with the gloo backend."""

    def __init__(self, stage, rank: int, world: int, dist, n_minibatches: int, group=None, first: int | None = None,
                 count: int = 1):
        self.stage, self.rank, self.world, self.dist, self.group = stage, rank, world, dist, group
        self.first = rank if first is None else first
        self.count = count
        self.n = n_minibatches                  # chunk k is busy at iterations k .. n + k - 1, then the pipe drains
        self.t = 0
        self.pending = []                       # send requests of the last two iterations
        if rank > 0:
            self.act_in, self.lab_in = stage.input_buffers()
        self.lab_out = [None, None]
        self.labels = []                        # labels of the minibatches inside this rank, oldest first

    def step(self, x=None, y=None):
        """Iteration t of n_minibatches + K - 1.  Rank 0 takes minibatch t (x, y); every other rank takes what its
        predecessor sent at iteration t-1, i.e. the output of chunk first-1 for minibatch t - first.  Returns the
        stage's losses, or None while the rank is idle: nothing has reached it yet (t < first) or its last chunk
        has seen the last minibatch (t >= n + first + count - 1)."""
        d, r, t = self.dist, self.rank, self.t
        self.t += 1
        s = t - self.first                      # this rank's own step count
        if s < 0 or s >= self.n + self.count - 1:
            return None
        feeding = s < self.n                    # the first chunk still has input
        if r > 0 and feeding:
            ra = d.irecv(self.act_in, src=r - 1, group=self.group)
            rl = d.irecv(self.lab_in, src=r - 1, group=self.group)
            ra.wait()
            rl.wait()
        if r > 0:
            x, y = self.act_in, self.lab_in     # while draining the first chunk idles: stale input, not used
        elif not feeding:
            x, y = self.last_xy
        if r == 0 and feeding:
            self.last_xy = (x, y)
        while len(self.pending) >= 2:           # the buffers sent two iterations ago are about to be reused
            for q in self.pending.pop(0):
                q.wait()
        if feeding:
            self.labels.append(y.clone())
        loss, out = self.stage.step(x, y, max(0, s - self.n + 1))
        sending = self.count - 1 <= s < self.count - 1 + self.n     # the last chunk trained on real data
        y_out = self.labels.pop(0) if sending else None
        if sending and r + 1 < self.world:
            slot = t & 1
            if self.lab_out[slot] is None:
                self.lab_out[slot] = y_out.clone()
            else:
                self.lab_out[slot].copy_(y_out)
            self.pending.append((d.isend(out, dst=r + 1, group=self.group),
                                 d.isend(self.lab_out[slot], dst=r + 1, group=self.group)))
        return loss

    def drain(self):
        for qs in self.pending:
            for q in qs:
                q.wait()
        self.pending = []


# ----------------------------------------------------------------------------- launcher (one process per GPU)

def main(argv=None):
    """python -m torch.distributed.run --nnodes=1 --nproc-per-node K --master-addr 127.0.0.1 \\
           -m paper_2012_03837_b200.pipeline --workload c3 --minibatches 50
    The workload's K chunks are split over the ranks in consecutive ranges balanced by their multiply-add work
    (one chunk per rank when K equals the number of ranks), rank 0 feeds seeded synthetic minibatches, activations
    and labels travel rank to rank over NCCL.  Prints one JSON line on rank 0: minibatches, iterations,
    milliseconds (device-timed, maximum over ranks), the chunk ranges, and every rank's last finite loss."""
    import argparse
    import json
    import os
    import sys

    import torch
    import torch.distributed as dist

    sys.path.insert(0, os.path.dirname(os.path.dirname(os.path.abspath(__file__))))
    import lp_synth

    ap = argparse.ArgumentParser()
    ap.add_argument("--workload", default="c3")
    ap.add_argument("--minibatches", type=int, default=20)
    ap.add_argument("--override", action="append", default=[], metavar="KEY=JSON",
                    help="replace a field of the workload, e.g. --override 'blocks_per_chunk=[2,2]'")
    a = ap.parse_args(argv)
    rank, world = int(os.environ.get("RANK", 0)), int(os.environ.get("WORLD_SIZE", 1))
    torch.cuda.set_device(int(os.environ.get("LOCAL_RANK", 0)))
    dev = torch.device("cuda", torch.cuda.current_device())
    dist.init_process_group("nccl", rank=rank, world_size=world, device_id=dev)
    try:
        cfg = lp_synth.config(a.workload, **{k: json.loads(v) for k, v in (o.split("=", 1) for o in a.override)})
        K = lp_synth.num_chunks(cfg)
        if K < world:
            raise SystemExit(f"workload {a.workload} has {K} chunks: launch at most that many ranks")
        ranges = partition_chunks([chunk_flops(cfg, k) for k in range(K)], world)
        first, count = ranges[rank]
        params = lp_synth.init_params(cfg)
        stage = ChunkStage(cfg, first, params, count)
        pipe = ChunkPerGpuPipeline(stage, rank, world, dist, a.minibatches, first=first, count=count)
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        dist.barrier()
        torch.cuda.synchronize()
        e0.record()
        last = float("nan")
        for t in range(a.minibatches + K - 1):
            x = y = None
            if rank == 0 and t < a.minibatches:
                xn, yn = lp_synth.minibatch(cfg, t)
                x = torch.from_numpy(xn).to(dev)
                if cfg["family"] != "lm" and cfg["dtype"] == "bf16":
                    x = x.to(torch.bfloat16)
                x, y = x.contiguous(), torch.from_numpy(yn).to(dev).contiguous()
            loss = pipe.step(x, y)
            if loss is not None:
                fin = loss[torch.isfinite(loss)]
                if fin.numel():
                    last = fin[-1:].clone()
        pipe.drain()
        e1.record()
        torch.cuda.synchronize()
        ms = torch.tensor([e0.elapsed_time(e1)], device=dev)
        dist.all_reduce(ms, op=dist.ReduceOp.MAX)
        losses = [torch.zeros(1, device=dev) for _ in range(world)]
        dist.all_gather(losses, last if torch.is_tensor(last) else torch.full((1,), last, device=dev))
        if rank == 0:
            print(json.dumps({"workload": a.workload, "ranks": world, "minibatches": a.minibatches,
                              "iterations": a.minibatches + K - 1, "ms": float(ms[0]), "chunk_ranges": ranges,
                              "last_losses": [float(v[0]) for v in losses]}))
        stage.close()
    finally:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
