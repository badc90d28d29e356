"""One chunk per GPU (Sec. 6): every rank owns one chunk of the chain, trains it with its own local update,
and hands the chunk's output activation, together with the labels of the minibatch it came from, to the
next rank.  No gradient ever travels between ranks (Sec. 3), so the only traffic is one activation tensor
and one label tensor per step and direction, sent point to point (NCCL over NVLink for device tensors).

At iteration t rank r trains on the activation rank r-1 produced at iteration t-1, i.e. on minibatch t-r:
the pipelined schedule of the single-GPU step, with the ranks idle until their first input arrives.

Host-side plumbing only: the chunk itself runs inside the library (``ChunkStage`` wraps one handle whose
model is that chunk alone; chunks after the first are built with ``input_is_activation``).
"""
from __future__ import annotations

import numpy as np

from . import binding as B


# ----------------------------------------------------------------------------- one chunk as a model of its own

def _conv_out(n: int, stride: int) -> int:
    return (n + 2 - 3) // stride + 1


def stage_config(cfg: dict, r: int) -> dict:
    """Workload dictionary of chunk r of `cfg` as a stand-alone one-chunk model."""
    c = {k: v for k, v in cfg.items()}
    c["schedule"] = "sync"
    fam = cfg["family"]
    if fam == "mlp":
        c["chunks"] = [list(cfg["chunks"][r])]
        if r > 0:
            c["d_in"] = cfg["chunks"][r - 1][-1]
    elif fam == "lm":
        c["blocks_per_chunk"] = [cfg["blocks_per_chunk"][r]]
    else:
        c["stage_channels"] = [cfg["stage_channels"][r]]
        if r > 0:
            h, w = cfg["height"], cfg["width"]
            for k in range(1, r):                       # stage 0 keeps the size, every later stage halves it
                h, w = _conv_out(h, 2), _conv_out(w, 2)
            c["height"], c["width"] = h, w
            c["in_channels"] = cfg["stage_channels"][r - 1]
            c["stem_channels"] = c["in_channels"]
    c["input_is_activation"] = r > 0
    return c


def global_name(cfg: dict, r: int, local: str) -> str:
    """Name, in the whole model, of the tensor the stand-alone chunk r calls `local` ("c0....")."""
    assert local.startswith("c0.")
    rest = local[3:]
    if cfg["family"] == "lm" and rest.startswith("b"):
        j, tail = rest[1:].split(".", 1)
        off = sum(cfg["blocks_per_chunk"][:r])
        rest = f"b{off + int(j)}.{tail}"
    return f"c{r}.{rest}"


class ChunkStage:
    """Chunk r of `cfg` on the current CUDA device: one library handle, device buffers for what it receives
    and what it hands on."""

    def __init__(self, cfg: dict, r: int, params: dict | None = None):
        import torch
        self.torch = torch
        self.cfg, self.r = cfg, r
        self.scfg = stage_config(cfg, r)
        m, K, hd, op = B.specs_from_config(self.scfg)
        assert K == 1
        self.h = B.lp_create(m, K, hd, op)
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
        self.out = [torch.empty(B.lp_chunk_output_bytes(self.h, 0) // esize, dtype=self.act_dtype, device=dev)
                    for _ in range(2)]
        self.loss = torch.zeros(1, dtype=torch.float32, device=dev)
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

    def step(self, x, y):
        """One local update of this chunk on (x, y), device tensors; returns (loss tensor, output activation)."""
        stream = self.torch.cuda.current_stream().cuda_stream
        out = self.out[self.steps & 1]
        B.lp_step(self.h, x, y, B.LP_SYNC, stream, self.loss)
        B.lp_chunk_output(self.h, 0, out, out.numel() * out.element_size(), stream)
        self.steps += 1
        return self.loss, out

    def close(self):
        if self.h:
            B.lp_destroy(self.h)
            self.h = None


# ----------------------------------------------------------------------------- the exchange between ranks

class ChunkPerGpuPipeline:
    """Rank `rank` of `world` ranks, one chunk each.  `stage` needs step(x, y) -> (loss, out) and
    input_buffers() -> (activation, labels); `dist` is torch.distributed (or an object with isend / irecv of
    the same meaning), so the exchange can be exercised on CPU tensors with the gloo backend."""

    def __init__(self, stage, rank: int, world: int, dist, n_minibatches: int, group=None):
        self.stage, self.rank, self.world, self.dist, self.group = stage, rank, world, dist, group
        self.n = n_minibatches                  # rank r is busy at iterations r .. n + r - 1, then the pipe drains
        self.t = 0
        self.pending = []                       # send requests of the last two iterations
        if rank > 0:
            self.act_in, self.lab_in = stage.input_buffers()
        self.lab_out = [None, None]

    def step(self, x=None, y=None):
        """Iteration t of n_minibatches + world - 1.  Rank 0 takes minibatch t (x, y); every other rank takes
        what its predecessor sent at iteration t-1, i.e. minibatch t - rank.  A rank is idle (returns None)
        while nothing has reached it yet (t < rank) and once its last minibatch is done (t >= n + rank)."""
        d, r, t = self.dist, self.rank, self.t
        self.t += 1
        if t < r or t >= self.n + r:
            return None
        if r > 0:
            ra = d.irecv(self.act_in, src=r - 1, group=self.group)
            rl = d.irecv(self.lab_in, src=r - 1, group=self.group)
            ra.wait()
            rl.wait()
            x, y = self.act_in, self.lab_in
        while len(self.pending) >= 2:           # the buffers sent two iterations ago are about to be reused
            for q in self.pending.pop(0):
                q.wait()
        loss, out = self.stage.step(x, y)
        if r + 1 < self.world:
            slot = t & 1
            if self.lab_out[slot] is None:
                self.lab_out[slot] = y.clone()
            else:
                self.lab_out[slot].copy_(y)
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
    Rank r holds chunk r of the workload (its chunk count must equal the number of ranks), rank 0 feeds
    seeded synthetic minibatches, activations and labels travel rank to rank over NCCL.  Prints one JSON
    line on rank 0: minibatches, iterations, milliseconds (device-timed, maximum over ranks), and every
    rank's last loss."""
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
        if lp_synth.num_chunks(cfg) != world:
            raise SystemExit(f"workload {a.workload} has {lp_synth.num_chunks(cfg)} chunks: launch that many ranks")
        params = lp_synth.init_params(cfg)
        stage = ChunkStage(cfg, rank, params)
        pipe = ChunkPerGpuPipeline(stage, rank, world, dist, a.minibatches)
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        dist.barrier()
        torch.cuda.synchronize()
        e0.record()
        last = float("nan")
        for t in range(a.minibatches + world - 1):
            x = y = None
            if rank == 0 and t < a.minibatches:
                xn, yn = lp_synth.minibatch(cfg, t)
                x = torch.from_numpy(xn).to(dev)
                if cfg["family"] != "lm" and cfg["dtype"] == "bf16":
                    x = x.to(torch.bfloat16)
                x, y = x.contiguous(), torch.from_numpy(yn).to(dev).contiguous()
            loss = pipe.step(x, y)
            if loss is not None:
                last = loss
        pipe.drain()
        e1.record()
        torch.cuda.synchronize()
        ms = torch.tensor([e0.elapsed_time(e1)], device=dev)
        dist.all_reduce(ms, op=dist.ReduceOp.MAX)
        losses = [torch.zeros(1, device=dev) for _ in range(world)]
        dist.all_gather(losses, last if torch.is_tensor(last) else torch.full((1,), last, device=dev))
        if rank == 0:
            print(json.dumps({"workload": a.workload, "ranks": world, "minibatches": a.minibatches,
                              "iterations": a.minibatches + world - 1, "ms": float(ms[0]),
                              "last_losses": [float(v[0]) for v in losses]}))
        stage.close()
    finally:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
