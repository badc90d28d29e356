#!/usr/bin/env python
"""Benchmark of the local update step (paper Sec. 3 / Sec. 6) on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload c1..c5] [--impl ours|reference]

Prints ONE JSON line.  A step is one full local update (every chunk: trunk forward, auxiliary head
and loss, truncated backward, optimizer update) on one synthetic minibatch.  `value` is timed with
CUDA events with the minibatches already resident in device memory; `e2e` is the same metric through
lp_step_host with pinned host buffers (host->device copies of x, y and the device->host read of the K
losses inside the timed region).  With N > 1 (launched by torch.distributed.run) every rank runs an
independent replica on its own GPU (the method, as built here, runs on one GPU with no inter-GPU
exchange); the time is the maximum over ranks and the value the sum of all replicas' units.
"""
from __future__ import annotations

import argparse
import json
import os
import subprocess
import sys
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

import lp_synth  # noqa: E402

DEFAULT_WORKLOAD = "c5"
DEFAULT_STEPS = {"c1": 200, "c2": 40, "c3": 10, "c4": 10, "c5": 6}
L2_BYTES = 126 * 1024 * 1024


def metric_of(cfg):
    if cfg["family"] == "lm":
        return "local-update train step tokens/s", "tokens/s"
    return "local-update train step samples/s", "samples/s"


def n_parameters(cfg):
    return int(sum(int(np.prod(t["shape"])) for t in lp_synth.param_table(cfg) if not t.get("buffer")))


def flushes_l2(cfg):
    """Workloads whose per-step working set (parameters, moments and gradients: >= 16 bytes per parameter) is not
    several times the 126 MB L2 get the cache flushed between timed steps."""
    return 16 * n_parameters(cfg) < 4 * L2_BYTES


def describe(cfg, world=1):
    """The `config` object of the JSON line; both arms (GPU library and CPU oracle) print the same one."""
    d = dict(workload=cfg["name"], family=cfg["family"], K=lp_synth.num_chunks(cfg), schedule=cfg["schedule"],
             optimizer=cfg["optim"]["kind"], batch=cfg["batch"])
    for k in ("seq_len", "vocab", "d_model", "n_heads", "d_ffn", "d_in", "classes"):
        if k in cfg:
            d[k] = cfg[k]
    if cfg["family"] == "mlp":
        d["chunks"] = cfg["chunks"]
    d["l2"] = "flushed between steps" if flushes_l2(cfg) else "not flushed: the step's working set is many times the 126 MB L2"
    d["parallelism"] = "replicas" if world > 1 else "1 GPU"
    return d


# DRAM bytes (dram__bytes_read.sum + dram__bytes_write.sum) per launch of the dominant kernel, from the ncu
# capture summarised under profiles/ and scaled to the launches of a full step.  A figure is only
# valid for the kernel source it was captured on: it is dropped when that file has changed since.
TRAFFIC = {
    # per chunk (ncu): head products 1.95 GB (forward 0.57, input gradient 0.61 and weight gradient 0.77 on the
    # 256x512 tiles), block products 0.76 GB; every chunk streams its own operands, so a 24-chunk step moves
    # 24 x 2.71 GB = 65 GB over its thirteen GEMM launches
    "c5": dict(bytes_per_launch=5.0e9, chunks=24, kernel_file="paper_2012_03837_b200/csrc/gemm_tc.cu",
               kernel_sha256="38616d45d63a33ff10b9ee02f9b0c1ba6f1147f3479332c7671486713343fb3b"),
}


def measured_traffic(workload, chunks):
    rec = TRAFFIC.get(workload)
    if not rec or rec["bytes_per_launch"] is None or rec["chunks"] != chunks:
        return None
    import hashlib
    try:
        with open(os.path.join(ROOT, rec["kernel_file"]), "rb") as f:
            sha = hashlib.sha256(f.read()).hexdigest()
    except OSError:
        return None
    return rec["bytes_per_launch"] if sha == rec["kernel_sha256"] else None


# Datasheet figures of the part (NVIDIA HGX B200: 2.25 PFLOP/s dense bf16 -- half of the 4.5 PFLOP/s quoted with
# 2:4 sparsity -- and 7.7 TB/s of HBM3e bandwidth per GPU); context beside the measured denominators.
NOMINAL_TENSOR_TFLOPS = 2250.0
NOMINAL_HBM_GBS = 7700.0


def peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        with open(p) as f:
            j = json.load(f)
        return dict(hbm=j["hbm_gbs"], tensor_burst=j["bf16_tflops"], tensor_sustained=j["bf16_tflops_sustained"], source="measured")
    return dict(hbm=6650.0, tensor_burst=1590.0, tensor_sustained=1400.0, source="fallback")


# ----------------------------------------------------------------------------- CPU oracle timing

def oracle_sample(cfg):
    """(callable running one bounded sample, samples per step, description).

    Small workloads: one whole step.  Transformer workloads: the local update of one generic chunk
    (chunk 1: trunk forward, head, truncated backward, optimizer update) of a two-chunk model with
    the workload's dimensions, on a fraction of the batch; a step costs K times that chunk times the
    batch fraction's inverse (every chunk >= 1 has the same layers; chunk 0 adds the embedding)."""
    from oracle.local_step import LocalUpdateOracle
    K = lp_synth.num_chunks(cfg)
    if cfg["family"] == "lm":
        frac = 8 if cfg["d_model"] >= 1024 else 1
        small = lp_synth.config(cfg["name"], blocks_per_chunk=[1, 1], batch=max(1, cfg["batch"] // frac))
        orc = LocalUpdateOracle(small, lp_synth.init_params(small), dtype=np.float32)
        x, y = lp_synth.minibatch(small, 0)
        h, _ = orc.chunk_forward(0, x)

        def run():
            _, _, g = orc.local_grads(1, h, y)
            orc.apply_update(1, g)
        scale = K * (cfg["batch"] / small["batch"])
        return run, scale, (
            f"oracle fp32: local update of chunk 1 of a 2-chunk model with this workload's dimensions on "
            f"{small['batch']} of {cfg['batch']} sequences; step time = sample x {scale:g}")
    orc = LocalUpdateOracle(cfg, lp_synth.init_params(cfg), dtype=np.float32)
    state = {"t": 0}

    def run():
        orc.step(*lp_synth.minibatch(cfg, state["t"]))
        state["t"] += 1
    return run, 1.0, "oracle fp32: whole steps of the workload"


def time_oracle(cfg, steps, warmup, budget_s=25.0):
    """Times the oracle as it stands on the host cores: (units/s, seconds per sample, seconds per step,
    samples timed, threads used, description of the sample)."""
    run, scale, desc = oracle_sample(cfg)
    for _ in range(warmup):
        run()
    times = []
    t_start = time.perf_counter()
    for _ in range(steps):
        t0 = time.perf_counter()
        run()
        times.append(time.perf_counter() - t0)
        if budget_s and time.perf_counter() - t_start > budget_s:
            break
    t = float(np.mean(times))
    try:
        from threadpoolctl import threadpool_info
        cores = max([i.get("num_threads", 1) for i in threadpool_info()] + [1])
    except Exception:
        cores = os.cpu_count()
    return lp_synth.units_per_step(cfg) / (t * scale), t, t * scale, len(times), cores, desc


def run_reference(args, cfg):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    metric, unit = metric_of(cfg)
    value, t_sample, t_step, n, cores, desc = time_oracle(cfg, args.steps, args.warmup, budget_s=0)
    line = dict(impl="reference", metric=metric, value=value, unit=unit, n_gpus=args.gpus, steps=n, warmup=args.warmup,
                ms_per_step=t_step * 1e3, sample_seconds=t_sample, higher_is_better=True, scaling="weak", vs_baseline=None,
                dtype="f32", data="synthetic", config=describe(cfg, args.gpus),
                cpu_baseline=dict(value=value, unit=unit, cores=cores, kind="oracle", sample=desc),
                e2e=dict(value=value, unit=unit, h2d_bytes_per_step=0, d2h_bytes_per_step=0))
    print(json.dumps(line))


# ----------------------------------------------------------------------------- clocks

class ClockSampler:
    Q = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
         "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, index):
        self.rows = []
        self.proc = None
        try:
            self.proc = subprocess.Popen(["nvidia-smi", "-i", str(index), f"--query-gpu={self.Q}", "--format=csv,noheader,nounits",
                                          "-lms", "100"], stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.th = threading.Thread(target=self._read, daemon=True)
            self.th.start()
        except Exception:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.rows.append((time.perf_counter(), line.strip()))

    def stop(self, t0, t1):
        if not self.proc:
            return dict(sm_mhz=None, sm_max_mhz=None, reasons=["nvidia-smi unavailable"])
        time.sleep(0.15)
        self.proc.terminate()
        sm, mx, reasons = [], [], set()
        for t, line in self.rows:
            if not (t0 <= t <= t1 + 0.2):
                continue
            f = [v.strip() for v in line.split(",")]
            if len(f) < 7:
                continue
            try:
                sm.append(float(f[0])); mx.append(float(f[1]))
            except ValueError:
                continue
            for name, v in zip(("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"), f[3:7]):
                if v == "Active":
                    reasons.add(name)
        if not sm:
            return dict(sm_mhz=None, sm_max_mhz=None, reasons=["no sample inside the timed region"], samples=0)
        return dict(sm_mhz=float(np.median(sm)), sm_max_mhz=float(np.max(mx)), reasons=sorted(reasons), samples=len(sm))


# ----------------------------------------------------------------------------- N > 1: independent replicas

def replica_config(cfg, rank):
    """Every replica draws its own weights and data: the path has no exchange step, so N GPUs run N
    independent copies of the local update step (weak scaling)."""
    return dict(cfg, seed=cfg["seed"] + rank)


def max_over_ranks(values, dist, device):
    """Element-wise maximum of `values` over all ranks (the slowest replica sets the job's time)."""
    if dist is None:
        return [float(v) for v in values]
    import torch
    tt = torch.tensor(list(values), dtype=torch.float64, device=device)
    dist.all_reduce(tt, op=dist.ReduceOp.MAX)
    return tt.tolist()


def whole_job_rate(world, units_per_step, ms_per_step):
    """Units all replicas processed per second, given the slowest replica's step time."""
    return world * units_per_step / (ms_per_step * 1e-3)


# ----------------------------------------------------------------------------- the GPU arm

# Algorithmic bytes behind the HBM-bound kernel classes, as the library counts them when it builds a step's
# launch list (lp_profile_read returns their sums).
BYTE_FORMULAS = {
    "optim": "Adam: 16 B read (master, gradient, two moments) + 12 B written (master, two moments) per parameter, "
             "SGD-momentum 12 + 8; + 2 B per matrix element for the bf16 working copy",
    "xent": "one read and one write of the bf16 logits (dlogits in place) + the per-128-column softmax statistics",
    "norm": "LayerNorm forward: x read + y written; backward: dy and x read, dx written; BatchNorm: one read per "
            "statistics pass, read + write per apply pass",
    "reduce": "one read of the summed matrix (bias gradients) or of the fp32 partial sums",
    "embed": "gather: token and position rows read, activation written",
    "conv_aux": "im2col / col2im / pooling / layout change / residual add: operands read + result written",
}


def measure(lp, torch, cfg, steps, warmup, dist, dev, rank, world, local, cpu_steps):
    """Times `steps` local update steps of `cfg` on this rank's GPU; rank 0 returns the JSON line's dictionary."""
    m, K, hd, op = lp.specs_from_config(cfg)
    h = lp.lp_create(m, K, hd, op)
    names = {}
    for i in range(lp.lp_num_tensors(h)):
        info = lp.lp_tensor_info_get(h, i)
        names[info["name"]] = (i, info)
    stream = torch.cuda.current_stream().cuda_stream
    cfg_r = replica_config(cfg, rank)
    for n, a in lp_synth.init_params(cfg_r).items():
        if a.ndim == 4:
            a = np.ascontiguousarray(a.transpose(0, 2, 3, 1))
        lp.lp_set_tensor(h, names[n][0], lp.LP_MASTER, np.ascontiguousarray(a, dtype=np.float32), stream)
    sched = lp.LP_SYNC if cfg["schedule"] == "sync" else lp.LP_PIPELINED

    NB = 4                                              # distinct minibatches, cycled
    host, devb = [], []
    for t in range(NB):
        x, y = lp_synth.minibatch(cfg_r, t)
        xt = torch.from_numpy(x)
        if cfg["family"] != "lm" and cfg["dtype"] == "bf16":
            xt = xt.to(torch.bfloat16)
        yt = torch.from_numpy(y)
        host.append((xt.contiguous().pin_memory(), yt.contiguous().pin_memory()))
        devb.append((host[-1][0].to(dev), host[-1][1].to(dev)))
    losses = torch.zeros(K, dtype=torch.float32, device=dev)
    losses_host = torch.zeros(K, dtype=torch.float32).pin_memory()

    working_set = lp.lp_device_bytes(h)
    flush = flushes_l2(cfg)
    flush_buf = torch.empty(2 * L2_BYTES, dtype=torch.uint8, device=dev) if flush else None

    def barrier():
        torch.cuda.synchronize()
        if dist is not None:
            dist.barrier()
            torch.cuda.synchronize()

    for t in range(warmup):
        lp.lp_step(h, devb[t % NB][0], devb[t % NB][1], sched, stream, losses)
    barrier()
    lp.lp_status_poll(h, stream)

    # The per-class event brackets cost host time per launch.  Steps of a few milliseconds hide it; for the
    # launch-bound small workloads the breakdown is taken in a second pass of the same steps instead.
    p0, p1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    p0.record()
    for t in range(3):
        lp.lp_step(h, devb[t % NB][0], devb[t % NB][1], sched, stream, losses)
    p1.record()
    barrier()
    separate_profile = p0.elapsed_time(p1) / 3 < 2.0

    clocks = ClockSampler(local) if rank == 0 else None
    lp.lp_profile_enable(h, not separate_profile)
    evs = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(steps)]
    barrier()
    t_wall0 = time.perf_counter()
    launches = 0
    for t in range(steps):
        if flush:
            flush_buf.fill_(t & 0xff)
        xb, yb = devb[(warmup + t) % NB]
        evs[t][0].record()
        lp.lp_step(h, xb, yb, sched, stream, losses)
        evs[t][1].record()
        launches += lp.lp_last_step_launches(h)
    barrier()
    t_wall1 = time.perf_counter()
    clock_rec = clocks.stop(t_wall0, t_wall1) if clocks else None
    ms_total = sum(a.elapsed_time(b) for a, b in evs)
    if separate_profile:
        lp.lp_profile_enable(h, True)
        for t in range(steps):
            if flush:
                flush_buf.fill_(t & 0xff)
            xb, yb = devb[(warmup + t) % NB]
            lp.lp_step(h, xb, yb, sched, stream, losses)
        barrier()
    lp.lp_profile_enable(h, False)
    prof = lp.lp_profile_read(h)
    ms_profiled = sum(v[0] for v in prof.values())
    final_losses = losses.cpu().numpy().tolist()
    lp.lp_status_poll(h, stream)

    # end to end: host buffers in, host losses out, every step
    e2e_steps = max(3, min(steps, 20))
    for t in range(2):
        lp.lp_step_host(h, host[t % NB][0], host[t % NB][1], sched, stream, losses_host)
    barrier()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for t in range(e2e_steps):
        lp.lp_step_host(h, host[t % NB][0], host[t % NB][1], sched, stream, losses_host)
    e1.record()
    barrier()
    ms_e2e = e0.elapsed_time(e1) / e2e_steps

    ms_total, ms_e2e = max_over_ranks([ms_total, ms_e2e], dist, dev)
    units = lp_synth.units_per_step(cfg)
    ms_step = ms_total / steps
    value = whole_job_rate(world, units, ms_step)
    e2e_value = whole_job_rate(world, units, ms_e2e)
    h2d = int(host[0][0].numel() * host[0][0].element_size() + host[0][1].numel() * 4)
    lp.lp_destroy(h)
    del devb, host, flush_buf
    torch.cuda.empty_cache()
    if rank != 0:
        return None

    metric, unit = metric_of(cfg)
    pk = peaks()
    gms, gflop, gl = prof["gemm_tc"]
    if gl > 0 and gms > 0:
        achieved = gflop / (gms * 1e-3) / 1e12
        roof = dict(bound="tensor", kernel="gemm_tc_kernel (grouped tcgen05 bf16 GEMM)", achieved=achieved,
                    peak=pk["tensor_sustained"], unit="TFLOP/s", frac=achieved / pk["tensor_sustained"],
                    peak_source=pk["source"] + " sustained cuBLAS bf16",
                    frac_of_nominal=achieved / NOMINAL_TENSOR_TFLOPS, nominal_peak=NOMINAL_TENSOR_TFLOPS,
                    nominal_source="datasheet, dense bf16 (half of the figure quoted with 2:4 sparsity)",
                    traffic=measured_traffic(cfg["name"], K),
                    launches=gl, ms_per_launch=gms / gl, share_of_step=gms / ms_profiled)
    else:
        ams, aflop, al = prof["gemm_alu"]
        achieved = aflop / max(ams * 1e-3, 1e-12) / 1e12
        peak = 148 * 128 * 2 * 1.965e9 / 1e12        # FP32 FMA lanes x 2 FLOP x max SM clock
        one_launch = launches == steps
        roof = dict(bound="alu",
                    kernel=("fused_mlp_step_kernel (the whole step as one cooperative launch: a chain of dependent "
                            "phases, bound by their latency, not by the FP32 lanes)") if one_launch
                    else "gemm_simt_kernel (grouped FP32-ALU GEMM)", achieved=achieved, peak=peak,
                    unit="TFLOP/s", frac=achieved / peak, peak_source="148 SMs x 128 FP32 lanes x 2 x 1.965 GHz",
                    traffic=None, launches=al, ms_per_launch=ams / max(al, 1), share_of_step=ams / ms_profiled)
    breakdown = {}
    for k, (ms, work, n) in prof.items():
        if n == 0:
            continue
        is_flop = k in ("gemm_tc", "gemm_alu", "attn")
        rate = work / max(ms * 1e-3, 1e-12)
        if is_flop:
            breakdown[k] = dict(ms_per_step=ms / steps, launches_per_step=n / steps, share=ms / ms_profiled, tflops=rate / 1e12)
        else:
            frac = rate / 1e9 / pk["hbm"]
            breakdown[k] = dict(ms_per_step=ms / steps, launches_per_step=n / steps, share=ms / ms_profiled, gbs=rate / 1e9,
                                frac_of_hbm_peak=frac, frac_of_nominal_hbm=rate / 1e9 / NOMINAL_HBM_GBS,
                                bytes_per_step=work / steps, bytes_counted=BYTE_FORMULAS.get(k, "operands read + results written"))
            if frac > 1.0:
                # the denominator is a measured copy kernel (MEASURED_PEAKS.json), not the hardware's limit
                breakdown[k]["note"] = (f"above the {pk['source']} copy rate of {pk['hbm']:.0f} GB/s; "
                                        f"{rate / 1e9 / NOMINAL_HBM_GBS:.2f} of the nominal {NOMINAL_HBM_GBS:.0f} GB/s")
    cpu = None
    if world == 1 and cpu_steps > 0:
        v, t_sample, t_step, n, cores, desc = time_oracle(cfg, cpu_steps, 1 if cpu_steps > 1 else 0)
        cpu = dict(value=v, unit=unit, cores=cores, kind="oracle", sample=desc, sample_seconds=t_sample, samples=n)
    return dict(metric=metric, value=value, unit=unit, n_gpus=world, steps=steps, warmup=warmup,
                ms_per_step=ms_step, higher_is_better=True, scaling="weak", vs_baseline=None,
                dtype="bf16" if cfg["dtype"] == "bf16" else "f32", data="synthetic",
                config=describe(cfg, world),
                e2e=dict(value=e2e_value, unit=unit, h2d_bytes_per_step=h2d, d2h_bytes_per_step=4 * K, ms_per_step=ms_e2e),
                gpu_launches=launches, clocks=clock_rec, roofline=roof, kernels=breakdown,
                hbm_peak=dict(value=pk["hbm"], unit="GB/s", source=pk["source"] + " device copy"),
                kernel_timing="second pass of the same steps (launch-bound workload)" if separate_profile else "timed region",
                cpu_baseline=cpu,
                final_losses=final_losses, device_bytes=working_set)


def run_ours(args, cfg, also):
    import torch
    from paper_2012_03837_b200 import build as lpbuild
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if local == 0:
        lpbuild.build()
    torch.cuda.set_device(local)
    dist = None
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))
        dist.barrier()
    from paper_2012_03837_b200 import binding as lp
    dev = torch.device("cuda", local)
    line = measure(lp, torch, cfg, args.steps, args.warmup, dist, dev, rank, world, local,
                   0 if args.no_cpu_baseline else 3)
    # the other workloads, each a short run of the same kind, reported under "workloads"
    others = {}
    for name in also:
        c = lp_synth.config(name)
        rec = measure(lp, torch, c, DEFAULT_STEPS[name], max(args.warmup, 3), dist, dev, rank, world, local,
                      0 if args.no_cpu_baseline else (3 if name in ("c1", "c2") else 1))
        if rec is not None:
            others[name] = {k: rec[k] for k in ("metric", "value", "unit", "steps", "warmup", "ms_per_step", "dtype", "config", "e2e",
                                                "gpu_launches", "clocks", "roofline", "kernels", "kernel_timing", "cpu_baseline")}
    if rank == 0:
        if others:
            line["workloads"] = others
        print(json.dumps(line))
    if dist is not None:
        dist.barrier()
        dist.destroy_process_group()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=None)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--workload", default=None, choices=["c1", "c2", "c3", "c4", "c5"],
                    help="time this workload alone; by default the headline line is c5 and short runs of c1-c4 are "
                         "added under its \"workloads\" key")
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--chunks", type=int, default=None,
                    help="LM workloads: keep only the first N chunks (a small case of the same kernels for profiler captures; "
                         "the line's config then shows K=N, so it is not the benchmark's number)")
    args = ap.parse_args()
    workload = args.workload or DEFAULT_WORKLOAD
    cfg = lp_synth.config(workload)
    if args.chunks is not None:
        if cfg["family"] != "lm" or not 1 <= args.chunks <= len(cfg["blocks_per_chunk"]):
            ap.error("--chunks applies to the LM workloads, 1 <= N <= K")
        cfg = lp_synth.config(workload, blocks_per_chunk=cfg["blocks_per_chunk"][:args.chunks])
    if args.impl == "reference":
        if args.steps is None:
            args.steps = 3
        run_reference(args, cfg)
        return
    if args.steps is None:
        args.steps = DEFAULT_STEPS[workload]
    args.warmup = max(args.warmup, 3)
    also = [w for w in ("c1", "c2", "c3", "c4") if args.workload is None and args.chunks is None]
    run_ours(args, cfg, also)


if __name__ == "__main__":
    main()
