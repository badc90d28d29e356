"""Chunks spread over GPUs (Sec. 6).  On CPU: the stand-alone chunk configurations (single chunks and ranges of
consecutive chunks) cover the whole model tensor by tensor; the partition of the chunks over the ranks is
contiguous and balanced; and the point-to-point exchange, run by gloo ranks on CPU tensors with stand-in stages,
gives chunk k at iteration t the activation and labels of minibatch t-k, with one chunk per rank and with uneven
ranges of chunks per rank.  On one GPU: the ranks are emulated in one process, one library handle per rank,
stepped in turn with the hand-over done by device copies; losses and weights against the oracle's pipelined
schedule with idle ramp-up, including the drain at the end of a run."""
import os
import sys

import numpy as np
import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
sys.path.insert(0, ROOT)
import lp_synth  # noqa: E402
from paper_2012_03837_b200 import pipeline as P  # noqa: E402

SMALL = {
    "mlp": lp_synth.config("c1", batch=6, d_in=7, chunks=[[6], [5, 4], [6]], classes=5),
    "lm": lp_synth.config("c3", batch=2, seq_len=5, vocab=11, d_model=8, n_heads=2, d_ffn=12,
                          blocks_per_chunk=[1, 2, 1]),
    "resnet": lp_synth.config("c4", batch=3, height=8, width=8, stem_channels=4, stage_channels=[4, 6, 8],
                              blocks_per_stage=2, classes=3),
}


@pytest.mark.parametrize("fam", sorted(SMALL))
def test_stand_alone_chunks_cover_the_model(fam):
    cfg = SMALL[fam]
    full = {t["name"]: (t["shape"], t["chunk"]) for t in lp_synth.param_table(cfg)}
    got = {}
    for r in range(lp_synth.num_chunks(cfg)):
        sc = P.stage_config(cfg, r)
        assert lp_synth.num_chunks(sc) == 1 and bool(sc["input_is_activation"]) == (r > 0)
        for t in lp_synth.param_table(sc):
            g = P.global_name(cfg, r, t["name"])
            assert g not in got
            got[g] = (t["shape"], r)
    assert got == full


@pytest.mark.parametrize("fam", sorted(SMALL))
def test_ranges_of_chunks_cover_the_model(fam):
    cfg = SMALL[fam]
    full = {t["name"]: t["shape"] for t in lp_synth.param_table(cfg)}
    got = {}
    for first, count in ((0, 2), (2, 1)):
        sc = P.stage_config(cfg, first, count)
        assert lp_synth.num_chunks(sc) == count and bool(sc["input_is_activation"]) == (first > 0)
        for t in lp_synth.param_table(sc):
            g = P.global_name(cfg, first, t["name"])
            assert g not in got
            got[g] = t["shape"]
    assert got == full


def test_partition_is_contiguous_and_balanced():
    import itertools
    for costs, world in (([5, 1, 1, 1, 1, 1, 1], 3), ([1] * 24, 8), ([3, 1, 4, 1, 5, 9, 2, 6], 4), ([2, 2], 2), ([7], 1)):
        parts = P.partition_chunks(costs, world)
        assert len(parts) == world and parts[0][0] == 0 and all(c >= 1 for _, c in parts)
        assert all(parts[i][0] + parts[i][1] == parts[i + 1][0] for i in range(world - 1))
        assert parts[-1][0] + parts[-1][1] == len(costs)
        worst = max(sum(costs[f:f + c]) for f, c in parts)
        # brute force over all ways to cut
        best = min(max(sum(costs[a:b]) for a, b in zip((0,) + cuts, cuts + (len(costs),)))
                   for cuts in itertools.combinations(range(1, len(costs)), world - 1))
        assert worst == best, (costs, world, parts)
    c5 = lp_synth.config("c5")
    parts = P.partition_chunks([P.chunk_flops(c5, k) for k in range(24)], 8)
    assert [c for _, c in parts] == [3] * 8                     # equal blocks: three chunks per GPU
    with pytest.raises(ValueError):
        P.partition_chunks([1, 2], 3)


class FakeStage:
    """Stand-in for a rank's chunks: chunk k computes out = 2 x + (k + 1), one iteration after its predecessor;
    remembers what its first chunk was given and which chunks idled."""

    def __init__(self, first, n, count=1):
        self.first, self.n, self.count = first, n, count
        self.seen, self.idle = [], []
        self.regs = [None] * count                 # regs[j]: output of local chunk j at the previous step

    def input_buffers(self):
        return torch.empty(self.n, dtype=torch.float32), torch.empty(3, dtype=torch.int32)

    def step(self, x, y, idle_first=0):
        self.idle.append(idle_first)
        if idle_first == 0:
            self.seen.append((x.clone(), y.clone()))
        new = []
        for j in range(self.count):
            src = x if j == 0 else self.regs[j - 1]
            new.append(None if (src is None or j < idle_first) else src * 2 + (self.first + j + 1))
        self.regs = new
        last = new[-1]
        return torch.tensor([float(x.sum())]), (last if last is not None else torch.zeros(self.n))


def _rank_main(rank, world, port, steps, out, ranges=None):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        first, count = ranges[rank] if ranges else (rank, 1)
        K = sum(c for _, c in ranges) if ranges else world
        stage = FakeStage(first, 4, count)
        pipe = P.ChunkPerGpuPipeline(stage, rank, world, dist, n_minibatches=steps, first=first, count=count)
        idle = []
        for t in range(steps + K - 1):
            x = torch.full((4,), float(t)) if rank == 0 else None
            y = torch.full((3,), t, dtype=torch.int32) if rank == 0 else None
            idle.append(pipe.step(x, y) is None)
        pipe.drain()
        out.put((rank, idle, [(float(x[0]), int(y[0])) for x, y in stage.seen], stage.idle))
    finally:
        dist.destroy_process_group()


def test_three_ranks_hand_on_activations_and_labels():
    world, steps = 3, 6
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    port = 31500 + os.getpid() % 2000
    procs = [ctx.Process(target=_rank_main, args=(r, world, port, steps, out)) for r in range(world)]
    for p in procs:
        p.start()
    res = {}
    for _ in range(world):
        r, idle, seen, _ = out.get(timeout=60)
        res[r] = (idle, seen)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    for r in range(world):
        idle, seen = res[r]
        assert idle == [t < r or t >= steps + r for t in range(steps + world - 1)]   # ramp-up and drain
        assert len(seen) == steps                                  # every rank sees every minibatch
        for i, (x0, y0) in enumerate(seen):
            t = r + i                                              # iteration; the minibatch is t - r
            want = float(t - r)
            for q in range(r):                                     # through the chunks before this one
                want = 2 * want + (q + 1)
            assert x0 == want and y0 == t - r, (r, t, x0, y0)


def test_uneven_ranges_of_chunks_per_rank():
    """Seven chunks on three ranks as (2, 1, 4): every rank's first chunk sees every minibatch with its labels, one
    iteration after the chunk before it; a rank is busy from its first chunk's first minibatch to its last chunk's
    last; while the pipeline drains the rank tells its stage how many of its leading chunks idle."""
    ranges, steps = [(0, 2), (2, 1), (3, 4)], 5
    world, K = len(ranges), 7
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    port = 33500 + os.getpid() % 2000
    procs = [ctx.Process(target=_rank_main, args=(r, world, port, steps, out, ranges)) for r in range(world)]
    for p in procs:
        p.start()
    res = {}
    for _ in range(world):
        r, idle, seen, drained = out.get(timeout=60)
        res[r] = (idle, seen, drained)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    for r, (first, count) in enumerate(ranges):
        idle, seen, drained = res[r]
        assert idle == [t < first or t >= steps + first + count - 1 for t in range(steps + K - 1)]
        assert len(seen) == steps
        for i, (x0, y0) in enumerate(seen):                        # minibatch i reaches chunk `first` at iteration first + i
            want = float(i)
            for q in range(first):
                want = 2 * want + (q + 1)
            assert x0 == want and y0 == i, (r, i, x0, y0)
        # busy steps s = 0 .. steps + count - 2; from s = steps on, s - steps + 1 leading chunks idle
        assert drained == [max(0, s - steps + 1) for s in range(steps + count - 1)]


# ----------------------------------------------------------------------------- one GPU, ranks emulated in turn

LOSS_TOL = {"fp32": 1e-4, "bf16": 2e-2}
W_TOL = {"fp32": 1e-3, "bf16": 2e-2}
V_TOL = {"fp32": 1e-3, "bf16": 2e-1}


def run_emulated(cfg, steps, w_tol=None, v_tol=None):
    from tests import lp_testlib as T
    from oracle.local_step import LocalUpdateOracle
    K = lp_synth.num_chunks(cfg)
    params = lp_synth.init_params(cfg)
    stages = [P.ChunkStage(cfg, r, params) for r in range(K)]
    orc = LocalUpdateOracle(cfg, params, dtype=np.float32, ramp="idle")
    dev = torch.device("cuda:0")
    mail = [None] * (K + 1)                       # mail[r]: what rank r-1 handed on at the previous iteration
    gl, ol = [], []
    for t in range(steps):
        x, y = lp_synth.minibatch(cfg, t)
        ol.append(orc.step(x, y, "pipelined"))
        xt = torch.from_numpy(x).to(dev)
        if cfg["family"] != "lm" and cfg["dtype"] == "bf16":
            xt = xt.to(torch.bfloat16)
        yt = torch.from_numpy(y).to(dev).contiguous()
        row = np.full(K, np.nan)
        for r in reversed(range(K)):              # rank r reads what r-1 produced one iteration earlier
            src = (xt.contiguous(), yt) if r == 0 else mail[r]
            if src is None:
                continue
            loss, out = stages[r].step(src[0], src[1])
            row[r] = float(loss.cpu()[0])
            mail[r + 1] = (out.clone(), src[1].clone())
        gl.append(row)
    gl, ol = np.array(gl), np.array(ol)
    assert np.array_equal(np.isnan(gl), np.isnan(ol))            # the same chunks idle on both sides
    assert np.isnan(gl[0, 1:]).all() and not np.isnan(gl[K - 1]).any()
    act = ~np.isnan(ol)
    dt = cfg["dtype"]
    lerr = np.abs(gl[act] - ol[act]) / np.abs(ol[act])
    worst = {"matrix": (0.0, ""), "vector": (0.0, "")}
    for r in range(K):
        got = stages[r].get_params()
        assert set(got) == set(orc.names_of_chunk[r])
        for n, a in got.items():
            if n in orc.buffers:
                continue
            a = T.strip_key_bias(n, a.astype(np.float64))
            b = T.strip_key_bias(n, orc.p[n].astype(np.float64))
            i0 = T.strip_key_bias(n, np.asarray(params[n], dtype=np.float64))
            e = np.linalg.norm(a - b)
            kind = "matrix" if got[n].ndim >= 2 else "vector"
            den = np.linalg.norm(b) if kind == "matrix" else np.linalg.norm(b - i0)
            worst[kind] = max(worst[kind], (e / max(den, 1e-30), n))
        stages[r].close()
    print("chunk per GPU, emulated:", cfg["family"], dt, "loss rel err", f"{lerr.max():.2e}", "weights", worst)
    assert lerr.max() <= LOSS_TOL[dt]
    assert worst["matrix"][0] <= (w_tol or W_TOL[dt]), worst
    assert worst["vector"][0] <= (v_tol or V_TOL[dt]), worst


def run_emulated_ranges(cfg, ranges, n, w_tol=None, v_tol=None):
    """Ranks that hold several consecutive chunks, through a whole run of n minibatches including the drain: chunk k
    trains on minibatch t - k at iteration t and stops after minibatch n - 1.  The oracle's pipelined schedule with
    idle ramp-up is stepped alongside (it has no drain: it is fed further minibatches, and chunk k's parameters
    are taken right after its n-th update, which nothing later in the chain can have influenced, Sec. 3)."""
    from tests import lp_testlib as T
    from oracle.local_step import LocalUpdateOracle
    K = lp_synth.num_chunks(cfg)
    assert sum(c for _, c in ranges) == K
    params = lp_synth.init_params(cfg)
    stages = [P.ChunkStage(cfg, f, params, c) for f, c in ranges]
    orc = LocalUpdateOracle(cfg, params, dtype=np.float32, ramp="idle")
    dev = torch.device("cuda:0")
    mail = [None] * (len(ranges) + 1)
    snap = {}
    dt = cfg["dtype"]
    worst_loss = 0.0

    def to_dev(x, y):
        xt = torch.from_numpy(x).to(dev)
        if cfg["family"] != "lm" and dt == "bf16":
            xt = xt.to(torch.bfloat16)
        return xt.contiguous(), torch.from_numpy(y).to(dev).contiguous()

    for t in range(n + K - 1):
        x, y = lp_synth.minibatch(cfg, t)
        ol = orc.step(x, y, "pipelined")
        k_done = t - n + 1                                   # this chunk has just made its n-th update
        if 0 <= k_done < K:
            snap.update({name: orc.p[name].copy() for name in orc.names_of_chunk[k_done]})
        for r in reversed(range(len(ranges))):
            first, count = ranges[r]
            s_ = t - first
            if s_ < 0 or s_ >= n + count - 1:
                continue
            if r == 0:
                src = to_dev(*lp_synth.minibatch(cfg, min(t, n - 1)))      # stale once the first chunk idles
            else:
                src = mail[r]
            loss, out = stages[r].step(src[0], src[1], max(0, s_ - n + 1))
            lv = loss.cpu().numpy().astype(np.float64)
            for j in range(count):
                k = first + j
                active = 0 <= t - k < n
                assert np.isnan(lv[j]) == (not active), (t, k, lv)
                if active:
                    worst_loss = max(worst_loss, abs(lv[j] - ol[k]) / abs(ol[k]))
            if count - 1 <= s_ < count - 1 + n:              # the last chunk trained: hand its output on
                m = t - (first + count - 1)
                mail[r + 1] = (out.clone(), to_dev(*lp_synth.minibatch(cfg, m))[1])
    worst = {"matrix": (0.0, ""), "vector": (0.0, "")}
    for r, (first, count) in enumerate(ranges):
        got = stages[r].get_params()
        assert set(got) == {nm for k in range(first, first + count) for nm in orc.names_of_chunk[k]}
        for nm, a in got.items():
            if nm in orc.buffers:
                continue
            a = T.strip_key_bias(nm, a.astype(np.float64))
            b = T.strip_key_bias(nm, snap[nm].astype(np.float64))
            i0 = T.strip_key_bias(nm, np.asarray(params[nm], dtype=np.float64))
            e = np.linalg.norm(a - b)
            kind = "matrix" if got[nm].ndim >= 2 else "vector"
            den = np.linalg.norm(b) if kind == "matrix" else np.linalg.norm(b - i0)
            worst[kind] = max(worst[kind], (e / max(den, 1e-30), nm))
        stages[r].close()
    print("ranges of chunks per GPU, emulated:", cfg["family"], dt, ranges, "loss rel err", f"{worst_loss:.2e}", "weights", worst)
    assert worst_loss <= LOSS_TOL[dt]
    assert worst["matrix"][0] <= (w_tol or W_TOL[dt]), worst
    assert worst["vector"][0] <= (v_tol or V_TOL[dt]), worst


@pytest.mark.gpu
def test_emulated_ranges_mlp_fp32_with_drain():
    cfg = lp_synth.config("c1", batch=37, d_in=50, chunks=[[48], [40, 33], [48], [24], [40], [32]], classes=7,
                          optim=dict(kind="adam", lr=1e-3, beta1=0.9, beta2=0.999, eps=1e-8))
    run_emulated_ranges(cfg, [(0, 2), (2, 1), (3, 3)], 6)


@pytest.mark.gpu
def test_emulated_ranges_lm_bf16_with_drain():
    cfg = lp_synth.config("c3", batch=2, seq_len=72, vocab=512, d_model=128, n_heads=2, d_ffn=256,
                          blocks_per_chunk=[1, 1, 2, 1, 1])
    run_emulated_ranges(cfg, [(0, 3), (3, 2)], 5)


@pytest.mark.gpu
def test_emulated_ranges_resnet_fp32_with_drain():
    cfg = lp_synth.config("c4", dtype="fp32", batch=6, height=16, width=16, stem_channels=8,
                          stage_channels=[8, 12, 16, 24], blocks_per_stage=1, classes=5)
    run_emulated_ranges(cfg, [(0, 1), (1, 3)], 5, w_tol=5e-3, v_tol=5e-2)


@pytest.mark.gpu
def test_emulated_ranks_mlp_fp32_adam():
    cfg = lp_synth.config("c1", batch=37, d_in=50, chunks=[[48], [40, 33], [48], [24]], classes=7,
                          optim=dict(kind="adam", lr=1e-3, beta1=0.9, beta2=0.999, eps=1e-8))
    run_emulated(cfg, 8)


@pytest.mark.gpu
def test_emulated_ranks_lm_fp32():
    cfg = lp_synth.config("c3", dtype="fp32", batch=3, seq_len=24, vocab=96, d_model=128, n_heads=2, d_ffn=160,
                          blocks_per_chunk=[1, 2, 1])
    run_emulated(cfg, 8)


@pytest.mark.gpu
def test_emulated_ranks_lm_bf16():
    cfg = lp_synth.config("c3", batch=4, seq_len=64, vocab=512, d_model=128, n_heads=2, d_ffn=256,
                          blocks_per_chunk=[1, 1, 1])
    run_emulated(cfg, 8)


@pytest.mark.gpu
def test_emulated_ranks_resnet_fp32():
    cfg = lp_synth.config("c4", dtype="fp32", batch=6, height=12, width=12, stem_channels=8,
                          stage_channels=[8, 16, 24], blocks_per_stage=2, classes=5)
    run_emulated(cfg, 8, w_tol=5e-3, v_tol=5e-2)


@pytest.mark.gpu
def test_emulated_ranks_resnet_bf16():
    cfg = lp_synth.config("c4", batch=32, height=16, width=16, stem_channels=64,
                          stage_channels=[64, 128], blocks_per_stage=2, classes=10)
    run_emulated(cfg, 8, v_tol=0.3)


@pytest.mark.gpu
def test_chunk_output_needs_a_step_and_a_large_enough_buffer():
    from paper_2012_03837_b200 import binding as B
    cfg = SMALL["mlp"]
    st = P.ChunkStage(cfg, 1, lp_synth.init_params(cfg))
    nbytes = B.lp_chunk_output_bytes(st.h, 0)
    assert nbytes == cfg["batch"] * cfg["chunks"][1][-1] * 4 and B.lp_chunk_output_bytes(st.h, 1) == 0
    buf = torch.empty(nbytes // 4, dtype=torch.float32, device="cuda:0")
    with pytest.raises(B.LpError):
        B.lp_chunk_output(st.h, 0, buf, nbytes)                   # no step yet
    x = torch.randn(cfg["batch"], cfg["chunks"][0][-1], device="cuda:0")
    y = torch.zeros(cfg["batch"], dtype=torch.int32, device="cuda:0")
    st.step(x, y)
    with pytest.raises(B.LpError):
        B.lp_chunk_output(st.h, 0, buf, nbytes - 4)
    with pytest.raises(B.LpError):
        B.lp_chunk_output(st.h, 1, buf, nbytes)
    B.lp_chunk_output(st.h, 0, buf, nbytes)
    torch.cuda.synchronize()
    assert torch.isfinite(buf).all() and (buf >= 0).all()          # the output of a ReLU layer
    st.close()
