"""Pins for the oracle's local update step (Sec. 3, Sec. 6): K=1 is back-propagation, the last
chunk's gradients are back-propagation's, finite differences with the chunk input frozen,
independence of the chunks, schedule agreement, pipeline data flow."""
import math

import numpy as np
import pytest
import torch
import torch.nn.functional as F

import lp_synth
from oracle.local_step import LocalUpdateOracle

TINY = {
    "mlp": lp_synth.config("c1", batch=6, d_in=7, chunks=[[6], [5, 4], [6]], classes=5),
    "lm": lp_synth.config("c3", batch=2, seq_len=5, vocab=11, d_model=8, n_heads=2, d_ffn=12,
                          blocks_per_chunk=[1, 2, 1]),
    "resnet": lp_synth.config("c4", batch=3, height=4, width=4, stem_channels=4,
                              stage_channels=[4, 6], blocks_per_stage=2, classes=3),
    # bottleneck blocks (1x1 - 3x3 - 1x1, four times the inner width out), two then one block per stage
    "bottleneck": lp_synth.config("c4", batch=3, height=4, width=4, stem_channels=4, block="bottleneck",
                                  stage_channels=[2, 3], blocks_per_stage=[2, 1], classes=3),
}
FAMS = ["mlp", "lm", "resnet", "bottleneck"]


def one_chunk(cfg):
    c = lp_synth.config(cfg["name"], **{k: v for k, v in cfg.items() if k not in ("name",)})
    if cfg["family"] == "mlp":
        c["chunks"] = [[w for ch in cfg["chunks"] for w in ch]]
    elif cfg["family"] == "lm":
        c["blocks_per_chunk"] = [sum(cfg["blocks_per_chunk"])]
    return c


def spread_params(cfg, seed=5):
    """Initial parameters with every tensor perturbed so that no gradient is trivially zero."""
    p = lp_synth.init_params(dict(cfg, dtype="fp32"))
    g = np.random.default_rng(seed)
    return {n: (a.astype(np.float64) + 0.3 * g.standard_normal(a.shape)) for n, a in p.items()}


# ---------------------------------------------------------------- independent reverse mode (torch)

def torch_forward(cfg, P, x, upto=None):
    """The same networks written with torch's own operators; returns the trunk output after
    chunk `upto` (default: the last).  P maps oracle parameter names to torch tensors."""
    fam = cfg["family"]
    K = lp_synth.num_chunks(cfg)
    upto = K - 1 if upto is None else upto
    if fam == "mlp":
        h = x
        for k in range(upto + 1):
            for i in range(len(cfg["chunks"][k])):
                h = F.relu(F.linear(h, P[f"c{k}.l{i}.W"], P[f"c{k}.l{i}.b"]))
        return h
    if fam == "lm":
        d, H = cfg["d_model"], cfg["n_heads"]
        B, T = x.shape
        h = P["c0.tok"][x] + P["c0.pos"][None]
        blk = 0
        for k in range(upto + 1):
            for _ in range(cfg["blocks_per_chunk"][k]):
                n = f"c{k}.b{blk}"
                a = F.layer_norm(h, (d,), P[n + ".ln1.g"], P[n + ".ln1.b"], 1e-5)
                qkv = F.linear(a, P[n + ".Wqkv"], P[n + ".bqkv"])
                q, kk, v = (t.reshape(B, T, H, d // H).transpose(1, 2) for t in qkv.split(d, dim=-1))
                o = F.scaled_dot_product_attention(q, kk, v, is_causal=True)
                h = h + F.linear(o.transpose(1, 2).reshape(B, T, d), P[n + ".Wo"], P[n + ".bo"])
                a = F.layer_norm(h, (d,), P[n + ".ln2.g"], P[n + ".ln2.b"], 1e-5)
                h = h + F.linear(F.gelu(F.linear(a, P[n + ".W1"], P[n + ".b1"])), P[n + ".W2"], P[n + ".b2"])
                blk += 1
        return h
    h = x
    for k in range(upto + 1):
        if k == 0:
            h = F.relu(F.batch_norm(F.conv2d(h, P["c0.stem.conv"], padding=1), None, None,
                                    P["c0.stem.bn.g"], P["c0.stem.bn.b"], True, 0.1, 1e-5))
        for j in range(lp_synth.resnet_stage_blocks(cfg, k)):
            n = f"c{k}.r{j}"
            s = lp_synth.resnet_stage_stride(cfg, k) if j == 0 else 1
            bn = lambda t, m: F.batch_norm(t, None, None, P[m + ".g"], P[m + ".b"], True, 0.1, 1e-5)
            if cfg.get("block") == "bottleneck":
                u = F.relu(bn(F.conv2d(h, P[n + ".conv1"]), n + ".bn1"))
                u = F.relu(bn(F.conv2d(u, P[n + ".conv2"], stride=s, padding=1), n + ".bn2"))
                u = bn(F.conv2d(u, P[n + ".conv3"]), n + ".bn3")
                sc = bn(F.conv2d(h, P[n + ".sc.conv"], stride=s), n + ".sc.bn") if n + ".sc.conv" in P else h
                h = F.relu(u + sc)
                continue
            u = F.conv2d(h, P[n + ".conv1"], stride=s, padding=1)
            u = F.relu(F.batch_norm(u, None, None, P[n + ".bn1.g"], P[n + ".bn1.b"], True, 0.1, 1e-5))
            u = F.conv2d(u, P[n + ".conv2"], padding=1)
            u = F.batch_norm(u, None, None, P[n + ".bn2.g"], P[n + ".bn2.b"], True, 0.1, 1e-5)
            if n + ".sc.conv" in P:
                sc = F.conv2d(h, P[n + ".sc.conv"], stride=s)
                sc = F.batch_norm(sc, None, None, P[n + ".sc.bn.g"], P[n + ".sc.bn.b"], True, 0.1, 1e-5)
            else:
                sc = h
            h = F.relu(u + sc)
    return h


def torch_head_loss(cfg, P, k, h, y, bn_buffers=None, bn_training=True):
    """bn_buffers: (running means, running variances) by BatchNorm name, for the BatchNorm of App. B.3's head."""
    fam = cfg["family"]
    if fam == "lm":
        a = F.layer_norm(h, (cfg["d_model"],), P[f"c{k}.head.ln.g"], P[f"c{k}.head.ln.b"], 1e-5)
        z = F.linear(a, P[f"c{k}.head.W"], P[f"c{k}.head.b"])
        return F.cross_entropy(z.reshape(-1, z.shape[-1]), y.reshape(-1).long(), ignore_index=-1)
    if fam == "resnet":
        if cfg.get("head") == "bn_relu_gap":
            m = f"c{k}.head.bn"
            rm, rv = (bn_buffers[0][m], bn_buffers[1][m]) if bn_buffers else (None, None)
            h = F.relu(F.batch_norm(h, rm, rv, P[m + ".g"], P[m + ".b"], bn_training, 0.1, 1e-5))
        h = h.mean(dim=(2, 3))
    return F.cross_entropy(F.linear(h, P[f"c{k}.head.W"], P[f"c{k}.head.b"]), y.long())


def torch_backprop_grads(cfg, params, x, y, head_chunk):
    """Ordinary full back-propagation of the loss of head `head_chunk` through everything below."""
    P = {n: torch.tensor(a, dtype=torch.float64, requires_grad=True) for n, a in params.items()}
    xt = torch.tensor(x) if cfg["family"] == "lm" else torch.tensor(x, dtype=torch.float64)
    h = torch_forward(cfg, P, xt, upto=head_chunk)
    loss = torch_head_loss(cfg, P, head_chunk, h, torch.tensor(y))
    loss.backward()
    return float(loss.detach()), {n: (None if t.grad is None else t.grad.numpy()) for n, t in P.items()}


def rel(a, b):
    return np.abs(a - b).max() / max(np.abs(b).max(), 1e-30)


# ---------------------------------------------------------------- P1: K = 1 is back-propagation

@pytest.mark.parametrize("fam", FAMS)
def test_single_chunk_equals_backprop(fam):
    cfg = TINY[fam]
    if fam in ("resnet", "bottleneck"):
        cfg = lp_synth.config("c4", **{k: v for k, v in cfg.items() if k != "name"})
        cfg["stage_channels"] = cfg["stage_channels"][:1]      # a ResNet chunk is a stage: one stage = one chunk
    else:
        cfg = one_chunk(cfg)
    params = spread_params(cfg)
    x, y = lp_synth.minibatch(cfg, 0)
    orc = LocalUpdateOracle(cfg, params, dtype=np.float64)
    loss, _, grads = orc.local_grads(0, orc._cast_input(x), y)
    tloss, tg = torch_backprop_grads(cfg, params, x, y, 0)
    assert abs(loss - tloss) < 1e-10 * max(1, abs(tloss))
    for n in params:
        if n in orc.buffers:               # running statistics: no gradient reaches them
            continue
        assert tg[n] is not None, n
        assert rel(grads[n], tg[n]) < 1e-9, n


# ---------------------------------------------------------------- P2: last chunk = backprop's gradient

@pytest.mark.parametrize("fam", FAMS)
def test_last_chunk_gradients_are_backprop_gradients(fam):
    cfg = TINY[fam]
    K = lp_synth.num_chunks(cfg)
    params = spread_params(cfg)
    x, y = lp_synth.minibatch(cfg, 0)
    orc = LocalUpdateOracle(cfg, params, dtype=np.float64)
    orc.cfg = dict(cfg, optim=dict(kind="sgdm", lr=0.0, momentum=0.0, weight_decay=0.0))
    orc.step(x, y, "sync")
    _, tg = torch_backprop_grads(cfg, params, x, y, K - 1)
    for n in orc.names_of_chunk[K - 1]:
        if n in orc.buffers:
            continue
        assert rel(orc.last_grads[n], tg[n]) < 1e-9, n
    # ... and an earlier chunk's local gradient is NOT the gradient of the last loss (Sec. 1)
    n0 = orc.names_of_chunk[0][0]
    assert rel(orc.last_grads[n0], tg[n0]) > 1e-3


# ---------------------------------------------------------------- P3: finite differences, input frozen

@pytest.mark.parametrize("fam", FAMS)
def test_local_gradients_match_finite_differences(fam):
    cfg = TINY[fam]
    K = lp_synth.num_chunks(cfg)
    params = spread_params(cfg, seed=9)
    x, y = lp_synth.minibatch(cfg, 0)
    orc = LocalUpdateOracle(cfg, params, dtype=np.float64)
    inp = orc._cast_input(x)
    rng = np.random.default_rng(0)
    for k in range(K):
        loss, h, grads = orc.local_grads(k, inp, y)
        for n in orc.names_of_chunk[k]:
            if n in orc.buffers:               # running statistics do not enter the training loss
                continue
            w = orc.p[n]
            flat = w.reshape(-1)
            for idx in rng.choice(flat.size, size=min(4, flat.size), replace=False):
                old = flat[idx]
                eps = 1e-6
                flat[idx] = old + eps
                lp = orc.local_grads(k, inp, y)[0]
                flat[idx] = old - eps
                lm = orc.local_grads(k, inp, y)[0]
                flat[idx] = old
                fd = (lp - lm) / (2 * eps)
                an = grads[n].reshape(-1)[idx]
                assert abs(fd - an) <= 2e-6 * max(1.0, abs(fd), np.abs(grads[n]).max()), (n, idx, fd, an)
        inp = h


# ---------------------------------------------------------------- P4: chunks are independent

@pytest.mark.parametrize("fam", FAMS)
def test_chunk_update_ignores_other_chunks_heads_and_losses(fam):
    cfg = TINY[fam]
    K = lp_synth.num_chunks(cfg)
    params = spread_params(cfg)
    x, y = lp_synth.minibatch(cfg, 0)
    a = LocalUpdateOracle(cfg, params, dtype=np.float64)
    a.step(x, y, "sync")
    for k in range(K - 1):
        p2 = {n: v.copy() for n, v in params.items()}
        for j in range(k + 1, K):          # later chunks: different heads (hence different losses)
            p2[f"c{j}.head.W"] = p2[f"c{j}.head.W"] * -3.0 + 1.0
        b = LocalUpdateOracle(cfg, p2, dtype=np.float64)
        b.step(x, y, "sync")
        for n in a.names_of_chunk[k]:
            assert np.array_equal(a.p[n], b.p[n]), n
            if n not in a.buffers:
                assert np.array_equal(a.last_grads[n], b.last_grads[n]), n


def test_stop_gradient_is_real():
    """The local gradient of chunk 0 differs from d(sum of all losses)/d(theta_0): later losses do
    depend on theta_0 through the forward pass, but that path is cut (Sec. 3, greedy)."""
    cfg = TINY["mlp"]
    params = spread_params(cfg)
    x, y = lp_synth.minibatch(cfg, 0)
    orc = LocalUpdateOracle(cfg, params, dtype=np.float64)
    orc.cfg = dict(cfg, optim=dict(kind="sgdm", lr=0.0, momentum=0.0, weight_decay=0.0))
    orc.step(x, y, "sync")
    n = "c0.l0.W"
    w = orc.p[n]
    idx = (1, 2)
    tot = lambda: float(orc.forward(x, y)[1].sum())
    old = w[idx]
    w[idx] = old + 1e-6; fp = tot()
    w[idx] = old - 1e-6; fm = tot()
    w[idx] = old
    fd_total = (fp - fm) / 2e-6
    first = lambda: float(orc.forward(x, y)[1][0])
    w[idx] = old + 1e-6; fp = first()
    w[idx] = old - 1e-6; fm = first()
    w[idx] = old
    fd_first = (fp - fm) / 2e-6
    g = orc.last_grads[n][idx]
    assert abs(g - fd_first) < 1e-6 * max(1, abs(g))
    assert abs(g - fd_total) > 1e-3 * max(1e-3, abs(g))


# ---------------------------------------------------------------- P5: schedules

@pytest.mark.parametrize("fam", FAMS)
def test_sync_and_pipelined_agree_on_step0(fam):
    cfg = TINY[fam]
    params = spread_params(cfg)
    x, y = lp_synth.minibatch(cfg, 0)
    a = LocalUpdateOracle(cfg, params, dtype=np.float64)
    b = LocalUpdateOracle(cfg, params, dtype=np.float64)
    la = a.step(x, y, "sync")
    lb = b.step(x, y, "pipelined")
    assert np.array_equal(la, lb)
    for n in a.p:
        assert np.array_equal(a.p[n], b.p[n]), n


def test_pipelined_chunk_k_sees_minibatch_t_minus_k_with_its_labels():
    cfg = TINY["mlp"]
    K = lp_synth.num_chunks(cfg)
    params = spread_params(cfg)
    orc = LocalUpdateOracle(cfg, params, dtype=np.float64)
    orc.cfg = dict(cfg, optim=dict(kind="sgdm", lr=0.0, momentum=0.0, weight_decay=0.0))
    frozen = LocalUpdateOracle(cfg, params, dtype=np.float64)
    batches = [lp_synth.minibatch(cfg, t) for t in range(6)]
    for t, (x, y) in enumerate(batches):
        losses = orc.step(x, y, "pipelined")
        for k in range(K):
            src = max(t - k, 0)                # with frozen weights the loss identifies the batch
            exp = frozen.forward(*batches[src])[1][k]
            assert abs(losses[k] - exp) < 1e-12, (t, k)


def test_pipelined_idle_rampup():
    cfg = TINY["mlp"]
    K = lp_synth.num_chunks(cfg)
    orc = LocalUpdateOracle(cfg, spread_params(cfg), dtype=np.float64, ramp="idle")
    for t in range(K + 1):
        losses = orc.step(*lp_synth.minibatch(cfg, t), "pipelined")
        assert [bool(np.isfinite(v)) for v in losses] == [k <= t for k in range(K)]


def test_forward_chain_uses_start_of_step_weights():
    """One forward per chunk per step, all with the weights the step began with (App. A.2, greedy:
    one forward and one backward pass per layer per step)."""
    cfg = TINY["mlp"]
    params = spread_params(cfg)
    x, y = lp_synth.minibatch(cfg, 0)
    orc = LocalUpdateOracle(cfg, params, dtype=np.float64)
    before = orc.forward(x, y)[1]
    losses = orc.step(x, y, "sync")
    assert np.allclose(losses, before, rtol=0, atol=1e-13)


# ---------------------------------------------------------------- P6, P12

def test_initial_lm_loss_is_log_vocab():
    cfg = lp_synth.config("c3", batch=2, seq_len=16, vocab=512, d_model=32, n_heads=2, d_ffn=64,
                          blocks_per_chunk=[1, 1])
    orc = LocalUpdateOracle(cfg, lp_synth.init_params(cfg), dtype=np.float64)
    losses = orc.forward(*lp_synth.minibatch(cfg, 0))[1]
    assert np.all(np.abs(losses - math.log(512)) < 5e-2)   # 30 valid rows: sampling noise ~1e-2


def test_determinism_and_dtype_modes():
    cfg = TINY["lm"]
    outs = []
    for _ in range(2):
        orc = LocalUpdateOracle(cfg, lp_synth.init_params(cfg), dtype=np.float32)
        ls = [orc.step(*lp_synth.minibatch(cfg, t)) for t in range(3)]
        outs.append((np.array(ls), {n: v.copy() for n, v in orc.p.items()}))
    assert np.array_equal(outs[0][0], outs[1][0])
    for n in outs[0][1]:
        assert np.array_equal(outs[0][1][n], outs[1][1][n])
        assert outs[0][1][n].dtype == np.float32
    o64 = LocalUpdateOracle(cfg, lp_synth.init_params(cfg), dtype=np.float64)
    l64 = np.array([o64.step(*lp_synth.minibatch(cfg, t)) for t in range(3)])
    assert np.allclose(outs[0][0], l64, rtol=1e-5)


def test_key_bias_gradient_is_identically_zero():
    """Softmax is invariant to a shift common to all scores of a row, so the key bias of an attention
    layer has zero gradient: what an fp32 run stores there is rounding noise (parity tests skip it)."""
    cfg = TINY["lm"]
    params = spread_params(cfg)
    orc = LocalUpdateOracle(cfg, params, dtype=np.float64)
    x, y = lp_synth.minibatch(cfg, 0)
    orc.cfg = dict(cfg, optim=dict(kind="sgdm", lr=0.0, momentum=0.0, weight_decay=0.0))
    orc.step(x, y, "sync")
    d = cfg["d_model"]
    for n, g in orc.last_grads.items():
        if n.endswith(".bqkv"):
            assert np.abs(g[d:2 * d]).max() < 1e-12 * np.abs(g[:d]).max()


def test_evaluate_counts_follow_the_logits_and_ties_take_the_lowest_index():
    """evaluate(): the prediction is the first largest logit; labels of -1 are not counted; the losses equal
    forward()'s.  A head with all-zero weights makes every logit equal, so every row predicts class 0."""
    cfg = lp_synth.config("c3", dtype="fp32", batch=2, seq_len=12, vocab=17, d_model=64, n_heads=1, d_ffn=32,
                          blocks_per_chunk=[1, 1])
    params = lp_synth.init_params(cfg)
    params["c1.head.W"] = np.zeros_like(params["c1.head.W"])
    orc = LocalUpdateOracle(cfg, params, dtype=np.float64)
    x, y = lp_synth.minibatch(cfg, 0)
    ev = orc.evaluate(x, y)
    _, losses = orc.forward(x, y)
    lab = y.reshape(-1)
    assert (lab == -1).sum() == cfg["batch"]                       # the last position of every sequence
    for k, r in enumerate(ev):
        assert abs(r["loss"] - losses[k]) < 1e-12
        brute = np.array([max(range(17), key=lambda c: (row[c], -c)) for row in r["logits"]])
        assert np.array_equal(r["pred"], brute)
        assert r["correct"] == sum(int(p == t) for p, t in zip(r["pred"], lab) if t >= 0)
    assert np.all(ev[1]["pred"] == 0)
    assert ev[1]["correct"] == int(np.sum(lab == 0))


def test_batchnorm_running_statistics_and_evaluation_mode_follow_the_library_routine():
    """BatchNorm's running mean / variance after training steps, and the evaluation-mode forward that uses
    them, against torch.nn.functional.batch_norm (momentum 0.1, unbiased variance in the running average);
    plus the closed form after one step from (0, 1): 0.1 * batch mean and 0.9 + 0.1 * n/(n-1) * batch variance."""
    cfg = lp_synth.config("c4", dtype="fp32", batch=4, height=6, width=6, stem_channels=4, stage_channels=[4, 8],
                          blocks_per_stage=1, classes=3)
    params = spread_params(cfg)
    for n in params:                       # the running statistics start from (0, 1)
        if n.endswith(".rm"):
            params[n] = np.zeros_like(params[n])
        if n.endswith(".rv"):
            params[n] = np.ones_like(params[n])
    orc = LocalUpdateOracle(cfg, params, dtype=np.float64)
    P = {n: torch.tensor(a, dtype=torch.float64) for n, a in params.items()}
    orc.cfg = dict(cfg, optim=dict(kind="sgdm", lr=0.0, momentum=0.0, weight_decay=0.0))   # weights stay put
    x0, y0 = lp_synth.minibatch(cfg, 0)
    # closed form for the stem after one step
    u = F.conv2d(torch.tensor(x0, dtype=torch.float64), P["c0.stem.conv"], padding=1).numpy()
    n = u.shape[0] * u.shape[2] * u.shape[3]
    orc.step(x0, y0, "sync")
    assert np.allclose(orc.p["c0.stem.bn.rm"], 0.1 * u.mean(axis=(0, 2, 3)), rtol=1e-12, atol=1e-14)
    assert np.allclose(orc.p["c0.stem.bn.rv"], 0.9 + 0.1 * u.var(axis=(0, 2, 3)) * n / (n - 1), rtol=1e-12)
    # two more steps, then every BatchNorm against the library's running buffers
    for t in (1, 2):
        orc.step(*lp_synth.minibatch(cfg, t), "sync")
    rm = {m[:-3]: torch.zeros(params[m].shape, dtype=torch.float64) for m in params if m.endswith(".rm")}
    rv = {m: torch.ones_like(v) for m, v in rm.items()}

    def torch_pass(xt, training):
        bn = lambda v, m: F.batch_norm(v, rm[m], rv[m], P[m + ".g"], P[m + ".b"], training, 0.1, 1e-5)
        h = F.relu(bn(F.conv2d(xt, P["c0.stem.conv"], padding=1), "c0.stem.bn"))
        outs = []
        for k in range(2):
            nm = f"c{k}.r0"
            s = lp_synth.resnet_stage_stride(cfg, k)
            v = F.relu(bn(F.conv2d(h, P[nm + ".conv1"], stride=s, padding=1), nm + ".bn1"))
            v = bn(F.conv2d(v, P[nm + ".conv2"], padding=1), nm + ".bn2")
            sc = bn(F.conv2d(h, P[nm + ".sc.conv"], stride=s), nm + ".sc.bn") if nm + ".sc.conv" in P else h
            h = F.relu(v + sc)
            outs.append(h)
        return outs
    for t in range(3):
        torch_pass(torch.tensor(lp_synth.minibatch(cfg, t)[0], dtype=torch.float64), True)
    for m in rm:
        assert rel(orc.p[m + ".rm"], rm[m].numpy()) < 1e-10, m
        assert rel(orc.p[m + ".rv"], rv[m].numpy()) < 1e-10, m
    # evaluation mode: losses from the running statistics, and nothing moves
    x3, y3 = lp_synth.minibatch(cfg, 3)
    before = {m: orc.p[m + ".rm"].copy() for m in rm}
    ev = orc.evaluate(x3, y3, bn="running")
    outs = torch_pass(torch.tensor(x3, dtype=torch.float64), False)
    for k in range(2):
        tl = float(torch_head_loss(cfg, P, k, outs[k], torch.tensor(y3)))
        assert abs(ev[k]["loss"] - tl) < 1e-10 * max(1.0, abs(tl)), k
    for m in rm:
        assert np.array_equal(before[m], orc.p[m + ".rm"])
    assert abs(orc.evaluate(x3, y3)[0]["loss"] - ev[0]["loss"]) > 1e-6      # batch statistics give another loss


def test_resnet_head_with_batchnorm_and_relu_follows_reverse_mode_and_the_library_buffers():
    """App. B.3's auxiliary head (BatchNorm -> ReLU -> spatial mean -> Linear): every chunk's local gradient,
    the head's own BatchNorm parameters included, against torch autograd of that chunk's loss with the chunk
    input detached; the head BatchNorm's running statistics and the evaluation-mode loss against torch's
    batch_norm buffers."""
    cfg = lp_synth.config("c4", dtype="fp32", batch=4, height=6, width=6, stem_channels=4, stage_channels=[4, 8],
                          blocks_per_stage=1, classes=3, head="bn_relu_gap")
    params = spread_params(cfg)
    assert "c0.head.bn.g" in params and "c1.head.bn.rv" in params
    for n in params:
        if n.endswith(".rm"):
            params[n] = np.zeros_like(params[n])
        if n.endswith(".rv"):
            params[n] = np.ones_like(params[n])
    orc = LocalUpdateOracle(cfg, params, dtype=np.float64)
    orc.cfg = dict(cfg, optim=dict(kind="sgdm", lr=0.0, momentum=0.0, weight_decay=0.0))
    x, y = lp_synth.minibatch(cfg, 0)
    orc.step(x, y, "sync")
    # chunk 1 (last): full back-propagation of its loss; chunk 0: back-propagation of head 0's loss
    for k in range(2):
        _, tg = torch_backprop_grads(cfg, params, x, y, k)
        for n in orc.names_of_chunk[k]:
            if n in orc.buffers:
                continue
            assert tg[n] is not None, n
            assert rel(orc.last_grads[n], tg[n]) < 1e-9, n
    assert np.abs(orc.last_grads["c0.head.bn.g"]).max() > 1e-6
    # running statistics of the head's BatchNorm after one step, closed form from (0, 1)
    P = {n: torch.tensor(a, dtype=torch.float64) for n, a in params.items()}
    h0 = torch_forward(cfg, P, torch.tensor(x, dtype=torch.float64), upto=0).numpy()
    n = h0.shape[0] * h0.shape[2] * h0.shape[3]
    assert np.allclose(orc.p["c0.head.bn.rm"], 0.1 * h0.mean(axis=(0, 2, 3)), rtol=1e-12, atol=1e-14)
    assert np.allclose(orc.p["c0.head.bn.rv"], 0.9 + 0.1 * h0.var(axis=(0, 2, 3)) * n / (n - 1), rtol=1e-12)
    # a forward pass or an evaluation moves nothing; evaluation on running statistics uses the head's buffers too
    before = orc.p["c1.head.bn.rm"].copy()
    orc.forward(x, y)
    x1, y1 = lp_synth.minibatch(cfg, 1)
    ev_run = orc.evaluate(x1, y1, bn="running")
    ev_bat = orc.evaluate(x1, y1)
    assert np.array_equal(before, orc.p["c1.head.bn.rm"])
    assert abs(ev_run[0]["loss"] - ev_bat[0]["loss"]) > 1e-6
    # chunk 0's evaluation loss on running statistics, rebuilt with torch from the oracle's buffers
    Pn = {n: torch.tensor(a, dtype=torch.float64) for n, a in orc.p.items()}
    bn = lambda v, m: F.batch_norm(v, Pn[m + ".rm"], Pn[m + ".rv"], Pn[m + ".g"], Pn[m + ".b"], False, 0.1, 1e-5)
    h = F.relu(bn(F.conv2d(torch.tensor(x1, dtype=torch.float64), Pn["c0.stem.conv"], padding=1), "c0.stem.bn"))
    v = F.relu(bn(F.conv2d(h, Pn["c0.r0.conv1"], padding=1), "c0.r0.bn1"))
    v = bn(F.conv2d(v, Pn["c0.r0.conv2"], padding=1), "c0.r0.bn2")
    h = F.relu(v + h)
    bufs = ({"c0.head.bn": Pn["c0.head.bn.rm"]}, {"c0.head.bn": Pn["c0.head.bn.rv"]})
    tl = float(torch_head_loss(cfg, Pn, 0, h, torch.tensor(y1), bufs, False))
    assert abs(ev_run[0]["loss"] - tl) < 1e-10 * max(1.0, abs(tl))


# ---------------------------------------------------------------- overlapping local parallelism (Sec. 3, Fig. 2 c)

@pytest.mark.parametrize("fam", FAMS)
def test_overlapping_updates_average_the_two_backprop_gradients_of_the_shared_layer(fam):
    """With overlap, the last layer (transformer: last block) of every chunk but the final one also belongs to
    the next chunk's block.  Its gradient from either loss is that loss's ordinary back-propagation gradient
    (truncating further down does not change it), so the update must use the mean of two torch autograd
    gradients; every other parameter keeps its plain local gradient."""
    cfg = TINY[fam]
    K = lp_synth.num_chunks(cfg)
    params = spread_params(cfg, seed=3)
    x, y = lp_synth.minibatch(cfg, 0)
    lr = 0.25
    sgd = dict(kind="sgdm", lr=lr, momentum=0.0, weight_decay=0.0)
    plain = LocalUpdateOracle(dict(cfg, optim=sgd), params, dtype=np.float64)
    over = LocalUpdateOracle(dict(cfg, optim=sgd), params, dtype=np.float64, overlap=True)
    lp_, lo = plain.step(x, y, "sync"), over.step(x, y, "sync")
    assert np.array_equal(lp_, lo)                      # the forward pass is shared: same losses
    tg = [torch_backprop_grads(cfg, params, x, y, k)[1] for k in range(K)]
    shared = set()
    for k in range(K - 1):
        if fam == "mlp":
            last = len(cfg["chunks"][k]) - 1
            names = [f"c{k}.l{last}.W", f"c{k}.l{last}.b"]
        elif fam == "lm":
            blk = over._lm_block_names(k)[-1]
            names = [n for n in over.names_of_chunk[k] if n.startswith(blk + ".")]
            assert len(names) == 12
        else:
            blk = f"c{k}.r{lp_synth.resnet_stage_blocks(cfg, k) - 1}"
            names = [n for n in over.names_of_chunk[k] if n.startswith(blk + ".") and n not in over.buffers]
            assert len(names) == (9 if fam == "bottleneck" else 6)
        for n in names:
            shared.add(n)
            want = 0.5 * (tg[k][n] + tg[k + 1][n])
            assert rel(over.last_grads[n], want) < 1e-9, n
            assert rel(over.last_grads[n], plain.last_grads[n]) > 1e-4, n      # and it is not the greedy gradient
            assert rel(over.p[n], params[n] - lr * want) < 1e-12, n             # the update applies the average
    for n in params:
        if n not in shared:
            if n not in over.buffers:
                assert np.array_equal(over.last_grads[n], plain.last_grads[n]), n
            assert np.array_equal(over.p[n], plain.p[n]), n


def test_overlapping_updates_need_the_synchronous_schedule():
    cfg = TINY["mlp"]
    over = LocalUpdateOracle(cfg, lp_synth.init_params(cfg), dtype=np.float64, overlap=True)
    with pytest.raises(ValueError):
        over.step(*lp_synth.minibatch(cfg, 0), "pipelined")
