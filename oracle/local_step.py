"""CPU oracle of the per-chunk local update step.  TEST INFRASTRUCTURE ONLY: plain NumPy, slow,
shares no code with the CUDA path; only tests, the smoke check and the benchmark's CPU-baseline
leg may use it.

What it computes (Sec. 3): the network is cut into a sequence of blocks ("chunks" here, K of
them); chunk k receives the output of chunk k-1 (chunk 0 the minibatch), runs its layers, feeds
the result to an auxiliary head whose loss has the same form as the global objective, and
back-propagates that loss into its own layers only.  The activation handed to the next chunk
carries no gradient (greedy / chunked local parallelism, Sec. 3; Fig. 2 b, d).  Back-propagation
is the special case of a single chunk (Sec. 3, "Backpropagation").  Every chunk then applies its
own optimizer update (Sec. 1, Sec. 6).

Schedules:
  * synchronous: all chunks train on the same minibatch; inside a chunk the forward pass runs
    before the backward pass for that same minibatch (App. E.1).  Every chunk's forward uses the
    weights the step started with, so the K updates of a step do not depend on one another.
  * pipelined (Sec. 6 and the draft Methods text on pipelining): chunk k works on the activation
    chunk k-1 produced one step earlier, for an older minibatch, and the labels of that minibatch
    travel forward with the activation.  Ramp-up: the first pipelined step fills every boundary
    buffer by a forward pass of its own minibatch with the initial weights (`ramp="prime"`), so
    that step equals a synchronous step; `ramp="idle"` instead leaves chunk k idle (no update,
    loss NaN) until real data reaches it at step k.

Overlapping local parallelism (Sec. 3; cost model in App. A.2): with overlap=True the block trained by
chunk k's loss also contains the last layer of chunk k-1 (transformer: its last block; ResNet: its last
BasicBlock), so that
loss is back-propagated one layer past the chunk boundary and stops at that layer's input.  The
shared layer exists once (one forward pass through the network); it receives two gradients, from
its own chunk's loss and from the next chunk's, and is updated with their average.  Defined for
the synchronous schedule (both gradients belong to the same minibatch).

Readings the paper leaves open are fixed here: mean loss over valid rows; LM targets are the ids
shifted left with the last position ignored; LayerNorm/BatchNorm eps 1e-5; exact (erf) GELU; no
dropout; pre-LayerNorm residual blocks; ResNet shortcut = 1x1 stride-2 convolution + BatchNorm
where the shape changes; weight decay added to the gradient of matrices and filters only.
"""
from __future__ import annotations

import numpy as np

import lp_synth
from . import layers as L
from . import optim as O


class LocalUpdateOracle:
    def __init__(self, cfg: dict, params: dict, dtype=np.float32, ramp: str = "prime", overlap: bool = False):
        self.cfg = cfg
        self.dtype = np.dtype(dtype).type
        self.K = lp_synth.num_chunks(cfg)
        self.table = lp_synth.param_table(cfg)
        self.p = {t["name"]: np.array(params[t["name"]], dtype=dtype) for t in self.table}
        self.state = {t["name"]: {} for t in self.table}
        self.names_of_chunk = [[t["name"] for t in self.table if t["chunk"] == k] for k in range(self.K)]
        self.decay = {t["name"]: t["decay"] for t in self.table}
        self.buffers = {t["name"] for t in self.table if t.get("buffer")}   # state no gradient reaches
        self.bn_mode = "batch"   # "running": BatchNorm normalises with its running statistics (evaluation)
        self.training = False    # True inside a training step: BatchNorm then updates its running statistics
        self.ramp = ramp
        self.overlap = overlap   # overlapping local parallelism (Sec. 3, Fig. 2 c): synchronous schedule only
        self.buf = None          # pipelined: buf[k] = (activation, labels) chunk k+1 reads next
        self.t = 0               # pipelined steps taken since the last reset
        self.last_grads = {}

    # ---------------------------------------------------------------- chunk forward / backward

    def chunk_forward(self, k, inp):
        """Trunk of chunk k applied to its input with the current weights: (output, cache)."""
        fam = self.cfg["family"]
        if fam == "mlp":
            return self._mlp_fwd(k, inp)
        if fam == "lm":
            return self._lm_fwd(k, inp)
        return self._resnet_fwd(k, inp)

    def chunk_backward(self, k, dout, cache):
        """Gradients of chunk k's trunk parameters given the gradient at its output.  The gradient
        with respect to the chunk input is not propagated anywhere (Sec. 3)."""
        fam = self.cfg["family"]
        if fam == "mlp":
            return self._mlp_bwd(k, dout, cache)
        if fam == "lm":
            return self._lm_bwd(k, dout, cache)
        return self._resnet_bwd(k, dout, cache)

    def head(self, k, h, y, training=False):
        """Auxiliary head of chunk k on the chunk output h: (loss, logits, dh, head gradients).  The ResNet
        head is spatial mean + Linear, or, with cfg["head"] == "bn_relu_gap", App. B.3's BatchNorm -> ReLU ->
        spatial mean -> Linear (its BatchNorm follows self.bn_mode; under running statistics dh is None)."""
        fam = self.cfg["family"]
        p = self.p
        g = {}
        if fam == "mlp":
            z, c = L.linear_fwd(h, p[f"c{k}.head.W"], p[f"c{k}.head.b"])
            loss, dz = L.softmax_xent(z, y)
            dh, g[f"c{k}.head.W"], g[f"c{k}.head.b"] = L.linear_bwd(dz, c)
        elif fam == "lm":
            b, t, d = h.shape
            a, cln = L.layernorm_fwd(h, p[f"c{k}.head.ln.g"], p[f"c{k}.head.ln.b"])
            z, c = L.linear_fwd(a.reshape(b * t, d), p[f"c{k}.head.W"], p[f"c{k}.head.b"])
            loss, dz = L.softmax_xent(z, y.reshape(-1))
            da, g[f"c{k}.head.W"], g[f"c{k}.head.b"] = L.linear_bwd(dz, c)
            dh, g[f"c{k}.head.ln.g"], g[f"c{k}.head.ln.b"] = L.layernorm_bwd(da.reshape(b, t, d), cln)
        else:
            bn_head = self.cfg.get("head") == "bn_relu_gap"
            r = h
            if bn_head:
                self.training = training
                try:
                    u, cb = self._bn(h, f"c{k}.head.bn")
                finally:
                    self.training = False
                r, cr = L.relu_fwd(u)
            a, cg = L.gap_fwd(r)
            z, c = L.linear_fwd(a, p[f"c{k}.head.W"], p[f"c{k}.head.b"])
            loss, dz = L.softmax_xent(z, y)
            da, g[f"c{k}.head.W"], g[f"c{k}.head.b"] = L.linear_bwd(dz, c)
            dh = L.gap_bwd(da, cg)
            if bn_head:
                if cb is None:
                    return loss, z, None, {}
                du = L.relu_bwd(dh, cr)
                dh, g[f"c{k}.head.bn.g"], g[f"c{k}.head.bn.b"] = L.batchnorm_bwd(du, cb)
        return loss, z, dh, g

    # MLP chunk: a run of Linear + ReLU layers (App. A.1).
    def _mlp_fwd(self, k, x):
        caches = []
        for i in range(len(self.cfg["chunks"][k])):
            u, c1 = L.linear_fwd(x, self.p[f"c{k}.l{i}.W"], self.p[f"c{k}.l{i}.b"])
            x, c2 = L.relu_fwd(u)
            caches.append((c1, c2))
        return x, caches

    def _mlp_bwd(self, k, dx, caches):
        g = {}
        for i in reversed(range(len(caches))):
            c1, c2 = caches[i]
            du = L.relu_bwd(dx, c2)
            dx, g[f"c{k}.l{i}.W"], g[f"c{k}.l{i}.b"] = L.linear_bwd(du, c1)
        self._dx_in = dx         # gradient at the chunk input: used only by the overlapping variant
        return g

    # LM chunk: (token + position embedding in chunk 0), then pre-LayerNorm transformer blocks
    # (App. B.2): h <- h + Wo Attn(LN1 h); h <- h + W2 GELU(W1 LN2 h).
    def _lm_block_names(self, k):
        first = sum(self.cfg["blocks_per_chunk"][:k])
        return [f"c{k}.b{first + j}" for j in range(self.cfg["blocks_per_chunk"][k])]

    def _lm_fwd(self, k, inp):
        p = self.p
        cache = {}
        if k == 0:
            h, cache["emb"] = L.embedding_fwd(inp, p["c0.tok"], p["c0.pos"])
        else:
            h = inp
        b, t, d = h.shape
        cache["blocks"] = []
        for n in self._lm_block_names(k):
            a1, cl1 = L.layernorm_fwd(h, p[n + ".ln1.g"], p[n + ".ln1.b"])
            qkv, cq = L.linear_fwd(a1.reshape(b * t, d), p[n + ".Wqkv"], p[n + ".bqkv"])
            o, ca = L.attention_fwd(qkv.reshape(b, t, 3 * d), self.cfg["n_heads"])
            r1, co = L.linear_fwd(o.reshape(b * t, d), p[n + ".Wo"], p[n + ".bo"])
            h = h + r1.reshape(b, t, d)
            a2, cl2 = L.layernorm_fwd(h, p[n + ".ln2.g"], p[n + ".ln2.b"])
            u, c1 = L.linear_fwd(a2.reshape(b * t, d), p[n + ".W1"], p[n + ".b1"])
            gl, cg = L.gelu_fwd(u)
            r2, c2 = L.linear_fwd(gl, p[n + ".W2"], p[n + ".b2"])
            h = h + r2.reshape(b, t, d)
            cache["blocks"].append((n, cl1, cq, ca, co, cl2, c1, cg, c2))
        return h, cache

    def _lm_block_bwd(self, dh, block_cache, g):
        """Backward of one transformer block: fills g with its parameter gradients, returns the gradient
        at the block input."""
        (n, cl1, cq, ca, co, cl2, c1, cg, c2) = block_cache
        b, t, d = dh.shape
        dgl, g[n + ".W2"], g[n + ".b2"] = L.linear_bwd(dh.reshape(b * t, d), c2)
        du = L.gelu_bwd(dgl, cg)
        da2, g[n + ".W1"], g[n + ".b1"] = L.linear_bwd(du, c1)
        dx, g[n + ".ln2.g"], g[n + ".ln2.b"] = L.layernorm_bwd(da2.reshape(b, t, d), cl2)
        dh = dh + dx
        do, g[n + ".Wo"], g[n + ".bo"] = L.linear_bwd(dh.reshape(b * t, d), co)
        dqkv = L.attention_bwd(do.reshape(b, t, d), ca)
        da1, g[n + ".Wqkv"], g[n + ".bqkv"] = L.linear_bwd(dqkv.reshape(b * t, 3 * d), cq)
        dx, g[n + ".ln1.g"], g[n + ".ln1.b"] = L.layernorm_bwd(da1.reshape(b, t, d), cl1)
        return dh + dx

    def _lm_bwd(self, k, dh, cache):
        g = {}
        for block_cache in reversed(cache["blocks"]):
            dh = self._lm_block_bwd(dh, block_cache, g)
        self._dx_in = dh         # gradient at the chunk input: used only by the overlapping variant
        if k == 0:
            g["c0.tok"], g["c0.pos"] = L.embedding_bwd(dh, cache["emb"])
        return g

    # ResNet chunk: one stage of BasicBlocks or bottleneck blocks (stem convolution in chunk 0), App. B.3.
    def _resnet_fwd(self, k, x):
        p = self.p
        cache = {"blocks": []}
        if k == 0:
            u, cc = L.conv2d_fwd(x, p["c0.stem.conv"], 1, 1)
            u, cb = self._bn(u, "c0.stem.bn")
            x, cr = L.relu_fwd(u)
            cache["stem"] = (cc, cb, cr)
        for j in range(lp_synth.resnet_stage_blocks(self.cfg, k)):
            n = f"c{k}.r{j}"
            s = lp_synth.resnet_stage_stride(self.cfg, k) if j == 0 else 1
            if self.cfg.get("block") == "bottleneck":
                x, bc = self._bottleneck_fwd(x, n, s)
                cache["blocks"].append(bc)
                continue
            u, cc1 = L.conv2d_fwd(x, p[n + ".conv1"], s, 1)
            u, cb1 = self._bn(u, n + ".bn1")
            u, cr1 = L.relu_fwd(u)
            u, cc2 = L.conv2d_fwd(u, p[n + ".conv2"], 1, 1)
            u, cb2 = self._bn(u, n + ".bn2")
            if n + ".sc.conv" in p:
                sc, ccs = L.conv2d_fwd(x, p[n + ".sc.conv"], s, 0)
                sc, cbs = self._bn(sc, n + ".sc.bn")
                csc = (ccs, cbs)
            else:
                sc, csc = x, None
            x, cr2 = L.relu_fwd(u + sc)
            cache["blocks"].append((n, cc1, cb1, cr1, cc2, cb2, csc, cr2))
        return x, cache

    def _bottleneck_fwd(self, x, n, s):
        """Bottleneck block of the deeper residual networks (Sec. 4.3 trains a ResNet-50; App. B.3): 1x1
        convolution to the stage's inner width, 3x3 convolution (carrying the block's stride), 1x1 convolution
        to four times that width, each followed by BatchNorm and the first two by ReLU; the shortcut is the
        identity or, where the shape changes, a 1x1 convolution with the block's stride and BatchNorm; ReLU
        after the sum."""
        p = self.p
        u, cc1 = L.conv2d_fwd(x, p[n + ".conv1"], 1, 0)
        u, cb1 = self._bn(u, n + ".bn1")
        u, cr1 = L.relu_fwd(u)
        u, cc2 = L.conv2d_fwd(u, p[n + ".conv2"], s, 1)
        u, cb2 = self._bn(u, n + ".bn2")
        u, cr2 = L.relu_fwd(u)
        u, cc3 = L.conv2d_fwd(u, p[n + ".conv3"], 1, 0)
        u, cb3 = self._bn(u, n + ".bn3")
        if n + ".sc.conv" in p:
            sc, ccs = L.conv2d_fwd(x, p[n + ".sc.conv"], s, 0)
            sc, cbs = self._bn(sc, n + ".sc.bn")
            csc = (ccs, cbs)
        else:
            sc, csc = x, None
        y, cr3 = L.relu_fwd(u + sc)
        return y, ("bottleneck", n, cc1, cb1, cr1, cc2, cb2, cr2, cc3, cb3, csc, cr3)

    def _bottleneck_bwd(self, dx, block_cache, g):
        (_, n, cc1, cb1, cr1, cc2, cb2, cr2, cc3, cb3, csc, cr3) = block_cache
        ds = L.relu_bwd(dx, cr3)
        du, g[n + ".bn3.g"], g[n + ".bn3.b"] = L.batchnorm_bwd(ds, cb3)
        du, g[n + ".conv3"] = L.conv2d_bwd(du, cc3)
        du = L.relu_bwd(du, cr2)
        du, g[n + ".bn2.g"], g[n + ".bn2.b"] = L.batchnorm_bwd(du, cb2)
        du, g[n + ".conv2"] = L.conv2d_bwd(du, cc2)
        du = L.relu_bwd(du, cr1)
        du, g[n + ".bn1.g"], g[n + ".bn1.b"] = L.batchnorm_bwd(du, cb1)
        dx, g[n + ".conv1"] = L.conv2d_bwd(du, cc1)
        if csc is not None:
            ccs, cbs = csc
            dsc, g[n + ".sc.bn.g"], g[n + ".sc.bn.b"] = L.batchnorm_bwd(ds, cbs)
            dsc, g[n + ".sc.conv"] = L.conv2d_bwd(dsc, ccs)
            return dx + dsc
        return dx + ds

    def _bn(self, x, name):
        """BatchNorm `name` on x.  Training and plain forward passes use the batch statistics (App. B.3's
        networks are trained with them); a training step also moves the running statistics.  In
        evaluation mode (bn_mode "running") the running statistics normalise instead."""
        p = self.p
        if self.bn_mode == "running":
            return L.batchnorm_eval(x, p[name + ".g"], p[name + ".b"], p[name + ".rm"], p[name + ".rv"]), None
        y, cache = L.batchnorm_fwd(x, p[name + ".g"], p[name + ".b"])
        if self.training:
            n = x.shape[0] * x.shape[2] * x.shape[3]
            rm, rv = L.batchnorm_running_update(p[name + ".rm"], p[name + ".rv"], cache, n)
            p[name + ".rm"], p[name + ".rv"] = rm.astype(p[name + ".rm"].dtype), rv.astype(p[name + ".rv"].dtype)
        return y, cache

    def _resnet_block_bwd(self, dx, block_cache, g):
        """Backward of one BasicBlock (or bottleneck block): fills g with its parameter gradients, returns the
        gradient at the block input (main branch plus shortcut)."""
        if block_cache[0] == "bottleneck":
            return self._bottleneck_bwd(dx, block_cache, g)
        (n, cc1, cb1, cr1, cc2, cb2, csc, cr2) = block_cache
        ds = L.relu_bwd(dx, cr2)
        du, g[n + ".bn2.g"], g[n + ".bn2.b"] = L.batchnorm_bwd(ds, cb2)
        du, g[n + ".conv2"] = L.conv2d_bwd(du, cc2)
        du = L.relu_bwd(du, cr1)
        du, g[n + ".bn1.g"], g[n + ".bn1.b"] = L.batchnorm_bwd(du, cb1)
        dx, g[n + ".conv1"] = L.conv2d_bwd(du, cc1)
        if csc is not None:
            ccs, cbs = csc
            dsc, g[n + ".sc.bn.g"], g[n + ".sc.bn.b"] = L.batchnorm_bwd(ds, cbs)
            dsc, g[n + ".sc.conv"] = L.conv2d_bwd(dsc, ccs)
            return dx + dsc
        return dx + ds

    def _resnet_bwd(self, k, dx, cache):
        g = {}
        for block_cache in reversed(cache["blocks"]):
            dx = self._resnet_block_bwd(dx, block_cache, g)
        self._dx_in = dx         # gradient at the stage input: used only by the overlapping variant
        if "stem" in cache:
            cc, cb, cr = cache["stem"]
            du = L.relu_bwd(dx, cr)
            du, g["c0.stem.bn.g"], g["c0.stem.bn.b"] = L.batchnorm_bwd(du, cb)
            _, g["c0.stem.conv"] = L.conv2d_bwd(du, cc)
        return g

    # ---------------------------------------------------------------- the step

    def _cast_input(self, x):
        return x if self.cfg["family"] == "lm" else np.asarray(x, dtype=self.dtype)

    def local_grads(self, k, inp, y):
        """Steps 2-4 for one chunk: forward, auxiliary loss, backward truncated at `inp`."""
        self.training = True
        try:
            h, cache = self.chunk_forward(k, inp)
        finally:
            self.training = False
        loss, _, dh, g = self.head(k, h, y, training=True)
        g.update(self.chunk_backward(k, dh, cache))
        self._last_cache = cache
        return loss, h, g

    def overlap_grads(self, k_prev, dx, cache_prev):
        """Overlapping local parallelism (Sec. 3): the gradient of the NEXT chunk's loss with respect to
        the parameters of the last layer of chunk k_prev (its last Linear+ReLU, its last transformer block,
        or its last BasicBlock), given that loss's gradient dx at chunk k_prev's output; truncated at that layer's input."""
        fam = self.cfg["family"]
        g = {}
        if fam == "mlp":
            c1, c2 = cache_prev[-1]
            i = len(cache_prev) - 1
            du = L.relu_bwd(dx, c2)
            _, g[f"c{k_prev}.l{i}.W"], g[f"c{k_prev}.l{i}.b"] = L.linear_bwd(du, c1)
        elif fam == "lm":
            self._lm_block_bwd(dx, cache_prev["blocks"][-1], g)
        else:
            self._resnet_block_bwd(dx, cache_prev["blocks"][-1], g)
        return g

    def apply_update(self, k, grads):
        """Optimizer update of chunk k's trunk and head from its own gradients only."""
        o = self.cfg["optim"]
        for n in self.names_of_chunk[k]:
            if n in self.buffers:
                continue
            if o["kind"] == "sgdm":
                self.p[n] = O.sgdm_update(self.p[n], grads[n], self.state[n], o["lr"], o["momentum"],
                                          o.get("weight_decay", 0.0), self.decay[n])
            else:
                self.p[n] = O.adam_update(self.p[n], grads[n], self.state[n], o["lr"], o["beta1"],
                                          o["beta2"], o["eps"])

    def reset_pipeline(self):
        self.buf = None
        self.t = 0

    def step(self, x, y, schedule=None):
        """One local update step on minibatch (x, y); returns the K auxiliary losses."""
        schedule = schedule or self.cfg["schedule"]
        K = self.K
        x = self._cast_input(x)
        losses = np.full(K, np.nan, dtype=np.float64)
        all_grads = [None] * K
        if self.overlap and schedule != "sync":
            raise ValueError("overlapping updates are defined for the synchronous schedule")
        if schedule == "sync":
            inp, prev_cache = x, None
            for k in range(K):
                losses[k], h, all_grads[k] = self.local_grads(k, inp, y)
                if self.overlap and k > 0:
                    # chunk k's loss reaches one layer further back; that layer's update is the average of
                    # its two gradients (App. A.2: "an additional average of gradients")
                    for n, g2 in self.overlap_grads(k - 1, self._dx_in, prev_cache).items():
                        all_grads[k - 1][n] = ((all_grads[k - 1][n] + g2) * 0.5).astype(g2.dtype)
                prev_cache = self._last_cache
                inp = h                      # handed on as a constant: no gradient flows back
        else:
            if self.buf is None:
                self.buf = [None] * (K - 1)
                if self.ramp == "prime":
                    h = x
                    for k in range(K - 1):
                        h, _ = self.chunk_forward(k, h)
                        self.buf[k] = (h, y)
            new_buf = [None] * (K - 1)
            for k in range(K):
                src = (x, y) if k == 0 else self.buf[k - 1]
                if src is None:
                    continue                 # idle ramp-up: nothing has reached this chunk yet
                losses[k], h, all_grads[k] = self.local_grads(k, src[0], src[1])
                if k < K - 1:
                    new_buf[k] = (h, src[1])
            self.buf = new_buf
            self.t += 1
        for k in range(K):
            if all_grads[k] is not None:
                self.apply_update(k, all_grads[k])
        self.last_grads = {n: v for g in all_grads if g is not None for n, v in g.items()}
        return losses

    def forward(self, x, y=None):
        """Forward chain with the current weights, no update: (last head's logits, K losses)."""
        h = self._cast_input(x)
        losses = np.full(self.K, np.nan)
        z = None
        for k in range(self.K):
            h, _ = self.chunk_forward(k, h)
            if y is not None or k == self.K - 1:
                yy = y if y is not None else np.zeros(self._head_rows(h), dtype=np.int32)
                loss, z, _, _ = self.head(k, h, yy)
                if y is not None:
                    losses[k] = loss
        return z, losses

    def evaluate(self, x, y, bn="batch"):
        """Forward chain with the current weights on a labelled minibatch: per chunk the auxiliary loss,
        the logits [rows, classes], the predicted class of every row (largest logit, lowest index among
        equal ones) and the number of rows predicted correctly (rows labelled -1 are not counted).  Every
        chunk's head is trained to predict the target on its own (Sec. 3).  bn="running": BatchNorm
        normalises with its running statistics instead of this minibatch's."""
        h = self._cast_input(x)
        out = []
        self.bn_mode = bn        # "running": BatchNorm uses its running statistics instead of this minibatch's
        try:
            heads = []
            for k in range(self.K):
                h, _ = self.chunk_forward(k, h)
                heads.append(self.head(k, h, y))
        finally:
            self.bn_mode = "batch"
        for k in range(self.K):
            loss, z, _, _ = heads[k]
            z2 = z.reshape(-1, z.shape[-1])
            pred = np.argmax(z2, axis=1).astype(np.int32)
            lab = np.asarray(y).reshape(-1)
            out.append(dict(loss=float(loss), logits=z2, pred=pred, correct=int(np.sum((lab >= 0) & (pred == lab)))))
        return out

    def _head_rows(self, h):
        return h.shape[:2] if self.cfg["family"] == "lm" else h.shape[0]
