"""Failure handling of the C ABI, with every failure made on the host: bad labels and token ids, a
non-finite input, an allocator that counts, guards or refuses, and damaged checkpoints.  No case here
faults, traps or hangs the GPU: out-of-range indices are clamped or ignored by the kernels and only flagged
in the device status word that lp_status_poll reads (what a step must do: Sec. 3; the entry points follow
include/lp.h)."""
import numpy as np
import pytest
import torch

import lp_synth
from paper_2012_03837_b200 import binding as lp
from tests import lp_testlib as T

pytestmark = pytest.mark.gpu


def small_mlp():
    return lp_synth.config("c1", batch=48, d_in=40, chunks=[[64], [48, 32]], classes=7, schedule="pipelined")


def small_lm():
    return lp_synth.config("c3", batch=2, seq_len=64, vocab=300, d_model=128, n_heads=2, d_ffn=192,
                           blocks_per_chunk=[1, 1], schedule="sync")


def raw_step(gm, x, y):
    """One step without the status poll of GpuModel.step; returns the losses."""
    xt, yt = gm.device_batch(x, y)
    sched = lp.LP_SYNC if gm.cfg["schedule"] == "sync" else lp.LP_PIPELINED
    lp.lp_step(gm.h, xt, yt, sched, gm.stream, gm.losses)
    torch.cuda.synchronize()
    return gm.losses.cpu().numpy().astype(np.float64)


def poll_code(gm):
    try:
        lp.lp_status_poll(gm.h, gm.stream)
        return "OK"
    except lp.LpError as e:
        return lp.LP_ERR[e.code]


def test_labels_out_of_range_are_flagged_and_ignored():
    """A label outside [0, classes) that is not the ignore value -1 raises LABEL_RANGE at the next poll; the
    row contributes no loss and no gradient, exactly as if it had been labelled -1."""
    cfg = dict(small_mlp(), schedule="sync")
    x, y = lp_synth.minibatch(cfg, 0)
    bad, ign = y.copy(), y.copy()
    rows = [3, 17, 40]
    bad[rows] = [cfg["classes"], cfg["classes"] + 1000, -5]
    ign[rows] = -1
    a, b = T.GpuModel(cfg), T.GpuModel(cfg)
    la = raw_step(a, x, bad)
    assert poll_code(a) == "LABEL_RANGE"
    assert poll_code(a) == "OK"                      # the word is cleared by the poll
    lb = raw_step(b, x, ign)
    assert poll_code(b) == "OK"
    assert np.array_equal(la, lb) and np.all(np.isfinite(la))
    wa, wb = a.get(), b.get()
    for n in wa:
        assert np.array_equal(wa[n], wb[n]), n
    la2 = raw_step(a, *lp_synth.minibatch(cfg, 1))   # the handle stays usable
    assert poll_code(a) == "OK" and np.all(np.isfinite(la2))
    a.close(); b.close()


def test_bad_labels_travel_down_the_pipeline_with_their_minibatch():
    """Pipelined schedule (Sec. 6): the labels ride with the activation, so the chunk that trains on the older
    minibatch one step later meets the same bad labels and flags them again; after that the pipeline is clean."""
    cfg = small_mlp()                                # two chunks, pipelined
    gm = T.GpuModel(cfg)
    x, y = lp_synth.minibatch(cfg, 0)
    bad = y.copy()
    bad[7] = 99
    raw_step(gm, x, bad)
    assert poll_code(gm) == "LABEL_RANGE"
    raw_step(gm, *lp_synth.minibatch(cfg, 1))        # chunk 1 now trains on minibatch 0 and its labels
    assert poll_code(gm) == "LABEL_RANGE"
    raw_step(gm, *lp_synth.minibatch(cfg, 2))
    assert poll_code(gm) == "OK"
    gm.close()


def test_token_ids_out_of_range_are_flagged_and_clamped():
    cfg = small_lm()
    x, y = lp_synth.minibatch(cfg, 0)
    bad = x.copy()
    bad[0, 5], bad[1, 60] = cfg["vocab"] + 7, -3
    clamped = np.clip(bad, 0, cfg["vocab"] - 1)
    a, b = T.GpuModel(cfg), T.GpuModel(cfg)
    la = raw_step(a, bad, y)
    assert poll_code(a) == "LABEL_RANGE"
    lb = raw_step(b, clamped, y)
    assert poll_code(b) == "OK"
    assert np.array_equal(la, lb)
    wa, wb = a.get(), b.get()
    for n in wa:
        assert np.array_equal(wa[n], wb[n]), n
    a.close(); b.close()


def test_non_finite_input_is_reported_as_nonfinite_loss():
    cfg = small_mlp()
    x, y = lp_synth.minibatch(cfg, 0)
    x = x.copy()
    x[5, 3] = np.nan
    gm = T.GpuModel(cfg)
    losses = raw_step(gm, x, y)
    assert not np.all(np.isfinite(losses))
    assert poll_code(gm) == "NONFINITE"
    gm.close()


class GuardedAllocator:
    """lp_alloc callbacks on top of torch's caching allocator: counts blocks, can refuse the n-th request,
    and surrounds every block with 256-byte guard zones whose pattern is checked at release."""
    GUARD = 256

    def __init__(self, fail_at=None):
        self.fail_at = fail_at
        self.calls = 0
        self.live = {}          # user pointer -> (raw pointer, bytes)
        self.damaged = []
        self.released = 0
        self._a = lp.LP_ALLOC_FN(self._alloc)
        self._r = lp.LP_RELEASE_FN(self._release)
        self.struct = lp.lp_alloc(self._a, self._r, None)

    def _guards(self, raw, nbytes):
        g = self.GUARD
        lo = _device_view(raw, g)
        hi = _device_view(raw + g + nbytes, g)
        return lo, hi

    def _alloc(self, nbytes, user):
        self.calls += 1
        if self.fail_at is not None and self.calls == self.fail_at:
            return None
        g = self.GUARD
        raw = torch.cuda.caching_allocator_alloc(nbytes + 2 * g)
        lo, hi = self._guards(raw, nbytes)
        lo.fill_(0xA5); hi.fill_(0x5A)
        self.live[raw + g] = (raw, nbytes)
        return raw + g

    def _release(self, ptr, user):
        raw, nbytes = self.live.pop(ptr)
        lo, hi = self._guards(raw, nbytes)
        torch.cuda.synchronize()
        if not (bool((lo == 0xA5).all()) and bool((hi == 0x5A).all())):
            self.damaged.append((ptr, nbytes))
        self.released += 1
        torch.cuda.caching_allocator_delete(raw)


def _device_view(ptr, nbytes):
    """uint8 torch view of raw device memory [ptr, ptr + nbytes)."""
    class _Iface:
        pass
    o = _Iface()
    o.__cuda_array_interface__ = dict(shape=(nbytes,), typestr="|u1", data=(ptr, False), version=2)
    return torch.as_tensor(o, device="cuda")


def create_with(cfg, allocator):
    m, K, hd, op = lp.specs_from_config(cfg)
    return lp.lp_create(m, K, hd, op, allocator.struct), K


def test_allocator_callbacks_back_every_block_and_guards_stay_intact():
    """Every device block of a handle comes from the caller's allocator and goes back at lp_destroy; no kernel
    of a training run writes outside the blocks it was given (guard zones around each block)."""
    for cfg in (small_mlp(), small_lm(),
                lp_synth.config("c4", batch=8, height=8, width=8, stem_channels=16, stage_channels=[16, 32],
                                blocks_per_stage=1, classes=5)):
        al = GuardedAllocator()
        free0 = torch.cuda.memory_allocated()
        h, K = create_with(cfg, al)
        assert al.calls > 3 and len(al.live) == al.calls
        assert lp.lp_device_bytes(h) == sum((b + 255) // 256 * 256 for _, b in al.live.values())
        gm = T.GpuModel.__new__(T.GpuModel)
        gm.cfg, gm.K, gm.h = cfg, K, h
        gm.index = {}
        for i in range(lp.lp_num_tensors(h)):
            info = lp.lp_tensor_info_get(h, i)
            gm.index[info["name"]] = (i, info)
        gm.dev = torch.device("cuda:0")
        gm.losses = torch.zeros(K, dtype=torch.float32, device=gm.dev)
        gm.stream = torch.cuda.current_stream().cuda_stream
        gm.set_params(lp_synth.init_params(cfg))
        for t in range(3):
            losses = gm.step(*lp_synth.minibatch(cfg, t))
            assert np.all(np.isfinite(losses))
        gm.close()
        del gm
        assert al.released == al.calls and not al.live
        assert not al.damaged, al.damaged
        assert torch.cuda.memory_allocated() == free0


@pytest.mark.parametrize("fail_at", [1, 4, 9])
def test_allocator_that_refuses_gives_alloc_error_and_leaks_nothing(fail_at):
    al = GuardedAllocator(fail_at=fail_at)
    cfg = small_lm()
    m, K, hd, op = lp.specs_from_config(cfg)
    with pytest.raises(lp.LpError) as e:
        lp.lp_create(m, K, hd, op, al.struct)
    assert lp.LP_ERR[e.value.code] == "ALLOC" and "alloc" in str(e.value).lower()
    assert al.calls == fail_at                       # nothing was requested after the refusal
    assert not al.live and al.released == fail_at - 1
    assert not al.damaged


def test_damaged_checkpoints_are_refused_and_the_handle_stays_usable():
    cfg = small_mlp()
    gm = T.GpuModel(cfg)
    other = T.GpuModel(lp_synth.config("c1", batch=48, d_in=40, chunks=[[64], [48], [32]], classes=7, schedule="pipelined"))
    for t in range(2):
        gm.step(*lp_synth.minibatch(cfg, t))
    n = lp.lp_state_size(gm.h)
    blob = np.empty(n, dtype=np.uint8)
    lp.lp_save_state(gm.h, blob)
    before = gm.get()

    def load_error(handle, arr):
        with pytest.raises(lp.LpError) as e:
            lp.lp_load_state(handle, arr)
        return lp.LP_ERR[e.value.code]

    bad_magic = blob.copy(); bad_magic[0] ^= 0xFF
    assert load_error(gm.h, bad_magic) == "STATE"
    bad_k = blob.copy(); bad_k[16:24] = np.frombuffer(np.int64(3).tobytes(), dtype=np.uint8)   # header field K
    assert load_error(gm.h, bad_k) == "STATE"
    assert load_error(gm.h, blob[:-8].copy()) == "SHAPE"
    assert load_error(other.h, np.zeros(lp.lp_state_size(other.h), dtype=np.uint8)) == "STATE"
    if lp.lp_state_size(other.h) != n:
        assert load_error(other.h, blob) == "SHAPE"   # a blob of another model
    # nothing changed, and the handle goes on: the next step equals the one of an undisturbed twin
    after = gm.get()
    for name in before:
        assert np.array_equal(before[name], after[name]), name
    twin = T.GpuModel(cfg)
    lp.lp_load_state(twin.h, blob)
    x, y = lp_synth.minibatch(cfg, 2)
    assert np.array_equal(gm.step(x, y), twin.step(x, y))
    gm.close(); twin.close(); other.close()
