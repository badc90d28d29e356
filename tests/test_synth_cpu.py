"""The seeded generators produce what the workloads state (they hold none of the method's arithmetic, so
parity between the two implementations cannot see a mistake here)."""
import numpy as np

import lp_synth


def test_lm_targets_are_the_ids_shifted_left_with_the_last_position_ignored():
    for name in ("c3", "c5"):
        cfg = lp_synth.config(name, batch=3, seq_len=17)
        for t in (0, 1, 5):
            x, y = lp_synth.minibatch(cfg, t)
            assert x.dtype == np.int32 and y.dtype == np.int32 and x.shape == y.shape == (3, 17)
            assert x.min() >= 0 and x.max() < cfg["vocab"]
            assert np.array_equal(y[:, :-1], x[:, 1:])          # next-token targets
            assert np.all(y[:, -1] == -1)                       # nothing follows the last position


def test_minibatches_are_reproducible_and_differ_between_steps():
    cfg = lp_synth.config("c2", batch=8, d_in=16)
    x0, y0 = lp_synth.minibatch(cfg, 0)
    x0b, y0b = lp_synth.minibatch(cfg, 0)
    x1, _ = lp_synth.minibatch(cfg, 1)
    assert np.array_equal(x0, x0b) and np.array_equal(y0, y0b) and not np.array_equal(x0, x1)
    assert np.array_equal(x0, lp_synth.bf16_round(x0))          # bf16 workloads start from bf16-representable inputs
    assert y0.min() >= 0 and y0.max() < cfg["classes"]
