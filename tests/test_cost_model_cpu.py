"""FLOP cost model of App. A through the C ABI (host arithmetic, no GPU): pinned by the values App. A.1 prints
for the 8-layer, 4096-unit MLP, by the model constants App. A.2 lists, by special cases that tie the methods
to one another, and compared with the oracle's own restatement of the formulas."""
import os

import pytest

from oracle import flops
from paper_2012_03837_b200 import binding as B

GOLD = os.path.join(os.path.dirname(__file__), "golden", "mlp_flops.txt")

# App. A.1: layers, forward cost per layer, auxiliary cost, backward multiplier, parameters
MODELS = {
    "resnet50": (17, 5479411.176470588, 3382457.3529411764, 2.0280375672996596, 38711720.0),
    "resnet18": (9, 1640544.352941176, 565900.6470588235, 2.08565879129763, 13170792.0),
    "transformer_small": (4, 13837446.0, 1163904.0, 1.6581083035860107, 0.0),
    "transformer_large": (6, 51037318.0, 4653696.0, 1.7526391044859857, 0.0),
}


def gold():
    vals = {}
    for line in open(GOLD):
        if line.strip() and not line.startswith("#"):
            k, v = line.split()
            vals[k] = float(v)
    return vals


def test_mlp_worked_example_matches_printed_values():
    g = gold()
    i, n, layers = int(g["input_size"]), int(g["hidden"]), int(g["layers"])
    mean_fwd = (B.lp_mlp_layer_flops(i, n) + (layers - 1) * B.lp_mlp_layer_flops(n, n)) / layers
    assert mean_fwd == g["mean_forward_flops"]
    assert B.lp_mlp_aux_flops(n, 10) == g["aux_flops"]


def test_mlp_layer_count_by_enumeration():
    # brute force on a tiny square layer: n dot products of n multiplies and n-1 adds, a bias add and the two
    # ReLU FLOPs per unit.  (For a rectangular layer App. A.1 subtracts the input size, not the unit count;
    # the library follows the printed formula.)
    n = 3
    count = 0
    for _ in range(n):
        count += n + (n - 1) + 1 + 2
    assert B.lp_mlp_layer_flops(n, n) == count
    assert B.lp_mlp_layer_flops(5, 3) == (2 * 5 * 3 - 5) + 3 + 2 * 3
    # classifier to c classes: c dot products of length n counted the same way, bias, 5 FLOPs per class
    assert B.lp_mlp_aux_flops(3, 3) == 3 * (3 + 2) + 3 + 5 * 3


@pytest.mark.parametrize("name", sorted(MODELS))
@pytest.mark.parametrize("method,chunks", [("backprop", 1), ("greedy", 1), ("overlapping", 1), ("chunked", 2),
                                           ("chunked", 3), ("last_layers", 1), ("last_layers", 2)])
def test_against_oracle_formulas(name, method, chunks):
    layers, f, a, bm, params = MODELS[name]
    batch, steps = 512, 12345
    r = B.lp_cost_model(method, layers, batch, steps, f, a, bm, params, chunks=chunks)
    per = flops.cost_per_example(method, f, a, bm, layers, chunks=chunks)
    tot = flops.total_cost(method, per, steps, batch, params)
    par = flops.parallelism(method, layers, chunks, bm)
    assert r["cost_per_example"] == pytest.approx(per, rel=1e-14)
    assert r["total_flops"] == pytest.approx(tot, rel=1e-14)
    assert r["parallelism"] == pytest.approx(par, rel=1e-14)
    assert r["sequential_flops"] == pytest.approx(tot / (batch * par), rel=1e-14)


def test_special_cases_tie_the_methods_together():
    layers, f, a, bm, params = MODELS["resnet18"]
    kw = dict(layers=layers, batch_size=64, steps=100, forward_cost=f, aux_cost=a, backward_multiplier=bm,
              parameters=params)
    bp = B.lp_cost_model("backprop", **kw)
    greedy = B.lp_cost_model("greedy", **kw)
    over = B.lp_cost_model("overlapping", **kw)
    # one chunk is back-propagation; one chunk per layer is the greedy method
    assert B.lp_cost_model("chunked", chunks=1, **kw) == bp
    per_layer = B.lp_cost_model("chunked", chunks=layers, **kw)
    assert all(per_layer[k] == pytest.approx(greedy[k], rel=1e-14) for k in greedy)
    # training all layers through "last layers" costs what back-propagation costs, with no parallelism
    last = B.lp_cost_model("last_layers", chunks=layers, **kw)
    assert last["cost_per_example"] == pytest.approx(bp["cost_per_example"], rel=1e-14)
    assert last["parallelism"] == pytest.approx(1.0, rel=1e-14)
    # overlapping = greedy + one more backward pass through every layer but the last, + 2 FLOPs per parameter
    extra = (layers - 1) * bm * f
    assert over["cost_per_example"] == pytest.approx(greedy["cost_per_example"] + extra, rel=1e-14)
    assert over["total_flops"] - greedy["total_flops"] == pytest.approx(
        extra * 100 * 64 + 100 * 2 * params, rel=1e-12)
    # hand-computed: L=2, f=3, a=1, bm=2, 10 parameters, batch 4, 5 steps
    r = B.lp_cost_model("backprop", 2, 4, 5, 3.0, 1.0, 2.0, 10.0)
    assert r["cost_per_example"] == 21.0 and r["total_flops"] == 21.0 * 20 + 5 * 100 and r["sequential_flops"] == 230.0
    r = B.lp_cost_model("greedy", 2, 4, 5, 3.0, 1.0, 2.0, 10.0)
    assert r["cost_per_example"] == 24.0 and r["sequential_flops"] == (24.0 * 20 + 500) / 8
    r = B.lp_cost_model("overlapping", 2, 4, 5, 3.0, 1.0, 2.0, 10.0)
    assert r["cost_per_example"] == 8.0 + 14.0 + 8.0 and r["total_flops"] == 30.0 * 20 + 5 * 120
    r = B.lp_cost_model("last_layers", 2, 4, 5, 3.0, 1.0, 2.0, 10.0, chunks=1)
    assert r["cost_per_example"] == 7.0 + 8.0 and r["parallelism"] == pytest.approx(4.0 / 3.0)


def test_sequential_flops_fall_with_parallelism():
    layers, f, a, bm, params = MODELS["transformer_large"]
    kw = dict(layers=layers, batch_size=256, steps=1000, forward_cost=f, aux_cost=a, backward_multiplier=bm,
              parameters=params)
    seq = [B.lp_cost_model("chunked", chunks=k, **kw)["sequential_flops"] for k in (1, 2, 3, 6)]
    tot = [B.lp_cost_model("chunked", chunks=k, **kw)["total_flops"] for k in (1, 2, 3, 6)]
    assert seq == sorted(seq, reverse=True) and tot == sorted(tot)


def test_rejects_bad_arguments():
    with pytest.raises(B.LpError):
        B.lp_cost_model("chunked", 4, 8, 1, 1.0, 1.0, 1.0, 0.0, chunks=5)
    with pytest.raises(B.LpError):
        B.lp_cost_model("backprop", 0, 8, 1, 1.0, 1.0, 1.0, 0.0)
    with pytest.raises(B.LpError):
        B.lp_cost_model("greedy", 4, 8, 1, -1.0, 1.0, 1.0, 0.0)
    spec = B.lp_cost_spec(9, 4, 1, 8, 1, 1.0, 1.0, 1.0, 0.0)
    out = B.lp_cost_result()
    import ctypes as C
    assert B._lib.lp_cost_model(C.byref(spec), C.byref(out)) == -1  # LP_ERR_INVALID_ARG
    assert B._lib.lp_cost_model(None, C.byref(out)) == -1  # LP_ERR_INVALID_ARG
