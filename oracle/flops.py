"""CPU oracle, FLOP cost model of App. A (host arithmetic only).  TEST INFRASTRUCTURE ONLY.

App. A.1 counts an MLP layer as a matrix-vector product (2*I*N - I), a bias add (N) and a ReLU
(2*N), and its auxiliary classifier as a matrix-vector product to 10 classes (2*N*10 - N), a bias
add (10) and a softmax cross-entropy at 5 FLOPs per class (5*10).  App. A.2 combines forward cost,
auxiliary cost, backward multiplier and optimizer cost (ten FLOPs per parameter) per method.
"""
from __future__ import annotations


def mlp_layer_forward_flops(i: int, n: int) -> int:
    return (2 * i * n - i) + n + 2 * n


def mlp_aux_flops(n: int, classes: int = 10) -> int:
    return (2 * n * classes - n) + classes + 5 * classes


def mlp_mean_forward_flops(input_size: int, n: int, layers: int) -> float:
    """Forward cost averaged over the layers: the first maps input_size -> n, the rest n -> n."""
    total = mlp_layer_forward_flops(input_size, n) + (layers - 1) * mlp_layer_forward_flops(n, n)
    return total / layers


def cost_per_example(method: str, forward_cost: float, aux_cost: float, backward_multiplier: float,
                     layers: int, chunks: int = 1) -> float:
    """Per-example cost of one step (App. A.2).  For "chunked", forward_cost is read as the cost of
    the whole stack (forward_cost * layers), by analogy with the back-propagation formula."""
    bm = backward_multiplier
    if method == "backprop":
        return (1 + bm) * (forward_cost * layers + aux_cost)
    if method == "greedy":
        return (1 + bm) * ((forward_cost + aux_cost) * layers)
    if method == "chunked":
        return (1 + bm) * (forward_cost * layers + chunks * aux_cost)
    if method == "overlapping":
        return ((forward_cost + aux_cost) * layers
                + (layers - 1) * bm * (2 * forward_cost + aux_cost)
                + bm * (forward_cost + aux_cost))
    if method == "last_layers":
        # full forward pass and one loss, backward pass through the last `chunks` layers only (the printed
        # formula lacks the "+" between the forward and the auxiliary cost)
        return (layers * forward_cost + aux_cost) + bm * (chunks * forward_cost + aux_cost)
    raise ValueError(method)


def total_cost(method: str, per_example: float, steps: int, batch_size: int, parameters: float) -> float:
    """Total FLOPs of a run (App. A.2): the optimizer costs ten FLOPs per parameter per step, and the
    overlapping method two more per parameter for averaging the shared layers' gradients."""
    optimizer = 10 * parameters + (2 * parameters if method == "overlapping" else 0)
    return per_example * steps * batch_size + steps * optimizer


def parallelism(method: str, layers: int, chunks: int = 1, backward_multiplier: float = 0.0) -> float:
    """Units that run at once per example (App. A.2); for "last_layers" the trained tail of `chunks`
    layers is the atomic unit and the remaining forward work is cut into pieces of that size."""
    if method == "last_layers":
        bm = backward_multiplier
        return (layers + chunks * bm) / (chunks * (1 + bm))
    return {"backprop": 1, "greedy": layers, "overlapping": layers, "chunked": chunks}[method]
