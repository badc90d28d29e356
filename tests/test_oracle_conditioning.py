"""tests/golden/c2_conditioning.json and c4_conditioning.json are what their script says: the gap between two
correct evaluations of a workload, measured with the CPU oracle alone.  Re-runs the first steps of the script for
c2 and reads the stored tables for the facts the GPU parity tests rely on."""
import importlib.util
import json
import os

import numpy as np

HERE = os.path.dirname(os.path.abspath(__file__))


def stored(name):
    return json.load(open(os.path.join(HERE, "golden", f"{name}_conditioning.json")))["steps"]


def test_stored_conditioning_table_is_reproduced_by_its_script():
    spec = importlib.util.spec_from_file_location("make_conditioning", os.path.join(HERE, "golden", "make_conditioning.py"))
    mod = importlib.util.module_from_spec(spec)
    spec.loader.exec_module(mod)
    table = stored("c2")
    assert [s["step"] for s in table] == list(range(1, 11))
    fresh = mod.run("c2", steps=2)
    for a, b in zip(fresh, table):
        for w in ("fp32_vs_fp64", "bf16io_vs_fp32"):
            # the BLAS of another machine may sum in another order: the gaps themselves are rounding effects,
            # so only their size is compared
            assert np.all(np.array(a[w]["weights"]) <= 3 * np.array(b[w]["weights"]) + 1e-5), (a["step"], w)
            assert np.all(np.array(b[w]["weights"]) <= 3 * np.array(a[w]["weights"]) + 1e-5), (a["step"], w)


def test_rounding_alone_moves_the_ten_step_results_past_the_nominal_tolerances():
    c2 = stored("c2")
    w64 = [max(s["fp32_vs_fp64"]["weights"]) for s in c2]
    wbf = [max(s["bf16io_vs_fp32"]["weights"]) for s in c2]
    assert all(x < y for x, y in zip(w64, w64[1:])) and all(x < y for x, y in zip(wbf, wbf[1:]))   # grows every step
    assert w64[-1] > 2e-2                      # fp32 against fp64: past 1e-3 at once, past 2e-2 after ten steps
    assert wbf[-1] > 5e-2 and min(t for t, w in enumerate(wbf, 1) if w > 2e-2) <= 5
    c4 = stored("c4")
    assert [s["step"] for s in c4] == list(range(1, 11))
    assert max(c4[-1]["bf16io_vs_fp32"]["weights"]) > 2e-2      # the small head matrices
