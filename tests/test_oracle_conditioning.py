"""tests/golden/c2_conditioning.json is what its script says: the gap between two correct evaluations of the
wide-MLP workload, measured with the CPU oracle alone.  Re-runs the first steps of the script and reads the
stored table for the facts the GPU parity test relies on."""
import importlib.util
import json
import os

import numpy as np

HERE = os.path.dirname(os.path.abspath(__file__))


def test_stored_conditioning_table_is_reproduced_by_its_script():
    spec = importlib.util.spec_from_file_location("make_c2_conditioning", os.path.join(HERE, "golden", "make_c2_conditioning.py"))
    mod = importlib.util.module_from_spec(spec)
    spec.loader.exec_module(mod)
    stored = json.load(open(os.path.join(HERE, "golden", "c2_conditioning.json")))["steps"]
    assert [s["step"] for s in stored] == list(range(1, 11))
    fresh = mod.run(steps=2)
    for a, b in zip(fresh, stored):
        for w in ("fp32_vs_fp64", "bf16io_vs_fp32"):
            # the BLAS of another machine may sum in another order: the gaps themselves are rounding effects,
            # so only their size is compared
            assert np.all(np.array(a[w]["weights"]) <= 3 * np.array(b[w]["weights"]) + 1e-5), (a["step"], w)
            assert np.all(np.array(b[w]["weights"]) <= 3 * np.array(a[w]["weights"]) + 1e-5), (a["step"], w)
    # what the table says: rounding alone moves the ten-step result past 2e-2
    w64 = [max(s["fp32_vs_fp64"]["weights"]) for s in stored]
    wbf = [max(s["bf16io_vs_fp32"]["weights"]) for s in stored]
    assert all(x < y for x, y in zip(w64, w64[1:])) and all(x < y for x, y in zip(wbf, wbf[1:]))   # grows every step
    assert w64[-1] > 2e-2 and wbf[3] > 2e-2 and wbf[-1] > 5e-2
    assert max(max(s["bf16io_vs_fp32"]["loss"]) for s in stored) < 2e-2
