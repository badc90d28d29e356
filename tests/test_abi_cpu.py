"""The C-ABI library loads without a GPU and exports every symbol include/lp.h declares."""
import ctypes
import os
import re

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def declared_symbols():
    text = open(os.path.join(ROOT, "include", "lp.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(lp_[a-z0-9_]+)\s*\(", text)))


def test_library_exports_every_declared_symbol():
    from paper_2012_03837_b200 import build
    lib = ctypes.CDLL(build.build())
    names = declared_symbols()
    assert "lp_create" in names and "lp_step" in names and "lp_forward" in names and "lp_destroy" in names
    for n in names:
        assert hasattr(lib, n), n


def test_binding_lists_the_same_entry_points():
    from paper_2012_03837_b200 import binding
    assert sorted(binding.EXPORTS) == declared_symbols()


def test_bad_arguments_are_rejected_without_a_gpu():
    from paper_2012_03837_b200 import binding as lp
    import lp_synth
    m, K, hd, op = lp.specs_from_config(lp_synth.config("c3", d_model=100))
    try:
        lp.lp_create(m, K, hd, op)
        assert False
    except lp.LpError as e:
        assert e.code == -2 and "64" in str(e)
    m, K, hd, op = lp.specs_from_config(lp_synth.config("c1"))
    hd.classes = 1
    try:
        lp.lp_create(m, K, hd, op)
        assert False
    except lp.LpError as e:
        assert e.code == -2
    assert lp._lib.lp_step(None, None, None, 0, None, None) == -1
    assert lp._lib.lp_destroy(None) == 0
