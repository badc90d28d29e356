"""Misuse of the C ABI is answered with error codes before anything touches a GPU: every case here runs on a
machine without one.  (What a step must do: Sec. 3; the entry points themselves follow include/lp.h.)"""
import ctypes as C

import pytest

import lp_synth
from paper_2012_03837_b200 import binding as lp

ERR = {v: k for k, v in lp.LP_ERR.items()}


def create_error(cfg, mutate=None, K=None):
    m, k, hd, op = lp.specs_from_config(cfg)
    if mutate:
        mutate(m, hd, op)
    with pytest.raises(lp.LpError) as e:
        lp.lp_create(m, K if K is not None else k, hd, op)
    return e.value


def test_lp_create_rejects_inconsistent_specifications():
    c1, c3, c4 = lp_synth.config("c1"), lp_synth.config("c3"), lp_synth.config("c4")
    cases = [
        (c1, lambda m, hd, op: setattr(m, "batch", 0), None, "SHAPE"),
        (c1, lambda m, hd, op: setattr(m, "dtype", 7), None, "INVALID_ARG"),
        (c1, lambda m, hd, op: setattr(m, "family", 9), None, "INVALID_ARG"),
        (c1, lambda m, hd, op: setattr(op, "kind", 5), None, "INVALID_ARG"),
        (c1, lambda m, hd, op: setattr(hd, "kind", lp.LP_HEAD_LN_LINEAR), None, "INVALID_ARG"),
        (c1, lambda m, hd, op: setattr(m, "n_layers", 5), None, "SHAPE"),        # chunks no longer sum to the layers
        (c1, None, 0, "SHAPE"),
        (c1, None, 5000, "SHAPE"),
        (c3, lambda m, hd, op: setattr(m, "n_heads", 3), None, "SHAPE"),          # head width must be 64
        (c3, lambda m, hd, op: setattr(hd, "classes", 100), None, "SHAPE"),       # LM head predicts the vocabulary
        (c3, lambda m, hd, op: setattr(m, "seq_len", 0), None, "SHAPE"),
        (c4, lambda m, hd, op: setattr(m, "height", 4), None, "SHAPE"),           # 4 stages halve a 4-pixel image away
        (c4, lambda m, hd, op: setattr(m, "blocks_per_stage", 0), None, "SHAPE"),
        (c4, lambda m, hd, op: setattr(hd, "kind", lp.LP_HEAD_LN_LINEAR), None, "INVALID_ARG"),
        (c1, lambda m, hd, op: setattr(hd, "kind", lp.LP_HEAD_BN_RELU_GAP_LINEAR), None, "INVALID_ARG"),
    ]
    for cfg, mutate, K, want in cases:
        e = create_error(cfg, mutate, K)
        assert lp.LP_ERR[e.code] == want, (cfg["name"], want, str(e))
        assert str(e)                                # a message comes with the code


def test_null_handles_and_pointers_are_refused():
    L = lp._lib
    assert L.lp_create(None, 1, None, None, None, None) == ERR["INVALID_ARG"]
    out = C.c_void_p()
    assert L.lp_create(None, 1, None, None, None, C.byref(out)) == ERR["INVALID_ARG"] and not out.value
    for call in (lambda: L.lp_step(None, None, None, 0, None, None),
                 lambda: L.lp_step_host(None, None, None, 0, None, None),
                 lambda: L.lp_forward(None, None, None, None, None, None),
                 lambda: L.lp_evaluate(None, None, None, None, 0, None, None, None),
                 lambda: L.lp_reset_pipeline(None),
                 lambda: L.lp_set_ramp(None, 0),
                 lambda: L.lp_set_drain(None, 0),
                 lambda: L.lp_set_fused_step(None, 1),
                 lambda: L.lp_set_overlap(None, 1),
                 lambda: L.lp_chunk_output(None, 0, None, 0, None),
                 lambda: L.lp_status_poll(None, None),
                 lambda: L.lp_get_tensor(None, 0, 0, None, 0, None),
                 lambda: L.lp_set_tensor(None, 0, 0, None, 0, None),
                 lambda: L.lp_tensor_info_get(None, 0, None),
                 lambda: L.lp_save_state(None, None, 0),
                 lambda: L.lp_load_state(None, None, 0)):
        assert call() == ERR["INVALID_ARG"]
    assert L.lp_destroy(None) == 0
    assert L.lp_num_tensors(None) == 0
    assert L.lp_state_size(None) == 0


def test_kernel_level_entries_check_their_arguments_first():
    L = lp._lib
    assert L.lp_gemm_bf16(0, None, 0, None, None) == ERR["INVALID_ARG"]
    assert L.lp_gemm_bf16_static(0, None, None) == ERR["INVALID_ARG"]
    too_many = (lp.lp_gemm_desc * (lp.LP_GEMM_STATIC_MAX + 1))()
    assert L.lp_gemm_bf16_static(lp.LP_GEMM_STATIC_MAX + 1, too_many, None) == ERR["SHAPE"]
    assert b"64" in L.lp_gemm_static_last_error()
    # descriptors that would make a kernel read or write where it must not are refused before any launch
    def desc(**kw):
        d = lp.lp_gemm_desc()
        base = dict(A=256, B=512, C=1024, M=64, N=64, K=64, a_ms=64, a_ks=1, b_ns=64, b_ks=1, ldc=64)
        base.update(kw)
        for k, v in base.items():
            setattr(d, k, v)
        return d
    bad = [dict(act=5), dict(act=-1), dict(act=2), dict(act=2, C2=2048, out_f32=1), dict(act=3), dict(act=4), dict(ldc=63),
           dict(a_ms=2, a_ks=2), dict(b_ns=0), dict(K=0), dict(A=0), dict(C=0), dict(out_f32=2)]
    for kw in bad:
        arr = (lp.lp_gemm_desc * 1)(desc(**kw))
        assert L.lp_gemm_bf16(1, arr, 0, None, None) == ERR["INVALID_ARG"], kw
        assert lp.lp_last_error(None), kw
        assert L.lp_gemm_bf16_static(1, arr, None) == ERR["INVALID_ARG"], kw
        assert b"problem 0" in L.lp_gemm_static_last_error(), kw
    assert L.lp_gemm_bf16(1, (lp.lp_gemm_desc * 1)(desc()), 2, None, None) == ERR["INVALID_ARG"]   # unknown backend
    assert L.lp_conv3x3_bf16(0, None, None, None, 1, 8, 8, 64, 64, None) == ERR["INVALID_ARG"]
    one = C.c_void_p(256)
    assert L.lp_attention_bf16(0, None, one, one, None, None, None, 1, 64, 1, None) == ERR["INVALID_ARG"]
    assert L.lp_attention_bf16(1, one, one, one, None, one, one, 1, 64, 1, None) == ERR["INVALID_ARG"]   # backward needs dout
    assert L.lp_attention_bf16(2, one, one, one, one, one, one, 1, 64, 1, None) == ERR["INVALID_ARG"]
    assert L.lp_attention_bf16(0, one, one, one, None, None, None, 0, 64, 1, None) == ERR["SHAPE"]
    assert L.lp_conv3x3_bf16(0, one, one, one, 0, 8, 8, 64, 64, None) == ERR["SHAPE"]
    assert L.lp_conv3x3_bf16(7, one, one, one, 1, 8, 8, 64, 64, None) == ERR["INVALID_ARG"]
