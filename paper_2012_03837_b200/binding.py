"""ctypes binding of liblp.so: the same entry points as include/lp.h, argument marshalling only.

Every step of the local update runs inside the library's CUDA kernels.  PyTorch appears only as
the owner of device buffers (``tensor.data_ptr()``) and streams.  If the library is missing the
import fails: there is no fallback path.
"""
from __future__ import annotations

import ctypes as C
import os

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_LIB_PATH = os.path.join(_HERE, "liblp.so")

LP_OK = 0
LP_ERR = {-1: "INVALID_ARG", -2: "SHAPE", -3: "UNSUPPORTED", -4: "ALLOC", -5: "CUDA", -6: "STATE",
          -7: "LABEL_RANGE", -8: "NONFINITE", -9: "TIMEOUT"}
LP_FAMILY_MLP, LP_FAMILY_LM, LP_FAMILY_RESNET = 0, 1, 2
LP_FP32, LP_BF16 = 0, 1
LP_BLOCK_BASIC, LP_BLOCK_BOTTLENECK = 0, 1
LP_HEAD_LINEAR, LP_HEAD_LN_LINEAR, LP_HEAD_GAP_LINEAR, LP_HEAD_BN_RELU_GAP_LINEAR = 0, 1, 2, 3
LP_OPT_SGDM, LP_OPT_ADAM = 0, 1
LP_SYNC, LP_PIPELINED = 0, 1
LP_MASTER, LP_WORKING, LP_MOMENT1, LP_MOMENT2, LP_GRAD = 0, 1, 2, 3, 4


class LpError(RuntimeError):
    def __init__(self, code, msg):
        super().__init__(f"LP_ERR_{LP_ERR.get(code, code)}: {msg}")
        self.code = code


class lp_model_spec(C.Structure):
    _fields_ = [("family", C.c_int), ("dtype", C.c_int), ("batch", C.c_int),
                ("d_in", C.c_int), ("n_layers", C.c_int),
                ("layer_widths", C.POINTER(C.c_int)), ("layers_per_chunk", C.POINTER(C.c_int)),
                ("vocab", C.c_int), ("seq_len", C.c_int), ("d_model", C.c_int), ("n_heads", C.c_int),
                ("d_ffn", C.c_int), ("blocks_per_chunk", C.POINTER(C.c_int)),
                ("in_channels", C.c_int), ("height", C.c_int), ("width", C.c_int),
                ("stem_channels", C.c_int), ("stage_channels", C.POINTER(C.c_int)),
                ("blocks_per_stage", C.c_int), ("gemm_backend", C.c_int), ("input_is_activation", C.c_int),
                ("block_kind", C.c_int), ("stage_blocks", C.POINTER(C.c_int))]


class lp_head_spec(C.Structure):
    _fields_ = [("kind", C.c_int), ("classes", C.c_int)]


class lp_optim_spec(C.Structure):
    _fields_ = [("kind", C.c_int), ("lr", C.c_float), ("momentum", C.c_float), ("weight_decay", C.c_float),
                ("beta1", C.c_float), ("beta2", C.c_float), ("eps", C.c_float)]


class lp_tensor_info(C.Structure):
    _fields_ = [("name", C.c_char * 48), ("chunk", C.c_int), ("ndim", C.c_int), ("shape", C.c_int64 * 4),
                ("numel", C.c_int64), ("has_working_bf16", C.c_int)]


EXPORTS = ["lp_create", "lp_step", "lp_step_host", "lp_forward", "lp_destroy", "lp_num_tensors",
           "lp_tensor_info_get", "lp_get_tensor", "lp_set_tensor", "lp_reset_pipeline", "lp_status_poll",
           "lp_state_size", "lp_save_state", "lp_load_state", "lp_last_step_launches", "lp_device_bytes",
           "lp_last_error", "lp_gemm_bf16", "lp_profile_enable", "lp_profile_read",
           "lp_attention_bf16", "lp_gemm_bf16_static", "lp_gemm_static_poll", "lp_gemm_static_last_error", "lp_conv3x3_bf16", "lp_conv2d_bf16", "lp_set_ramp", "lp_set_drain", "lp_set_fused_step", "lp_evaluate", "lp_set_overlap",
           "lp_cost_model", "lp_mlp_layer_flops", "lp_mlp_aux_flops", "lp_chunk_output_bytes", "lp_chunk_output"]
LP_KIND_NAMES = ["other", "gemm_tc", "gemm_alu", "norm", "xent", "attn", "optim", "reduce", "embed", "conv_aux"]


def load_library() -> C.CDLL:
    if not os.path.exists(_LIB_PATH):
        raise ImportError(f"{_LIB_PATH} is missing: run `python -m paper_2012_03837_b200.build` (needs nvcc)")
    lib = C.CDLL(_LIB_PATH)
    vp, ip = C.c_void_p, C.c_int
    lib.lp_create.argtypes = [C.POINTER(lp_model_spec), ip, C.POINTER(lp_head_spec), C.POINTER(lp_optim_spec), vp, C.POINTER(vp)]
    lib.lp_step.argtypes = [vp, vp, vp, ip, vp, vp]
    lib.lp_step_host.argtypes = [vp, vp, vp, ip, vp, vp]
    lib.lp_forward.argtypes = [vp, vp, vp, vp, vp, vp]
    lib.lp_evaluate.argtypes = [vp, vp, vp, vp, ip, vp, vp, vp]
    lib.lp_destroy.argtypes = [vp]
    lib.lp_num_tensors.argtypes = [vp]
    lib.lp_tensor_info_get.argtypes = [vp, ip, C.POINTER(lp_tensor_info)]
    lib.lp_get_tensor.argtypes = [vp, ip, ip, vp, C.c_size_t, vp]
    lib.lp_set_tensor.argtypes = [vp, ip, ip, vp, C.c_size_t, vp]
    lib.lp_reset_pipeline.argtypes = [vp]
    lib.lp_chunk_output_bytes.argtypes = [vp, ip]
    lib.lp_chunk_output_bytes.restype = C.c_size_t
    lib.lp_chunk_output.argtypes = [vp, ip, vp, C.c_size_t, vp]
    lib.lp_set_ramp.argtypes = [vp, ip]
    lib.lp_set_drain.argtypes = [vp, ip]
    lib.lp_set_fused_step.argtypes = [vp, ip]
    lib.lp_set_overlap.argtypes = [vp, ip]
    lib.lp_status_poll.argtypes = [vp, vp]
    lib.lp_state_size.argtypes = [vp]
    lib.lp_state_size.restype = C.c_size_t
    lib.lp_save_state.argtypes = [vp, vp, C.c_size_t]
    lib.lp_load_state.argtypes = [vp, vp, C.c_size_t]
    lib.lp_last_step_launches.argtypes = [vp]
    lib.lp_device_bytes.argtypes = [vp]
    lib.lp_device_bytes.restype = C.c_size_t
    lib.lp_last_error.argtypes = [vp]
    lib.lp_last_error.restype = C.c_char_p
    return lib


_lib = load_library()


def _check(h, code):
    if code != LP_OK:
        raise LpError(code, (_lib.lp_last_error(h) or b"").decode())


def _ints(seq):
    return (C.c_int * len(seq))(*[int(v) for v in seq])


def _ptr(t):
    """Device or host address of a torch tensor / numpy array / raw int."""
    if t is None:
        return None
    if isinstance(t, int):
        return t
    if isinstance(t, np.ndarray):
        return t.ctypes.data
    return t.data_ptr()


def specs_from_config(cfg: dict, gemm_backend: int = 0):
    """Translate a workload dictionary (see lp_synth.config) into the three C structs and K."""
    m = lp_model_spec()
    keep = []
    fam = cfg["family"]
    m.dtype = LP_BF16 if cfg["dtype"] == "bf16" else LP_FP32
    m.batch = cfg["batch"]
    m.gemm_backend = gemm_backend
    m.input_is_activation = 1 if cfg.get("input_is_activation") else 0
    hd = lp_head_spec()
    if fam == "mlp":
        m.family = LP_FAMILY_MLP
        widths = [w for ch in cfg["chunks"] for w in ch]
        per = [len(ch) for ch in cfg["chunks"]]
        m.d_in, m.n_layers = cfg["d_in"], len(widths)
        a, b = _ints(widths), _ints(per)
        keep += [a, b]
        m.layer_widths, m.layers_per_chunk = a, b
        K = len(per)
        hd.kind, hd.classes = LP_HEAD_LINEAR, cfg["classes"]
    elif fam == "lm":
        m.family = LP_FAMILY_LM
        m.vocab, m.seq_len, m.d_model = cfg["vocab"], cfg["seq_len"], cfg["d_model"]
        m.n_heads, m.d_ffn = cfg["n_heads"], cfg["d_ffn"]
        a = _ints(cfg["blocks_per_chunk"])
        keep.append(a)
        m.blocks_per_chunk = a
        K = len(cfg["blocks_per_chunk"])
        hd.kind, hd.classes = LP_HEAD_LN_LINEAR, cfg["vocab"]
    else:
        m.family = LP_FAMILY_RESNET
        m.in_channels, m.height, m.width = cfg["in_channels"], cfg["height"], cfg["width"]
        m.stem_channels = cfg["stem_channels"]
        a = _ints(cfg["stage_channels"])
        keep.append(a)
        m.stage_channels = a
        m.block_kind = LP_BLOCK_BOTTLENECK if cfg.get("block") == "bottleneck" else LP_BLOCK_BASIC
        if isinstance(cfg["blocks_per_stage"], (list, tuple)):
            sb = _ints(cfg["blocks_per_stage"])
            keep.append(sb)
            m.stage_blocks, m.blocks_per_stage = sb, max(cfg["blocks_per_stage"])
        else:
            m.blocks_per_stage = cfg["blocks_per_stage"]
        K = len(cfg["stage_channels"])
        hd.kind = LP_HEAD_BN_RELU_GAP_LINEAR if cfg.get("head") == "bn_relu_gap" else LP_HEAD_GAP_LINEAR
        hd.classes = cfg["classes"]
    o = cfg["optim"]
    op = lp_optim_spec()
    if o["kind"] == "sgdm":
        op.kind, op.lr, op.momentum, op.weight_decay = LP_OPT_SGDM, o["lr"], o["momentum"], o.get("weight_decay", 0.0)
    else:
        op.kind, op.lr, op.beta1, op.beta2, op.eps = LP_OPT_ADAM, o["lr"], o["beta1"], o["beta2"], o["eps"]
    m._keep = keep
    return m, K, hd, op


LP_ALLOC_FN = C.CFUNCTYPE(C.c_void_p, C.c_size_t, C.c_void_p)
LP_RELEASE_FN = C.CFUNCTYPE(None, C.c_void_p, C.c_void_p)


class lp_alloc(C.Structure):
    """Optional allocator for the handle's device memory: alloc(bytes, user) -> device pointer aligned
    to 256 bytes or NULL, release(ptr, user).  Keep the object alive as long as the handle."""
    _fields_ = [("alloc", LP_ALLOC_FN), ("release", LP_RELEASE_FN), ("user", C.c_void_p)]


def lp_create(model: lp_model_spec, K: int, head: lp_head_spec, optim: lp_optim_spec, alloc: lp_alloc | None = None) -> int:
    h = C.c_void_p()
    code = _lib.lp_create(C.byref(model), K, C.byref(head), C.byref(optim), C.byref(alloc) if alloc is not None else None,
                          C.byref(h))
    _check(None, code)
    return h.value


def lp_destroy(h):
    _check(h, _lib.lp_destroy(h))


def lp_step(h, x, y, schedule, stream, out_losses):
    _check(h, _lib.lp_step(h, _ptr(x), _ptr(y), schedule, stream, _ptr(out_losses)))


def lp_step_host(h, x_host, y_host, schedule, stream, out_losses_host):
    _check(h, _lib.lp_step_host(h, _ptr(x_host), _ptr(y_host), schedule, stream, _ptr(out_losses_host)))


def lp_forward(h, x, y, stream, out_logits, out_losses):
    _check(h, _lib.lp_forward(h, _ptr(x), _ptr(y), stream, _ptr(out_logits), _ptr(out_losses)))


LP_BN_BATCH, LP_BN_RUNNING = 0, 1


def lp_evaluate(h, x, y, stream, out_losses=None, out_correct=None, out_pred=None, bn_mode=LP_BN_BATCH):
    _check(h, _lib.lp_evaluate(h, _ptr(x), _ptr(y), stream, bn_mode, _ptr(out_losses), _ptr(out_correct), _ptr(out_pred)))


def lp_num_tensors(h) -> int:
    return _lib.lp_num_tensors(h)


def lp_tensor_info_get(h, i) -> dict:
    info = lp_tensor_info()
    _check(h, _lib.lp_tensor_info_get(h, i, C.byref(info)))
    return dict(name=info.name.decode(), chunk=info.chunk, shape=tuple(info.shape[:info.ndim]),
                numel=info.numel, has_working_bf16=bool(info.has_working_bf16))


def lp_get_tensor(h, i, which, host_array: np.ndarray, stream=None):
    _check(h, _lib.lp_get_tensor(h, i, which, host_array.ctypes.data, host_array.nbytes, stream))


def lp_set_tensor(h, i, which, host_array: np.ndarray, stream=None):
    _check(h, _lib.lp_set_tensor(h, i, which, host_array.ctypes.data, host_array.nbytes, stream))


def lp_reset_pipeline(h):
    _check(h, _lib.lp_reset_pipeline(h))


LP_RAMP_PRIME, LP_RAMP_IDLE = 0, 1


def lp_set_ramp(h, ramp: int):
    _check(h, _lib.lp_set_ramp(h, ramp))


def lp_set_drain(h, idle_first: int):
    _check(h, _lib.lp_set_drain(h, idle_first))


def lp_set_fused_step(h, on: bool):
    _check(h, _lib.lp_set_fused_step(h, 1 if on else 0))


def lp_chunk_output_bytes(h, k: int) -> int:
    return _lib.lp_chunk_output_bytes(h, k)


def lp_chunk_output(h, k: int, dst, nbytes: int, stream=None):
    _check(h, _lib.lp_chunk_output(h, k, _ptr(dst), nbytes, stream))


def lp_set_overlap(h, on: bool):
    _check(h, _lib.lp_set_overlap(h, 1 if on else 0))


def lp_status_poll(h, stream=None):
    _check(h, _lib.lp_status_poll(h, stream))


def lp_state_size(h) -> int:
    return _lib.lp_state_size(h)


def lp_save_state(h, host_array: np.ndarray):
    _check(h, _lib.lp_save_state(h, host_array.ctypes.data, host_array.nbytes))


def lp_load_state(h, host_array: np.ndarray):
    _check(h, _lib.lp_load_state(h, host_array.ctypes.data, host_array.nbytes))


def lp_profile_enable(h, on: bool):
    _lib.lp_profile_enable.argtypes = [C.c_void_p, C.c_int]
    _check(h, _lib.lp_profile_enable(h, 1 if on else 0))


def lp_profile_read(h) -> dict:
    """{class name: (milliseconds, algorithmic work, launches)} accumulated since the last read."""
    n = len(LP_KIND_NAMES)
    ms, work, launches = (C.c_double * n)(), (C.c_double * n)(), (C.c_int * n)()
    _lib.lp_profile_read.argtypes = [C.c_void_p, C.POINTER(C.c_double), C.POINTER(C.c_double), C.POINTER(C.c_int)]
    _check(h, _lib.lp_profile_read(h, ms, work, launches))
    return {LP_KIND_NAMES[i]: (ms[i], work[i], launches[i]) for i in range(n)}


def lp_last_step_launches(h) -> int:
    return _lib.lp_last_step_launches(h)


def lp_device_bytes(h) -> int:
    return _lib.lp_device_bytes(h)


def lp_last_error(h=None) -> str:
    return (_lib.lp_last_error(h) or b"").decode()


class lp_gemm_desc(C.Structure):
    _fields_ = [("A", C.c_void_p), ("B", C.c_void_p), ("C", C.c_void_p), ("C2", C.c_void_p),
                ("bias", C.c_void_p), ("resid", C.c_void_p), ("aux", C.c_void_p),
                ("M", C.c_int), ("N", C.c_int), ("K", C.c_int),
                ("a_ms", C.c_longlong), ("a_ks", C.c_longlong), ("b_ns", C.c_longlong), ("b_ks", C.c_longlong),
                ("ldc", C.c_int), ("act", C.c_int), ("out_f32", C.c_int)]


_lib.lp_gemm_bf16.argtypes = [C.c_int, C.POINTER(lp_gemm_desc), C.c_int, C.c_void_p, C.POINTER(C.c_int)]


def lp_gemm_bf16(descs: list, backend: int = 0, stream=None) -> int:
    """One grouped launch of bf16 GEMM problems (list of dicts with the fields of lp_gemm_desc;
    pointers may be torch tensors).  Returns how many problems ran on the tensor-core kernel."""
    arr = (lp_gemm_desc * len(descs))()
    for d, q in zip(arr, descs):
        for k, v in q.items():
            setattr(d, k, _ptr(v) if k in ("A", "B", "C", "C2", "bias", "resid", "aux") else int(v))
    used = C.c_int(0)
    _check(None, _lib.lp_gemm_bf16(len(descs), arr, backend, stream, C.byref(used)))
    return used.value


LP_GEMM_STATIC_MAX = 64
LP_CONV_FORWARD, LP_CONV_INPUT_GRAD, LP_CONV_FILTER_GRAD = 0, 1, 2
_lib.lp_conv3x3_bf16.argtypes = [C.c_int, C.c_void_p, C.c_void_p, C.c_void_p, C.c_int, C.c_int, C.c_int, C.c_int, C.c_int,
                                 C.c_void_p]


def lp_conv3x3_bf16(form: int, act, other, out, n: int, h: int, w: int, c_in: int, c_out: int, stream=None) -> None:
    """One implicit-GEMM 3x3 convolution (stride 1, padding 1) over bf16 NHWC tensors: forward, input
    gradient or filter gradient (see lp.h).  Tensors may be torch tensors or raw device pointers."""
    _check(None, _lib.lp_conv3x3_bf16(form, _ptr(act), _ptr(other), _ptr(out), n, h, w, c_in, c_out, stream))


LP_ATTN_FORWARD, LP_ATTN_BACKWARD = 0, 1
_lib.lp_attention_bf16.argtypes = [C.c_int] + [C.c_void_p] * 6 + [C.c_int] * 3 + [C.c_void_p]


def lp_attention_bf16(form: int, qkv, o, lse, dout, dqkv, delta, batch: int, seq_len: int, n_heads: int, stream=None) -> None:
    """Causal attention with heads of 64 over bf16 [batch, seq_len, 3*64*n_heads] (see lp.h): forward writes o and
    lse; backward reads them and dout and writes dqkv and delta.  Tensors may be torch tensors or raw pointers."""
    _check(None, _lib.lp_attention_bf16(form, _ptr(qkv), _ptr(o), _ptr(lse), _ptr(dout), _ptr(dqkv), _ptr(delta),
                                        batch, seq_len, n_heads, stream))


_lib.lp_conv2d_bf16.argtypes = [C.c_int, C.c_void_p, C.c_void_p, C.c_void_p] + [C.c_int] * 7 + [C.c_void_p]


def lp_conv2d_bf16(form: int, act, other, out, n: int, h: int, w: int, c_in: int, c_out: int, ksize: int, stride: int,
                   stream=None) -> None:
    """One implicit-GEMM convolution over bf16 NHWC tensors: 3x3 (padding 1) or 1x1, stride 1 or 2; forward, filter
    gradient, or (3x3 stride 1) input gradient (see lp.h)."""
    _check(None, _lib.lp_conv2d_bf16(form, _ptr(act), _ptr(other), _ptr(out), n, h, w, c_in, c_out, ksize, stride, stream))


_lib.lp_gemm_bf16_static.argtypes = [C.c_int, C.POINTER(lp_gemm_desc), C.c_void_p]
_lib.lp_gemm_static_last_error.restype = C.c_char_p


def lp_gemm_bf16_static(descs: list, stream=None) -> None:
    """lp_gemm_bf16 for callers that must not allocate device memory (a serving or real-time loop
    that may not take the driver's allocator lock, a plug-in whose host has handed out the whole
    device-memory budget): the problem table lives in a fixed array inside the library, at most
    LP_GEMM_STATIC_MAX problems per call.  Same descriptor dictionaries as lp_gemm_bf16.  Calls on
    one stream are ordered; calls that could overlap on the GPU share that array and race."""
    arr = (lp_gemm_desc * len(descs))()
    for d, q in zip(arr, descs):
        for k, v in q.items():
            setattr(d, k, _ptr(v) if k in ("A", "B", "C", "C2", "bias", "resid", "aux") else int(v))
    code = _lib.lp_gemm_bf16_static(len(descs), arr, stream)
    if code != LP_OK:
        raise LpError(code, (_lib.lp_gemm_static_last_error() or b"").decode())


_lib.lp_gemm_static_poll.argtypes = [C.c_void_p]


def lp_gemm_static_poll(stream=None) -> None:
    """Synchronise `stream`, read and clear the status word of lp_gemm_bf16_static's array; raises
    LpError (TIMEOUT) if a device-side wait of a call since the last poll gave up."""
    code = _lib.lp_gemm_static_poll(stream)
    if code != LP_OK:
        raise LpError(code, (_lib.lp_gemm_static_last_error() or b"").decode())


# ---- FLOP cost model (App. A): host arithmetic in the library, no device needed -------------------------
LP_COST_METHODS = {"backprop": 0, "greedy": 1, "overlapping": 2, "chunked": 3, "last_layers": 4}


class lp_cost_spec(C.Structure):
    _fields_ = [("method", C.c_int), ("layers", C.c_longlong), ("chunks", C.c_longlong),
                ("batch_size", C.c_longlong), ("steps", C.c_longlong), ("forward_cost", C.c_double),
                ("aux_cost", C.c_double), ("backward_multiplier", C.c_double), ("parameters", C.c_double)]


class lp_cost_result(C.Structure):
    _fields_ = [("cost_per_example", C.c_double), ("total_flops", C.c_double), ("parallelism", C.c_double),
                ("sequential_flops", C.c_double)]


_lib.lp_cost_model.argtypes = [C.POINTER(lp_cost_spec), C.POINTER(lp_cost_result)]
_lib.lp_cost_model.restype = C.c_int
_lib.lp_mlp_layer_flops.argtypes = [C.c_longlong, C.c_longlong]
_lib.lp_mlp_layer_flops.restype = C.c_double
_lib.lp_mlp_aux_flops.argtypes = [C.c_longlong, C.c_longlong]
_lib.lp_mlp_aux_flops.restype = C.c_double


def lp_cost_model(method: str, layers: int, batch_size: int, steps: int, forward_cost: float, aux_cost: float,
                  backward_multiplier: float, parameters: float, chunks: int = 1) -> dict:
    spec = lp_cost_spec(LP_COST_METHODS[method], layers, chunks, batch_size, steps, forward_cost, aux_cost,
                        backward_multiplier, parameters)
    out = lp_cost_result()
    _check(None, _lib.lp_cost_model(C.byref(spec), C.byref(out)))
    return {k: getattr(out, k) for k, _ in lp_cost_result._fields_}


def lp_mlp_layer_flops(input_size: int, units: int) -> float:
    return _lib.lp_mlp_layer_flops(input_size, units)


def lp_mlp_aux_flops(units: int, classes: int) -> float:
    return _lib.lp_mlp_aux_flops(units, classes)
