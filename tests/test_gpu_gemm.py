"""The grouped bf16 GEMM kernels against the oracle's Linear layer (forward, input gradient,
weight gradient), on ragged sizes that span several 128x256 tiles and a partial tail."""
import numpy as np
import pytest
import torch

import lp_synth
from oracle import layers as L
from paper_2012_03837_b200 import binding as lp

pytestmark = pytest.mark.gpu


def bf(a):
    return torch.from_numpy(lp_synth.bf16_round(a)).to("cuda").to(torch.bfloat16).contiguous()


def problems(M, N, K, rng):
    """Forward, dgrad and wgrad problems of one Linear layer y = x W^T + b with their oracle results."""
    x = lp_synth.bf16_round(rng.standard_normal((M, K)).astype(np.float32))
    W = lp_synth.bf16_round((rng.standard_normal((N, K)) / np.sqrt(K)).astype(np.float32))
    b = rng.standard_normal(N).astype(np.float32)
    dy = lp_synth.bf16_round(rng.standard_normal((M, N)).astype(np.float32))
    y, cache = L.linear_fwd(x.astype(np.float64), W.astype(np.float64), b.astype(np.float64))
    dx, dW, _ = L.linear_bwd(dy.astype(np.float64), cache)
    t = dict(x=bf(x), W=bf(W), dy=bf(dy), b=torch.from_numpy(b).cuda(),
             y=torch.zeros(M, N, dtype=torch.bfloat16, device="cuda"),
             dx=torch.zeros(M, K, dtype=torch.bfloat16, device="cuda"),
             dW=torch.zeros(N, K, dtype=torch.float32, device="cuda"))
    descs = [
        dict(A=t["x"], B=t["W"], C=t["y"], bias=t["b"], M=M, N=N, K=K, a_ms=K, a_ks=1, b_ns=K, b_ks=1, ldc=N),
        dict(A=t["dy"], B=t["W"], C=t["dx"], M=M, N=K, K=N, a_ms=N, a_ks=1, b_ns=1, b_ks=K, ldc=K),
        dict(A=t["dy"], B=t["x"], C=t["dW"], M=N, N=K, K=M, a_ms=1, a_ks=N, b_ns=1, b_ks=K, ldc=K, out_f32=1),
    ]
    return t, descs, dict(y=y, dx=dx, dW=dW)


def check(t, ref, tag):
    for name in ("y", "dx", "dW"):
        got = t[name].float().cpu().numpy().astype(np.float64)
        scale = np.abs(ref[name]).max()
        err = np.abs(got - ref[name]).max() / scale
        tol = 1e-2 if name != "dW" else 1e-4     # bf16 outputs carry one rounding (2^-9); fp32 output does not
        assert err < tol, (tag, name, err)


@pytest.mark.parametrize("backend", [1, 0])
@pytest.mark.parametrize("M,N,K", [(128, 256, 64), (256, 512, 128), (200, 264, 72), (1000, 520, 328), (136, 1000, 2048),
                                   # long reductions with 512-column outputs: the 256x512 tiles (input gradient over
                                   # 8192 columns; weight gradient over 8200 rows, ragged last k-slice)
                                   (264, 8192, 512), (8200, 512, 1024),
                                   # at most 128 output columns: column tiles of 64 and 128 (K-major B in 32-row boxes
                                   # per CTA of a pair; MN-major B in 64-column blocks), ragged in both directions
                                   (520, 64, 192), (300, 128, 64), (136, 96, 256), (1000, 40, 136)])
def test_linear_products(M, N, K, backend):
    rng = np.random.default_rng(M + N + K)
    t, descs, ref = problems(M, N, K, rng)
    used = 0
    for d in descs:                      # one launch per product
        used += lp.lp_gemm_bf16([d], backend)
    torch.cuda.synchronize()
    assert used == (0 if backend else 3)
    check(t, ref, (M, N, K, backend))


def test_grouped_launch_of_mixed_problems():
    rng = np.random.default_rng(7)
    sets = [problems(*s, rng) for s in [(256, 256, 128), (200, 264, 72), (384, 1000, 256)]]
    descs = [d for _, ds, _ in sets for d in ds]
    assert lp.lp_gemm_bf16(descs, 0) == len(descs)
    torch.cuda.synchronize()
    for i, (t, _, ref) in enumerate(sets):
        check(t, ref, i)


def test_epilogues_match_between_backends():
    """Bias + residual + GELU (two outputs), ReLU mask and GELU' epilogues: tensor-core kernel vs FP32-ALU kernel."""
    rng = np.random.default_rng(3)
    M, N, K = 264, 520, 136
    x, W = bf(rng.standard_normal((M, K)).astype(np.float32)), bf((rng.standard_normal((N, K)) / 12).astype(np.float32))
    b = torch.from_numpy(rng.standard_normal(N).astype(np.float32)).cuda()
    r = bf(rng.standard_normal((M, N)).astype(np.float32))
    aux = bf(rng.standard_normal((M, N)).astype(np.float32))
    outs = {}
    for backend in (1, 0):
        res = []
        for act in (1, 2, 3, 4):
            c = torch.zeros(M, N, dtype=torch.bfloat16, device="cuda")
            c2 = torch.zeros(M, N, dtype=torch.bfloat16, device="cuda")
            d = dict(A=x, B=W, C=c, C2=c2, bias=b, resid=r, aux=aux, M=M, N=N, K=K, a_ms=K, a_ks=1, b_ns=K, b_ks=1, ldc=N, act=act)
            lp.lp_gemm_bf16([d], backend)
            res += [c, c2]
        torch.cuda.synchronize()
        outs[backend] = [t.float().cpu().numpy() for t in res]
    for a, b_ in zip(outs[0], outs[1]):
        assert np.abs(a - b_).max() <= 2e-2 * max(1.0, np.abs(b_).max())
    # and each backend's GELU output equals the oracle's GELU of its own stored pre-activation (the tensor-core
    # epilogue evaluates Phi as the logistic function of a fitted quintic: 3e-5 from the erf form, below the bf16
    # step of the stored value)
    for backend in (1, 0):
        u, g = outs[backend][3], outs[backend][2]
        want = L.gelu_fwd(u.astype(np.float64))[0]
        assert np.abs(lp_synth.bf16_round(want.astype(np.float32)) - g).max() <= 2.0 ** -8 * max(1.0, np.abs(want).max()), backend
    # every epilogue against the oracle's layers, from the bf16 operands: z = x W^T + b + r
    xf, Wf = x.float().cpu().numpy().astype(np.float64), W.float().cpu().numpy().astype(np.float64)
    z = L.linear_fwd(xf, Wf, b.cpu().numpy().astype(np.float64))[0] + r.float().cpu().numpy().astype(np.float64)
    a64 = aux.float().cpu().numpy().astype(np.float64)
    refs = {0: L.relu_fwd(z)[0],                                   # act 1
            2: L.gelu_fwd(lp_synth.bf16_round(z.astype(np.float32)).astype(np.float64))[0],   # act 2: GELU of the stored u
            3: z,                                                  # act 2: C2 = the pre-activation
            4: np.where(a64 > 0, z, 0.0),                          # act 3: ReLU mask on aux
            6: L.gelu_bwd(z, (a64,))}                              # act 4: z * GELU'(aux)
    for backend in (1, 0):
        for i, want in refs.items():
            got = outs[backend][i].astype(np.float64)
            assert np.abs(got - want).max() <= 1e-2 * max(1.0, np.abs(want).max()), (backend, i)


# ------------------------------------------------------------------ implicit-GEMM 3x3 convolution

@pytest.mark.parametrize("n,h,w,c_in,c_out", [
    (3, 16, 16, 64, 128),     # boxes of 8 (4) rows inside an image; 768 pixels = three 256-row tiles
    (5, 8, 8, 128, 64),       # 128-pixel boxes span two images; 320 pixels: ragged last tile, box past the last image
    (9, 4, 4, 64, 64),        # boxes of eight (four) whole images; 144 pixels
    (2, 32, 32, 64, 72),      # four (two) rows of a 32 x 32 image per box; output channels not a multiple of 64
])
def test_implicit_convolution_against_the_oracle(n, h, w, c_in, c_out):
    """Forward, input gradient and filter gradient of a 3x3 stride-1 convolution (App. B.3's residual blocks)
    through lp_conv3x3_bf16 against the oracle's convolution, element by element."""
    rng = np.random.default_rng(n * 1000 + h * 10 + c_in)
    x = lp_synth.bf16_round(rng.standard_normal((n, c_in, h, w)).astype(np.float32))                   # NCHW (oracle layout)
    W = lp_synth.bf16_round((rng.standard_normal((c_out, c_in, 3, 3)) / np.sqrt(9 * c_in)).astype(np.float32))
    dy = lp_synth.bf16_round(rng.standard_normal((n, c_out, h, w)).astype(np.float32))
    y_ref, cache = L.conv2d_fwd(x.astype(np.float64), W.astype(np.float64), 1, 1)
    dx_ref, dW_ref = L.conv2d_bwd(dy.astype(np.float64), cache)
    nhwc = lambda a: np.ascontiguousarray(a.transpose(0, 2, 3, 1))
    xd, dyd = bf(nhwc(x)), bf(nhwc(dy))
    Wd = bf(np.ascontiguousarray(W.transpose(0, 2, 3, 1)))                                             # [c_out, 3, 3, c_in]
    y = torch.zeros(n, h, w, c_out, dtype=torch.bfloat16, device="cuda")
    dx = torch.zeros(n, h, w, c_in, dtype=torch.bfloat16, device="cuda")
    dW = torch.zeros(c_out, 3, 3, c_in, dtype=torch.float32, device="cuda")
    lp.lp_conv3x3_bf16(lp.LP_CONV_FORWARD, xd, Wd, y, n, h, w, c_in, c_out)
    if c_out % 64 == 0:
        lp.lp_conv3x3_bf16(lp.LP_CONV_INPUT_GRAD, dyd, Wd, dx, n, h, w, c_in, c_out)
    lp.lp_conv3x3_bf16(lp.LP_CONV_FILTER_GRAD, xd, dyd, dW, n, h, w, c_in, c_out)
    torch.cuda.synchronize()
    got = dict(y=y.float().cpu().numpy().transpose(0, 3, 1, 2), dW=dW.cpu().numpy().transpose(0, 3, 1, 2))
    ref = dict(y=y_ref, dW=dW_ref)
    if c_out % 64 == 0:
        got["dx"], ref["dx"] = dx.float().cpu().numpy().transpose(0, 3, 1, 2), dx_ref
    for name in got:
        err = np.abs(got[name].astype(np.float64) - ref[name]).max() / np.abs(ref[name]).max()
        tol = 1e-2 if name != "dW" else 1e-4     # bf16 outputs carry one rounding (2^-9); the fp32 output does not
        assert err < tol, (name, err)


@pytest.mark.parametrize("n,h,w,c_in,c_out,ksize,stride", [
    (3, 32, 32, 64, 128, 3, 2),    # first convolution of a stage: 32x32 -> 16x16, boxes step through the input by 2
    (6, 16, 16, 128, 256, 3, 2),   # 16x16 -> 8x8: 128-pixel boxes span two output images
    (20, 8, 8, 256, 128, 3, 2),    # 8x8 -> 4x4: boxes of eight (four) whole output images, ragged last tile
    (3, 32, 32, 64, 128, 1, 2),    # the 1x1 stride-2 shortcut
    (10, 8, 8, 128, 72, 1, 2),     # ... across images, output channels not a multiple of 64
    (2, 16, 16, 128, 64, 1, 1),    # a 1x1 stride-1 convolution (bottleneck blocks)
])
def test_strided_and_pointwise_implicit_convolutions_against_the_oracle(n, h, w, c_in, c_out, ksize, stride):
    """Forward and filter gradient of the stage-opening convolutions of App. B.3's networks (3x3 stride 2, 1x1
    stride 2) and of 1x1 convolutions, through lp_conv2d_bf16 against the oracle's convolution."""
    rng = np.random.default_rng(n * 1000 + h * 10 + c_in + ksize)
    pad = 1 if ksize == 3 else 0
    ho, wo = (h - 1) // stride + 1, (w - 1) // stride + 1
    x = lp_synth.bf16_round(rng.standard_normal((n, c_in, h, w)).astype(np.float32))
    W = lp_synth.bf16_round((rng.standard_normal((c_out, c_in, ksize, ksize)) / np.sqrt(ksize * ksize * c_in)).astype(np.float32))
    dy = lp_synth.bf16_round(rng.standard_normal((n, c_out, ho, wo)).astype(np.float32))
    y_ref, cache = L.conv2d_fwd(x.astype(np.float64), W.astype(np.float64), stride, pad)
    assert y_ref.shape == (n, c_out, ho, wo)
    _, dW_ref = L.conv2d_bwd(dy.astype(np.float64), cache)
    nhwc = lambda a: np.ascontiguousarray(a.transpose(0, 2, 3, 1))
    xd, dyd = bf(nhwc(x)), bf(nhwc(dy))
    Wd = bf(np.ascontiguousarray(W.transpose(0, 2, 3, 1)))
    y = torch.zeros(n, ho, wo, c_out, dtype=torch.bfloat16, device="cuda")
    dW = torch.zeros(c_out, ksize, ksize, c_in, dtype=torch.float32, device="cuda")
    lp.lp_conv2d_bf16(lp.LP_CONV_FORWARD, xd, Wd, y, n, h, w, c_in, c_out, ksize, stride)
    lp.lp_conv2d_bf16(lp.LP_CONV_FILTER_GRAD, xd, dyd, dW, n, h, w, c_in, c_out, ksize, stride)
    torch.cuda.synchronize()
    got = dict(y=y.float().cpu().numpy().transpose(0, 3, 1, 2), dW=dW.cpu().numpy().transpose(0, 3, 1, 2))
    ref = dict(y=y_ref, dW=dW_ref)
    for name in got:
        err = np.abs(got[name].astype(np.float64) - ref[name]).max() / np.abs(ref[name]).max()
        assert err < (1e-2 if name != "dW" else 1e-4), (name, err)
    with pytest.raises(lp.LpError) as e:                     # no input gradient in this form for a stride
        lp.lp_conv2d_bf16(lp.LP_CONV_INPUT_GRAD, dyd, Wd, y, n, h, w, c_in, c_out, ksize, 2)
    assert lp.LP_ERR[e.value.code] == "UNSUPPORTED"


def test_implicit_convolution_rejects_what_it_cannot_tile():
    t = torch.zeros(1 << 16, dtype=torch.bfloat16, device="cuda")
    for form, args in [(lp.LP_CONV_FORWARD, (2, 12, 12, 64, 64)),       # width does not divide 64
                       (lp.LP_CONV_FORWARD, (2, 16, 16, 32, 64)),       # shifted operand's channels not a multiple of 64
                       (lp.LP_CONV_FORWARD, (3, 12, 16, 64, 64)),       # h*w = 192 neither divides nor is divided by 128
                       (lp.LP_CONV_INPUT_GRAD, (2, 16, 16, 60, 64))]:   # filter columns not 16-byte aligned per tap
        with pytest.raises(lp.LpError) as e:
            lp.lp_conv3x3_bf16(form, t, t, t, *args)
        assert lp.LP_ERR[e.value.code] == "UNSUPPORTED"
