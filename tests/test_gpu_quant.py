"""GPU parity: q4_quant_params / q4_quantize / q4_dequantize against the float-boundary
oracle.  Codes, zero points and packed bytes are compared bit for bit; the scale and the
scaled-back floats too, because both sides use the same correctly rounded binary32
operations in the same order (tolerance 0, stated here on purpose)."""
import numpy as np
import pytest

import oracle
from paper_2009_06488_b200 import workloads as wl

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def q4():
    from paper_2009_06488_b200 import binding
    return binding


def dev(a):
    import torch
    return torch.from_numpy(np.ascontiguousarray(a)).cuda()


def params_on_gpu(q4, Xd):
    import torch
    qp = torch.full((2,), 0x5A5A5A5A, dtype=torch.int32, device="cuda")
    q4.q4_quant_params(Xd, qp)
    h = qp.cpu().numpy()
    return qp, h[:1].view(np.float32)[0], int(h[1])


SHAPES = [(1, 8), (3, 40), (7, 33), (64, 256), (5, 1001), (300, 264), (1, 1 << 20), (1025, 72)]


@pytest.mark.parametrize("shape", SHAPES)
@pytest.mark.parametrize("kind", ["signed", "nonneg", "neg", "zeros"])
def test_quantizer_matches_oracle(q4, shape, kind):
    import torch
    rows, cols = shape
    X = wl.rand_floats(17 + rows + cols, rows * cols).reshape(rows, cols)
    if kind == "nonneg":
        X = np.abs(X)
    elif kind == "neg":
        X = -np.abs(X) - np.float32(0.125)
    elif kind == "zeros":
        X = np.zeros_like(X)
    s, z = oracle.quant_params(X)
    Xd = dev(X)
    qp, gs, gz = params_on_gpu(q4, Xd)
    assert gs == s and gz == z
    kb = (cols + 1) // 2
    for ldq in (kb, (kb + 15) // 16 * 16 + 16):
        Q = torch.full((rows, ldq), 0xA5, dtype=torch.uint8, device="cuda")
        q4.q4_quantize(Xd, qp, Q[:, :ldq] if ldq == kb else Q)
        got = Q.cpu().numpy()
        want = oracle.quantize(X, s, z, ldq)
        assert (got[:, :kb] == want[:, :kb]).all()
        assert (got[:, kb:] == 0xA5).all()             # bytes past the row are not touched


def test_quantizer_on_a_strided_view(q4):
    import torch
    X = wl.rand_floats(5, 37 * 80).reshape(37, 80)
    Xd = dev(X)[:, 8:72]                                # pitch 80, 64 columns, 32-byte offset
    Xv = X[:, 8:72]
    s, z = oracle.quant_params(Xv)
    qp, gs, gz = params_on_gpu(q4, Xd)
    assert (gs, gz) == (s, z)
    Q = torch.zeros((37, 48), dtype=torch.uint8, device="cuda")
    q4.q4_quantize(Xd, qp, Q)
    assert (Q.cpu().numpy() == oracle.quantize(Xv, s, z, 48)).all()


def test_caller_supplied_parameters(q4):
    """A calibrated layer uploads its own scale and zero point; out-of-range values clamp."""
    import torch
    X = (wl.rand_floats(9, 4096).reshape(16, 256) * np.float32(40)).astype(np.float32)
    s, z = np.float32(0.37), 6
    words = np.array([np.float32(s).view(np.int32), z], dtype=np.int32)
    Q = torch.zeros((16, 128), dtype=torch.uint8, device="cuda")
    q4.q4_quantize(dev(X), dev(words), Q)
    assert (Q.cpu().numpy() == oracle.quantize(X, s, z)).all()


@pytest.mark.parametrize("shape", [(1, 4), (3, 7), (64, 64), (300, 264), (1000, 1000)])
def test_scale_back_matches_oracle(q4, shape):
    import torch
    rows, cols = shape
    rng = np.random.default_rng(rows * 131 + cols)
    C = rng.integers(-(1 << 26), 1 << 26, size=shape).astype(np.int32)
    C[0, 0] = (1 << 24) + 1                             # not a float32: must round, not truncate
    scale = np.float32(3.1e-4)
    R = torch.full((rows, cols + 4), 7.0, dtype=torch.float32, device="cuda")
    q4.q4_dequantize(dev(C), float(scale), R[:, :cols])
    got = R.cpu().numpy()
    assert (got[:, :cols] == oracle.dequantize(C, scale)).all()
    assert (got[:, cols:] == 7.0).all()


def test_float_in_float_out_layer(q4):
    """F -> Q -> F: quantize activations and weights, multiply with q4_gemm, scale back
    (Section III-B), every stage equal to the oracle's."""
    import torch
    M, N, K = 160, 72, 200
    Xf = wl.rand_floats(21, M * K).reshape(M, K)
    Wf = wl.rand_floats(22, N * K).reshape(N, K) * np.float32(0.1)
    sx, zx = oracle.quant_params(Xf)
    sw, zw = oracle.quant_params(Wf)
    A, Bt = oracle.quantize(Xf, sx, zx), oracle.quantize(Wf, sw, zw)
    want = oracle.dequantize(oracle.gemm(A, Bt, M, N, K, zx, zw), np.float32(sx * sw))

    Xd, Wd = dev(Xf), dev(Wf)
    qpx, gsx, gzx = params_on_gpu(q4, Xd)
    qpw, gsw, gzw = params_on_gpu(q4, Wd)
    Ad = torch.empty((M, K // 2), dtype=torch.uint8, device="cuda")
    Bd = torch.empty((N, K // 2), dtype=torch.uint8, device="cuda")
    q4.q4_quantize(Xd, qpx, Ad); q4.q4_quantize(Wd, qpw, Bd)
    C = torch.empty((M, N), dtype=torch.int32, device="cuda")
    q4.q4_gemm(Ad, Bd, C, M, N, K, gzx, gzw)
    R = torch.empty((M, N), dtype=torch.float32, device="cuda")
    q4.q4_dequantize(C, float(np.float32(gsx * gsw)), R)
    assert (R.cpu().numpy() == want).all()
    # and the quantized product approximates the float one (Eq. 2's "~="): loose sanity bound
    exact = Xf.astype(np.float64) @ Wf.astype(np.float64).T
    assert np.abs(want - exact).max() <= K * float(sx) * float(sw) * 15 * 2


def test_float_image_through_the_table2_layers_and_back_to_float(q4):
    """The layer model of Section III-B on the Table II topology with random weights: a float
    image is quantized (F -> Q), five layers hand 4-bit activations to the next (Q -> Q, with
    the fused integer re-quantization), and the last convolution's integer result is scaled
    back to float (Q -> F).  Every stage equals the oracle's."""
    import dataclasses
    import torch
    net = wl.paper_table2_net(batch=5)
    L0 = net.layers[0]
    img = np.abs(wl.rand_floats(31, L0.N * L0.H * L0.W)).reshape(L0.N * L0.H, L0.W)
    s_x, z_x = oracle.quant_params(img)
    assert z_x == 0                                      # non-negative image
    layers = [dataclasses.replace(L0, za=z_x)] + net.layers[1:]
    s_total = np.float32(s_x * np.float32(0.01))         # stand-in for the product of the layers' scales

    # ---- oracle
    Xo = oracle.quantize(img.reshape(1, -1), s_x, z_x).reshape(-1)
    for L in layers[:-1]:
        Xo = oracle_layer(L, Xo).reshape(-1)
    LL = layers[-1]
    do = oracle.ConvDesc(LL.N, LL.H, LL.W, LL.C, LL.OC, LL.KH, LL.KW, LL.stride, LL.stride, LL.pad, LL.pad)
    lda = (LL.K // 2 + 15) // 16 * 16
    Ao, _ = oracle.im2col(Xo, do, LL.za, lda)
    want = oracle.dequantize(oracle.gemm(Ao, LL.Wt, LL.M, LL.OC, LL.K, LL.za, LL.zb), s_total)

    # ---- GPU
    imgd = dev(img)
    qp, gs, gz = params_on_gpu(q4, imgd)
    assert (gs, gz) == (s_x, z_x)
    Xd = torch.zeros((img.size + 1) // 2 + 16, dtype=torch.uint8, device="cuda")
    q4.q4_quantize(imgd.reshape(-1), qp, Xd)
    for L in layers[:-1]:
        d = q4.ConvDesc(L.N, L.H, L.W, L.C, L.OC, L.KH, L.KW, L.stride, L.stride, L.pad, L.pad)
        ws = torch.empty(q4.q4_conv2d_workspace_bytes(d), dtype=torch.uint8, device="cuda")
        Y = torch.zeros((d.M, L.OC // 2), dtype=torch.uint8, device="cuda")
        q4.q4_conv2d(Xd, dev(L.Wt), d, L.za, L.zb,
                     q4.Requant(L.mult, L.shift, L.zo, L.clamp_lo, L.clamp_hi), Y, ws)
        Xd = Y.reshape(-1)
    d = q4.ConvDesc(LL.N, LL.H, LL.W, LL.C, LL.OC, LL.KH, LL.KW, LL.stride, LL.stride, LL.pad, LL.pad)
    A = torch.zeros((d.M, lda), dtype=torch.uint8, device="cuda")
    q4.q4_im2col(Xd, d, LL.za, A, None)
    C = torch.empty((d.M, LL.OC), dtype=torch.int32, device="cuda")
    q4.q4_gemm(A, dev(LL.Wt), C, d.M, LL.OC, d.K, LL.za, LL.zb)
    R = torch.empty((d.M, LL.OC), dtype=torch.float32, device="cuda")
    q4.q4_dequantize(C, float(s_total), R)
    assert q4.q4_last_device_status() == q4.Q4_OK
    assert (R.cpu().numpy() == want).all()


def oracle_layer(L, X):
    do = oracle.ConvDesc(L.N, L.H, L.W, L.C, L.OC, L.KH, L.KW, L.stride, L.stride, L.pad, L.pad)
    return oracle.conv2d(X, L.Wt, L.bias, do, L.za, L.zb,
                         oracle.Requant(L.mult, L.shift, L.zo, L.clamp_lo, L.clamp_hi))


@pytest.mark.parametrize("scale", [0.37, 1.0 / 3.0, 7.3e-5, 1234.567, 0.25, 3.0e-39, 2.5e38, 1.1754944e-38])
def test_codes_at_the_integer_boundaries_of_the_quotient(q4, scale):
    """Inputs that sit on, and a few units in the last place around, every multiple of the
    scale: where the floor of the rounded quotient is decided by the last bit (the kernel's
    division-free path must hand exactly these to the exact division)."""
    import torch
    s = np.float32(scale)
    k = np.arange(-24, 25, dtype=np.float32)
    with np.errstate(over="ignore"):
        base = (k * s).astype(np.float32)               # infinities (largest scale) are replaced below
    vals = [base]
    for _ in range(4):
        vals.append(np.nextafter(vals[-1], np.float32(np.inf)).astype(np.float32))
    lo = base
    for _ in range(4):
        lo = np.nextafter(lo, np.float32(-np.inf)).astype(np.float32)
        vals.append(lo)
    X = np.concatenate(vals + [np.array([0.0, -0.0, 1e-45, -1e-45], np.float32)])
    X = np.resize(X, (X.size + 7) // 8 * 8).reshape(1, -1)
    z = 7
    words = np.array([s.view(np.int32), z], dtype=np.int32)
    with np.errstate(over="ignore", invalid="ignore"):
        want = oracle.quantize(np.where(np.isfinite(X), X, 0).astype(np.float32), s, z)
    Xf = np.where(np.isfinite(X), X, 0).astype(np.float32)
    for cols in (Xf.shape[1], Xf.shape[1] - 3):              # word path and byte path
        Q = torch.zeros((1, (cols + 1) // 2), dtype=torch.uint8, device="cuda")
        q4.q4_quantize(dev(Xf[:, :cols]), dev(words), Q)
        with np.errstate(over="ignore", invalid="ignore"):
            assert (Q.cpu().numpy() == oracle.quantize(Xf[:, :cols], s, z)).all()
