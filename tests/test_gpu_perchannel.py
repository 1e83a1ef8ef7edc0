"""GPU parity: per-output-channel weight zero points and multipliers (q4_gemm with zb = 0, then
q4_requant_channels) against the per-channel oracle, byte for byte."""
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


def channel_params(seed, N, min_shift=0, max_shift=14):
    zb = wl.rand_ints(seed, 4, 0, 15, N).astype(np.int32)
    bias = wl.rand_ints(seed, 3, -512, 512, N).astype(np.int32)
    mult = wl.rand_ints(seed, 5, 1 << 30, (1 << 31) - 1, N).astype(np.int32)
    shift = wl.rand_ints(seed, 6, min_shift, max_shift, N).astype(np.int32)
    return zb, bias, mult, shift


def run(q4, A, Bt, M, N, K, za, zb, bias, mult, shift, zo, lo, hi, ldc_pad=0, ldq_pad=0):
    import torch
    Ad, Bd = dev(A), dev(Bt)
    C0 = torch.empty((M, N + ldc_pad), dtype=torch.int32, device="cuda")
    q4.q4_gemm(Ad, Bd, C0[:, :N] if ldc_pad else C0, M, N, K, za, 0)
    ra = torch.empty(M, dtype=torch.int32, device="cuda")
    q4.q4_row_sums(Ad, M, K, ra)
    Cq = torch.full((M, N // 2 + ldq_pad), 0xA5, dtype=torch.uint8, device="cuda")
    opt = lambda a: None if a is None else dev(a)
    q4.q4_requant_channels(C0[:, :N] if ldc_pad else C0, M, N, K, za, ra, opt(zb), opt(bias), dev(mult),
                           dev(shift), zo, lo, hi, Cq[:, :N // 2] if ldq_pad else Cq)
    out = Cq.cpu().numpy()
    assert (out[:, N // 2:] == 0xA5).all()
    return out[:, :N // 2]


SHAPES = [(1, 2, 1), (64, 64, 256), (130, 70, 100), (300, 264, 1000), (257, 136, 33), (1000, 520, 777),
          (259, 132, 65), (3, 4, 9), (2048, 1024, 512)]     # 132, 4: whole groups of four channels, not of eight


@pytest.mark.parametrize("shape", SHAPES)
@pytest.mark.parametrize("shifts", [(0, 14), (2, 14), (20, 31)])
def test_gemm_with_per_channel_parameters(q4, shape, shifts):
    M, N, K = shape
    seed = 9000 + sum(shape)
    c = wl.gemm_case("pc", M, N, K, seed=seed)
    zb, bias, mult, shift = channel_params(seed, N, *shifts)
    want = oracle.requant_channels(oracle.gemm_channels(c.A, c.Bt, M, N, K, c.za, zb, bias), mult, shift, 3, 1, 14)
    pad = 4 if M % 2 else 0
    got = run(q4, c.A, c.Bt, M, N, K, c.za, zb, bias, mult, shift, 3, 1, 14, ldc_pad=pad, ldq_pad=pad)
    assert (got == want).all()


FUSED_SHAPES = [(64, 64, 256), (130, 72, 100), (300, 264, 1000), (257, 136, 33), (1000, 520, 777),
                (256, 192, 128), (700, 200, 257), (512, 768, 64), (2048, 1024, 512)]


@pytest.mark.parametrize("variant", [3, 5, 6])       # single-CTA / CTA-pair kernel with 192- and 256-column tiles
@pytest.mark.parametrize("shape", FUSED_SHAPES)
@pytest.mark.parametrize("shifts", [(0, 14), (2, 14), (20, 31)])
def test_per_channel_parameters_in_the_gemm_epilogue(q4, variant, shape, shifts):
    """q4_gemm_requant_channels: the per-channel finish inside the GEMM kernel, against the
    per-channel oracle, with and without a workspace and given sums."""
    import torch
    M, N, K = shape
    seed = 9100 + sum(shape)
    ld = ((K + 1) // 2 + 15) // 16 * 16
    c = wl.gemm_case("pc", M, N, K, seed=seed, lda=ld, ldb=ld)
    zb, bias, mult, shift = channel_params(seed, N, *shifts)
    want = oracle.requant_channels(oracle.gemm_channels(c.A, c.Bt, M, N, K, c.za, zb, bias), mult, shift, 3, 1, 14)
    Ad, Bd = dev(c.A), dev(c.Bt)
    q4.q4_set_variant(variant)
    try:
        for use_ws, sums in ((False, False), (True, False), (False, True)):
            Cq = torch.full((M, N // 2 + 16), 0xA5, dtype=torch.uint8, device="cuda")
            ws = torch.full((q4.q4_gemm_workspace_bytes(M, N, K),), 0xA5, dtype=torch.uint8, device="cuda") \
                if use_ws else None
            ra = cb = None
            if sums:
                ra = q4.q4_row_sums(Ad, M, K, torch.empty(M, dtype=torch.int32, device="cuda"))
                cb = q4.q4_row_sums(Bd, N, K, torch.empty(N, dtype=torch.int32, device="cuda"))
            q4.q4_gemm_requant_channels(Ad, Bd, Cq[:, :N // 2], M, N, K, c.za, dev(zb), dev(mult), dev(shift),
                                        3, 1, 14, dev(bias), ra, cb, ws)
            assert q4.q4_last_device_status() == q4.Q4_OK
            out = Cq.cpu().numpy()
            assert (out[:, :N // 2] == want).all()
            assert (out[:, N // 2:] == 0xA5).all()
    finally:
        q4.q4_set_variant(0)


def test_per_channel_gemm_epilogue_at_the_benchmark_shape(q4):
    """8192^3 through the CTA-pair kernel: the whole packed matrix against the per-channel
    oracle's finishing pass applied to an int32 product (zb = 0) that exact Freivalds checks
    and sampled oracle rows have verified."""
    import torch
    c = wl.c2(8192)
    n = 8192
    zb, bias, mult, shift = channel_params(77, n, 8, 16)
    A, Bt = dev(c.A), dev(c.Bt)
    C0 = torch.empty((n, n), dtype=torch.int32, device="cuda")
    ws = torch.empty(q4.q4_gemm_workspace_bytes(n, n, n), dtype=torch.uint8, device="cuda")
    q4.q4_gemm(A, Bt, C0, n, n, n, c.za, 0, ws=ws)
    got0 = C0.cpu().numpy()
    del C0
    rows = np.unique(np.concatenate([np.random.default_rng(5).integers(0, n, 24), [0, 255, 256, n - 1]]))
    assert (got0[rows] == oracle.gemm(np.ascontiguousarray(c.A[rows]), c.Bt, len(rows), n, n, c.za, 0)).all()
    r = np.random.default_rng(6).integers(1, 1 << 20, n).astype(np.int64)
    y = np.zeros(n, np.int64)
    for n0 in range(0, n, 1024):
        y += oracle.unpack_rows(c.Bt[n0:n0 + 1024], n).astype(np.int64).T @ r[n0:n0 + 1024]
    for m0 in range(0, n, 1024):
        a = oracle.unpack_rows(c.A[m0:m0 + 1024], n).astype(np.int64) - c.za
        assert (got0[m0:m0 + 1024].astype(np.int64) @ r == a @ y).all()
    ra = oracle.unpack_rows(c.A, n).astype(np.int64).sum(axis=1)
    # the oracle's finishing pass: acc = C0 - zb[n] (rowsum - K za) + bias[n], then per-channel requant
    acc = got0.astype(np.int64) - zb.astype(np.int64)[None, :] * (ra - n * c.za)[:, None] + bias[None, :]
    want = oracle.requant_channels(acc.astype(np.int32), mult, shift, 0, 0, 15)
    Cq = torch.empty((n, n // 2), dtype=torch.uint8, device="cuda")
    q4.q4_gemm_requant_channels(A, Bt, Cq, n, n, n, c.za, dev(zb), dev(mult), dev(shift), 0, 0, 15,
                                dev(bias), ws=ws)
    assert q4.q4_last_device_status() == q4.Q4_OK
    assert (Cq.cpu().numpy() == want).all()


def test_optional_arrays_and_uniform_channels_match_the_fused_path(q4):
    """No zero points and no bias: the plain product; one zero point for every channel: the
    same bytes as q4_gemm_requant's fused epilogue."""
    import torch
    M, N, K = 200, 136, 520
    c = wl.gemm_case("pc", M, N, K, seed=12, lda=272, ldb=272)
    _, _, mult, shift = channel_params(12, N, 2)
    want = oracle.requant_channels(oracle.gemm_channels(c.A, c.Bt, M, N, K, c.za, [0] * N), mult, shift, 0, 0, 15)
    assert (run(q4, c.A, c.Bt, M, N, K, c.za, None, None, mult, shift, 0, 0, 15) == want).all()
    zb1 = np.full(N, c.zb, np.int32)
    m1, s1 = np.full(N, c.mult, np.int32), np.full(N, 7, np.int32)
    Cq = torch.empty((M, N // 2), dtype=torch.uint8, device="cuda")
    q4.q4_gemm_requant(dev(c.A), dev(c.Bt), Cq, M, N, K, c.za, c.zb, q4.Requant(c.mult, 7, 2, 0, 15))
    assert (run(q4, c.A, c.Bt, M, N, K, c.za, zb1, None, m1, s1, 2, 0, 15) == Cq.cpu().numpy()).all()


def test_conv_layer_with_per_channel_weights(q4):
    """Explicit path of a layer: q4_im2col (matrix and row sums), q4_gemm with zb = 0,
    q4_requant_channels."""
    import torch
    g = (3, 12, 14, 16, 24, 3, 3, 1, 1, 1, 1)
    N_, H, W, C, OC, KH, KW, sh, sw, ph, pw = g
    dq = q4.ConvDesc(*g)
    do = oracle.ConvDesc(*g)
    K = KH * KW * C
    X = wl.rand_flat_nibbles(31, 1, N_ * H * W * C)
    Wt = wl.rand_packed(31, 2, OC, K)
    zb, bias, mult, shift = channel_params(31, OC, 0)
    za = 6
    lda = (K // 2 + 15) // 16 * 16
    Ao, _ = oracle.im2col(X, do, za, lda)
    want = oracle.requant_channels(oracle.gemm_channels(Ao, Wt, dq.M, OC, K, za, zb, bias), mult, shift, 0, 0, 15)
    A = torch.zeros((dq.M, lda), dtype=torch.uint8, device="cuda")
    ra = torch.empty(dq.M, dtype=torch.int32, device="cuda")
    q4.q4_im2col(dev(X), dq, za, A, ra)
    C0 = torch.empty((dq.M, OC), dtype=torch.int32, device="cuda")
    q4.q4_gemm(A, dev(Wt), C0, dq.M, OC, K, za, 0, ra)
    Y = torch.empty((dq.M, OC // 2), dtype=torch.uint8, device="cuda")
    q4.q4_requant_channels(C0, dq.M, OC, K, za, ra, dev(zb), dev(bias), dev(mult), dev(shift), 0, 0, 15, Y)
    assert (Y.cpu().numpy() == want).all()


def test_argument_checks(q4):
    import torch
    C0 = torch.zeros((4, 8), dtype=torch.int32, device="cuda")
    v = torch.zeros(8, dtype=torch.int32, device="cuda")
    Cq = torch.zeros((4, 4), dtype=torch.uint8, device="cuda")
    with pytest.raises(q4.Q4Error) as e:
        q4.q4_requant_channels(C0, 4, 7, 16, 0, v, None, None, v, v, 0, 0, 15, Cq)       # odd N
    assert e.value.status == q4.Q4_ERR_INVALID_ARG
    with pytest.raises(q4.Q4Error) as e:
        q4.q4_requant_channels(C0, 4, 8, 16, 16, v, None, None, v, v, 0, 0, 15, Cq)      # za out of range
    assert e.value.status == q4.Q4_ERR_RANGE
    with pytest.raises(q4.Q4Error) as e:
        q4.q4_requant_channels(C0, 4, 8, 16, 0, v, None, None, None, v, 0, 0, 15, Cq)    # multipliers missing
    assert e.value.status == q4.Q4_ERR_INVALID_ARG


CONV_PC = [  # N, H, W, C, OC, KH, KW, sh, sw, ph, pw
    (3, 12, 14, 16, 24, 3, 3, 1, 1, 1, 1),      # packed copy
    (4, 16, 16, 8, 16, 3, 3, 2, 2, 1, 1),       # packed copy, stride 2
    (2, 20, 40, 32, 64, 3, 3, 1, 1, 1, 1),      # widest tile
    (5, 16, 16, 1, 8, 3, 3, 1, 1, 1, 1),        # gray-image first layer: four pixels per lane
    (9, 48, 48, 1, 8, 3, 3, 1, 1, 1, 1),        # ... tiles over two images
    (4, 20, 32, 1, 8, 3, 3, 1, 1, 1, 1),        # ... rows copied by bulk copies (16-byte rows)
    (6, 10, 24, 1, 8, 3, 3, 1, 1, 0, 1),        # ... no vertical padding
    (3, 16, 40, 1, 8, 3, 3, 1, 1, 1, 3),        # ... horizontal padding of three
    (5, 12, 20, 1, 8, 3, 3, 1, 1, 0, 0),        # output rows not groups of four: expanded copy, MMA kernel
    (2, 11, 9, 3, 24, 3, 3, 1, 1, 1, 1),        # odd channel count
    (40, 9, 10, 8, 40, 3, 3, 1, 1, 1, 1),       # many tiles
    # layer classes of the tensor-memory kernels (the others above that match one take it too)
    (3, 32, 32, 16, 32, 3, 3, 1, 1, 1, 1),      # 16 -> 32, stride 1, two pixels per GEMM row
    (5, 24, 24, 16, 32, 3, 3, 2, 2, 1, 1),      # 16 -> 32, stride 2
    (9, 12, 12, 32, 64, 3, 3, 2, 2, 1, 1),      # 32 -> 64, stride 2, one pixel per row
    (37, 10, 16, 8, 16, 3, 3, 2, 2, 1, 1),      # 8 -> 16, stride 2, four pixels per row, several images per tile
    (2, 16, 16, 64, 128, 3, 3, 1, 1, 1, 1),     # run-time-geometry kernel, 128 columns
    (2, 8, 8, 128, 256, 3, 3, 1, 1, 1, 1),      # ... channels split over two CTAs
    (3, 10, 14, 32, 96, 5, 5, 2, 1, 2, 2),      # ... 5x5, mixed strides
]


@pytest.mark.parametrize("g", CONV_PC)
@pytest.mark.parametrize("shifts", [(0, 12), (2, 12)])
def test_fused_conv_layer_with_per_channel_weights(q4, g, shifts):
    import torch
    N_, H, W, C, OC, KH, KW, sh, sw, ph, pw = g
    dq, do = q4.ConvDesc(*g), oracle.ConvDesc(*g)
    K = KH * KW * C
    seed = 500 + sum(g)
    X = wl.rand_flat_nibbles(seed, 1, N_ * H * W * C)
    Wt = wl.rand_packed(seed, 2, OC, K)
    zb, bias, mult, shift = channel_params(seed, OC, *shifts)
    za = 9
    lda = (K + 1) // 2
    Ao, _ = oracle.im2col(X, do, za, lda)
    want = oracle.requant_channels(oracle.gemm_channels(Ao, Wt, dq.M, OC, K, za, zb, bias), mult, shift, 2, 1, 14)
    Xd = torch.zeros((X.size + 31) // 16 * 16, dtype=torch.uint8, device="cuda")
    Xd[:X.size] = dev(X)
    Y = torch.full((dq.M, OC // 2), 0xA5, dtype=torch.uint8, device="cuda")
    n0 = q4.q4_launch_count()
    q4.q4_conv2d_channels(Xd, dev(Wt), dq, za, dev(zb), dev(mult), dev(shift), 2, 1, 14, Y, dev(bias))
    assert q4.q4_launch_count() - n0 == 1
    assert q4.q4_last_device_status() == q4.Q4_OK
    assert (Y.cpu().numpy() == want).all()


def test_fused_per_channel_layer_rejects_what_the_kernel_does_not_take(q4):
    import torch
    g = (1, 8, 8, 16, 72, 3, 3, 1, 1, 1, 1)              # 72 output channels
    dq = q4.ConvDesc(*g)
    v = torch.zeros(72, dtype=torch.int32, device="cuda")
    X = torch.zeros(1 * 8 * 8 * 8, dtype=torch.uint8, device="cuda")
    Wt = torch.zeros((72, 72), dtype=torch.uint8, device="cuda")
    Y = torch.zeros((dq.M, 36), dtype=torch.uint8, device="cuda")
    with pytest.raises(q4.Q4Error) as e:
        q4.q4_conv2d_channels(X, Wt, dq, 0, v, v, v, 0, 0, 15, Y)
    assert e.value.status == q4.Q4_ERR_UNSUPPORTED
