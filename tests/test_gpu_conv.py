"""GPU parity: q4_im2col / q4_conv2d and the layer chains against the CPU oracle,
byte for byte (pad nibbles included)."""
import numpy as np
import pytest

import oracle
from paper_2009_06488_b200 import workloads as wl

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def q4():
    from paper_2009_06488_b200 import binding
    binding.q4_set_variant(0)
    return binding


def dev(a):
    import torch
    return torch.from_numpy(np.ascontiguousarray(a)).cuda()


def descs(L):
    from paper_2009_06488_b200 import binding
    args = (L.N, L.H, L.W, L.C, L.OC, L.KH, L.KW, L.stride, L.stride, L.pad, L.pad)
    return binding.ConvDesc(*args), oracle.ConvDesc(*args)


IM2COL = [  # N, H, W, C, KH, KW, stride_h, stride_w, pad_h, pad_w
    (2, 6, 7, 3, 3, 3, 1, 1, 1, 1),        # odd channels: nibble-granular, byte kernel
    (1, 9, 8, 1, 3, 3, 2, 2, 1, 1),
    (2, 33, 25, 1, 5, 5, 1, 1, 0, 0),
    (3, 10, 11, 8, 3, 3, 2, 1, 0, 1),      # 4-byte taps
    (2, 12, 12, 16, 3, 3, 1, 1, 1, 1),     # 8-byte taps
    (2, 9, 9, 16, 3, 3, 2, 2, 1, 1),
    (2, 7, 6, 32, 3, 3, 2, 2, 1, 1),       # 16-byte taps
    (1, 5, 5, 64, 3, 3, 1, 1, 1, 1),       # 32-byte taps
    (3, 4, 4, 96, 1, 1, 1, 1, 0, 0),       # 48-byte taps, pointwise
    (1, 6, 6, 4, 3, 3, 1, 1, 2, 2),        # 2-byte taps -> byte kernel
    (2, 8, 8, 12, 5, 5, 1, 1, 2, 2),       # 6-byte taps -> byte kernel
    (5, 19, 17, 16, 3, 3, 1, 1, 1, 1),     # 1615 rows: many 32-row tiles and a ragged last one
    (7, 21, 13, 8, 3, 3, 2, 2, 1, 1),      # 4-byte taps, stride 2, 539 rows
    (3, 9, 11, 32, 3, 3, 1, 1, 1, 1),      # 16-byte taps, pitch 144
    (2, 9, 9, 128, 3, 3, 1, 1, 1, 1),      # pitch 576: tile kernel with three warps per block
    (1, 4, 4, 256, 3, 3, 1, 1, 1, 1),      # pitch 1152: beyond the tile kernel, chunk-per-thread kernel
]


@pytest.mark.parametrize("g", IM2COL)
@pytest.mark.parametrize("aligned_pitch", [True, False])
def test_im2col_matches_oracle(q4, g, aligned_pitch):
    import torch
    N, H, W, C, KH, KW, sh, sw, ph, pw = g
    dq = q4.ConvDesc(N, H, W, C, 2, KH, KW, sh, sw, ph, pw)
    do = oracle.ConvDesc(N, H, W, C, 2, KH, KW, sh, sw, ph, pw)
    X = wl.rand_flat_nibbles(sum(g), 1, N * H * W * C)
    K = KH * KW * C
    kb = (K + 1) // 2
    lda = (kb + 15) // 16 * 16 + (0 if aligned_pitch else 3)
    za = 11
    wantA, want_ra = oracle.im2col(X, do, za, lda)
    Xd = torch.zeros((X.size + 15) // 16 * 16, dtype=torch.uint8, device="cuda")
    Xd[:X.size] = dev(X)
    A = torch.full((dq.M, lda), 0xA5, dtype=torch.uint8, device="cuda")
    ra = torch.full((dq.M,), -7, dtype=torch.int32, device="cuda")
    q4.q4_im2col(Xd, dq, za, A, ra)
    assert (A.cpu().numpy() == wantA).all()
    assert (ra.cpu().numpy() == want_ra).all()
    A2 = torch.full((dq.M, lda), 0xA5, dtype=torch.uint8, device="cuda")
    q4.q4_im2col(Xd, dq, za, A2, None)                  # sums are optional
    assert (A2.cpu().numpy() == wantA).all()


def run_layer(q4, L, Xd):
    import torch
    dq, _ = descs(L)
    ws = torch.empty(q4.q4_conv2d_workspace_bytes(dq), dtype=torch.uint8, device="cuda")
    Y = torch.full((dq.M, L.OC // 2), 0xA5, dtype=torch.uint8, device="cuda")
    q4.q4_conv2d(Xd, dev(L.Wt), dq, L.za, L.zb,
                 q4.Requant(L.mult, L.shift, L.zo, L.clamp_lo, L.clamp_hi), Y, ws,
                 None if L.bias is None else dev(L.bias))
    assert q4.q4_last_device_status() == q4.Q4_OK
    return Y


def oracle_layer(L, X):
    _, do = descs(L)
    return oracle.conv2d(X, L.Wt, L.bias, do, L.za, L.zb,
                         oracle.Requant(L.mult, L.shift, L.zo, L.clamp_lo, L.clamp_hi))


def run_chain(q4, net):
    """Every layer's packed output, GPU and oracle, each fed by its own previous layer."""
    Xd, Xo = dev(net.X), net.X
    for L in net.layers:
        Yd = run_layer(q4, L, Xd.reshape(-1))
        Yo = oracle_layer(L, Xo)
        got = Yd.cpu().numpy()
        assert got.shape == Yo.shape
        assert (got == Yo).all(), L.name
        Xd, Xo = Yd, Yo.reshape(-1)
    return Xo


@pytest.mark.parametrize("variant", [0, 1, 3])     # fused kernel / unroll + general GEMM / unroll + tensor-core GEMM
def test_conv2d_small_layers(q4, variant):
    q4.q4_set_variant(variant)
    try:
        for seed, (N, H, W, C, OC, k, s, p) in enumerate([
                (2, 12, 12, 16, 32, 3, 1, 1), (3, 9, 10, 8, 16, 3, 2, 1), (2, 8, 8, 1, 8, 3, 1, 1),
                (1, 33, 25, 1, 8, 5, 1, 0), (2, 6, 6, 64, 6, 1, 1, 0), (1, 7, 9, 3, 4, 3, 2, 2),
                (3, 11, 13, 32, 64, 3, 2, 1), (2, 9, 7, 8, 8, 5, 1, 2), (5, 17, 19, 24, 16, 3, 1, 1),
                (1, 40, 40, 16, 32, 3, 1, 1)]):
            X = wl.rand_flat_nibbles(100 + seed, 1, N * H * W * C)
            kb = (k * k * C + 1) // 2
            # the forced tensor-core variant needs a 16-byte weight pitch
            Wt = wl.rand_packed(100 + seed, 2, OC, k * k * C, (kb + 15) // 16 * 16 if variant == 3 else None)
            bias = wl.rand_ints(100 + seed, 3, -512, 512, OC).astype(np.int32)
            L = wl.ConvLayer("t", N, H, W, C, OC, k, k, s, p, 5 + seed, 9 - seed, Wt, bias,
                             (1 << 30) + 4242, 3, 2, 2, 15)
            got = run_layer(q4, L, dev(X)).cpu().numpy()
            want = oracle_layer(L, X)
            assert (got == want).all()
            if seed < 6:
                assert len(np.unique(oracle.unpack_rows(want, OC))) > 3
    finally:
        q4.q4_set_variant(0)


def test_c3_conv_layer_full_batch(q4):
    net = wl.c3()
    out = run_chain(q4, net)
    hist = np.bincount(oracle.unpack(out, out.size * 2), minlength=16)
    assert (hist > 0).sum() >= 8         # calibrated requantizer spreads the outputs


@pytest.mark.parametrize("kw", [dict(seed=4000), dict(seed=4001), dict(seed=4002),
                                dict(seed=4000, centred=True)])
def test_c4_chain_small_batch(q4, kw):
    run_chain(q4, wl.c4(batch=16, **kw))


def test_c4_chain_full_batch(q4):
    run_chain(q4, wl.c4(batch=4096, seed=4000, centred=True))


def test_paper_table2_topology_with_random_weights(q4):
    run_chain(q4, wl.paper_table2_net(batch=3))


FUSED = [  # N, H, W, C, OC, KH, KW, sh, sw, ph, pw, byte offset of X, shift
    (3, 16, 16, 1, 8, 3, 3, 1, 1, 1, 1, 0, 5),      # pixel per lane, packed copy (rows are whole words)
    (5, 9, 8, 2, 16, 3, 3, 2, 2, 1, 1, 0, 5),       # pixel per lane, packed copy, two channels
    (2, 8, 24, 1, 8, 5, 5, 1, 1, 2, 2, 0, 1),       # ... 5x5, 64-bit rounding path (shift < 2)
    (3, 33, 25, 1, 8, 5, 5, 1, 1, 0, 0, 0, 6),      # pixel per lane, expanded copy (odd row length)
    (2, 7, 7, 3, 8, 2, 2, 1, 1, 0, 0, 0, 4),        # ... three channels, odd nibble offsets per row
    (4, 16, 16, 1, 8, 3, 3, 1, 1, 1, 1, 1, 5),      # ... forced by a misaligned input pointer
    (2, 11, 9, 3, 24, 3, 3, 1, 1, 1, 1, 0, 5),      # MMA, expanded copy, 24 outputs
    (2, 10, 12, 5, 32, 3, 2, 2, 1, 1, 0, 0, 5),     # MMA, expanded copy, rectangular filter and strides
    (3, 12, 12, 8, 16, 3, 3, 1, 1, 1, 1, 2, 5),     # MMA, expanded copy forced by a misaligned pointer
    (2, 9, 10, 8, 40, 3, 3, 1, 1, 1, 1, 0, 5),      # MMA, packed copy in 4-byte pieces, 40 outputs
    (2, 9, 12, 8, 56, 3, 3, 3, 3, 0, 2, 0, 0),      # MMA, packed copy in 16-byte pieces, stride 3, shift 0
    (300, 3, 3, 8, 8, 3, 3, 1, 1, 1, 1, 0, 5),      # tiles spanning dozens of images, OW < 8
    (90, 5, 6, 16, 48, 2, 3, 2, 1, 1, 1, 0, 5),     # OW < 8, rows of several images per thread
    (700, 1, 1, 8, 8, 1, 1, 1, 1, 0, 0, 0, 5),      # one pixel per image
    (2, 20, 40, 32, 64, 3, 3, 1, 1, 1, 1, 0, 7),    # widest tile the MMA kernel has
    (1, 30, 300, 8, 8, 1, 7, 1, 2, 0, 3, 0, 5),     # long rows: a tile inside one output row
    (9, 48, 48, 1, 8, 3, 3, 1, 1, 1, 1, 0, 1),      # four pixels per lane: tiles over two images, shift < 2
    (4, 20, 32, 1, 8, 3, 3, 1, 1, 1, 1, 0, 5),      # ... rows copied by bulk copies (16-byte rows)
    (6, 10, 24, 1, 8, 3, 3, 1, 1, 0, 1, 0, 9),      # ... no vertical padding
    (3, 16, 40, 1, 8, 3, 3, 1, 1, 1, 3, 0, 5),      # ... horizontal padding of three
    (5, 12, 20, 1, 8, 3, 3, 1, 1, 0, 0, 0, 5),      # output rows not groups of four: pixel per lane
]


@pytest.mark.parametrize("g", FUSED)
@pytest.mark.parametrize("given_sums", [False, True])
def test_conv2d_fused_modes(q4, g, given_sums):
    """Every staging mode and both kernels of the fused layer against the oracle."""
    import torch
    N, H, W, C, OC, KH, KW, sh, sw, ph, pw, xoff, shift = g
    seed = 7000 + sum(g)
    args = (N, H, W, C, OC, KH, KW, sh, sw, ph, pw)
    dq, do = q4.ConvDesc(*args), oracle.ConvDesc(*args)
    K = KH * KW * C
    X = wl.rand_flat_nibbles(seed, 1, N * H * W * C)
    Wt = wl.rand_packed(seed, 2, OC, K)
    bias = wl.rand_ints(seed, 3, -300, 300, OC).astype(np.int32)
    za, zb = (int(v) for v in wl.rand_ints(seed, 4, 0, 15, 2))
    rq = ((1 << 30) + 987654321 % (1 << 30), shift, 3, 1, 14)
    want = oracle.conv2d(X, Wt, bias, do, za, zb, oracle.Requant(*rq))
    Xbuf = torch.zeros(xoff + (X.size + 31) // 16 * 16, dtype=torch.uint8, device="cuda")
    Xd = Xbuf[xoff:xoff + X.size]
    Xd.copy_(dev(X))
    ws = torch.empty(q4.q4_conv2d_workspace_bytes(dq), dtype=torch.uint8, device="cuda")
    Y = torch.full((dq.M, OC // 2), 0xA5, dtype=torch.uint8, device="cuda")
    colsum = None
    if given_sums:
        colsum = dev(oracle.unpack_rows(Wt, K).astype(np.int64).sum(axis=1).astype(np.int32))
    n0 = q4.q4_launch_count()
    q4.q4_conv2d(Xd, dev(Wt), dq, za, zb, q4.Requant(*rq), Y, ws, dev(bias), colsum)
    assert q4.q4_launch_count() - n0 == 1            # the fused path: one kernel, no unrolled matrix
    assert q4.q4_last_device_status() == q4.Q4_OK
    assert (Y.cpu().numpy() == want).all()
