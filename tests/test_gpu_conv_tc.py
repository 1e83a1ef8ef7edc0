"""GPU parity of the tensor-memory (tcgen05) fused convolution kernel against the CPU
oracle, byte for byte: every layer class it has an instance for, with tiles that end in the
middle of a row / an image / the batch, several images per tile, one image over many tiles,
vertical paddings and strides it takes at run time, given and derived weight sums, the
32-bit and the 64-bit rounding path, and saturating clamps."""
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


def check_prepared_weights(q4, Xd, Wt, dq, za, zb, rq, bias, colsum, want):
    """The same layer from a weight image prepared ahead of time: one launch, the same bytes,
    nothing written past the image."""
    import torch
    nb = q4.q4_conv2d_weights_bytes(dq)
    assert nb > 0 and nb % 16 == 0
    img = torch.full((nb + 64,), 0xA5, dtype=torch.uint8, device="cuda")
    n0 = q4.q4_launch_count()
    q4.q4_conv2d_prepare_weights(dev(Wt), dq, za, zb, img[:nb], None if bias is None else dev(bias), colsum)
    assert q4.q4_launch_count() - n0 == 1
    Y = torch.full((dq.M + 64, dq.OC // 2), 0x3C, dtype=torch.uint8, device="cuda")
    n0 = q4.q4_launch_count()
    q4.q4_conv2d_prepared(Xd, img[:nb], dq, za, q4.Requant(*rq), Y[:dq.M])
    assert q4.q4_launch_count() - n0 == 1
    assert q4.q4_last_device_status() == q4.Q4_OK
    out = Y.cpu().numpy()
    assert (out[:dq.M] == want).all()
    assert (out[dq.M:] == 0x3C).all()
    assert (img[nb:].cpu().numpy() == 0xA5).all()


def test_weight_image_serves_other_batches_and_sizes_but_not_other_layers(q4):
    """An image depends on the layer class, the filter, the channel counts and za, not on the
    batch or the image size; given to another layer it is refused: nothing is written and
    the device status says so."""
    import torch
    rq = ((1 << 30) + 77, 5, 3, 1, 14)
    za, zb = 6, 9
    base = (3, 32, 32, 16, 32, 3, 3, 1, 1, 1, 1)
    seed = 9700
    Wt = wl.rand_packed(seed, 2, 32, 144)
    bias = wl.rand_ints(seed, 3, -300, 300, 32).astype(np.int32)
    d0 = q4.ConvDesc(*base)
    nb = q4.q4_conv2d_weights_bytes(d0)
    img = torch.empty(nb, dtype=torch.uint8, device="cuda")
    q4.q4_conv2d_prepare_weights(dev(Wt), d0, za, zb, img, dev(bias))
    for g in ((7, 20, 24, 16, 32, 3, 3, 1, 1, 1, 1), (1, 64, 40, 16, 32, 3, 3, 1, 1, 0, 1)):   # other batch / size / padding
        dq, do = q4.ConvDesc(*g), oracle.ConvDesc(*g)
        assert q4.q4_conv2d_weights_bytes(dq) == nb
        X = wl.rand_flat_nibbles(seed + g[0], 1, g[0] * g[1] * g[2] * g[3])
        want = oracle.conv2d(X, Wt, bias, do, za, zb, oracle.Requant(*rq))
        Y = torch.full((dq.M, 16), 0x3C, dtype=torch.uint8, device="cuda")
        q4.q4_conv2d_prepared(dev(X), img, dq, za, q4.Requant(*rq), Y)
        assert q4.q4_last_device_status() == q4.Q4_OK
        assert (Y.cpu().numpy() == want).all()
    # the stride-2 layer class of the same channel counts has an image of the same size, but another tag
    other = q4.ConvDesc(3, 32, 32, 16, 32, 3, 3, 2, 2, 1, 1)
    assert q4.q4_conv2d_weights_bytes(other) == nb
    X = dev(wl.rand_flat_nibbles(seed, 9, 3 * 32 * 32 * 16))
    Y = torch.full((other.M, 16), 0x3C, dtype=torch.uint8, device="cuda")
    q4.q4_conv2d_prepared(X, img, other, za, q4.Requant(*rq), Y)
    assert q4.q4_last_device_status() == q4.Q4_ERR_WEIGHT_IMAGE
    assert (Y.cpu().numpy() == 0x3C).all()                  # nothing written
    Y0 = torch.full((d0.M, 16), 0x3C, dtype=torch.uint8, device="cuda")
    q4.q4_conv2d_prepared(X, img, d0, za + 1, q4.Requant(*rq), Y0)                # another za
    assert (Y0.cpu().numpy() == 0x3C).all()
    assert q4.q4_last_device_status() == q4.Q4_ERR_WEIGHT_IMAGE
    assert q4.q4_last_device_status() == q4.Q4_OK            # reported once


TC_LAYERS = [  # N, H, W, C, OC, stride, pad_h, shift
    (2, 8, 8, 1, 8, 1, 1, 5),          # gray first layer, less than one tile
    (5, 48, 48, 1, 8, 1, 1, 5),        # ... tiles that end inside an image
    (70, 12, 16, 1, 8, 1, 1, 1),       # ... many images per tile, 64-bit rounding path
    (3, 20, 32, 1, 8, 1, 0, 6),        # ... no vertical padding
    (3, 48, 48, 8, 16, 2, 1, 5),       # 8 -> 16, stride 2 (c4 L2 geometry)
    (37, 10, 16, 8, 16, 2, 1, 0),      # ... several images per tile, shift 0
    (2, 9, 40, 8, 16, 2, 0, 5),        # ... odd height, no vertical padding
    (5, 24, 24, 16, 32, 2, 1, 5),      # 16 -> 32, stride 2 (c4 L3)
    (40, 6, 8, 16, 32, 2, 1, 4),       # ... tiny images
    (9, 12, 12, 32, 64, 2, 1, 6),      # 32 -> 64, stride 2 (c4 L4)
    (2, 30, 20, 32, 64, 2, 1, 1),
    (3, 32, 32, 16, 32, 1, 1, 5),      # 16 -> 32, stride 1 (c3)
    (1, 7, 12, 16, 32, 1, 1, 5),       # ... less than one tile
    (21, 5, 8, 16, 32, 1, 0, 3),       # ... several images per tile, no vertical padding
    (1, 200, 64, 16, 32, 1, 1, 5),     # ... one image over many tiles
]


@pytest.mark.parametrize("g", TC_LAYERS)
@pytest.mark.parametrize("given_sums", [False, True])
def test_tensor_memory_conv_kernel_matches_oracle(q4, g, given_sums):
    import torch
    N, H, W, C, OC, s, ph, shift = g
    seed = 9000 + sum(g)
    args = (N, H, W, C, OC, 3, 3, s, s, ph, 1)
    dq, do = q4.ConvDesc(*args), oracle.ConvDesc(*args)
    K = 9 * C
    X = wl.rand_flat_nibbles(seed, 1, N * H * W * C)
    Wt = wl.rand_packed(seed, 2, OC, K)
    bias = wl.rand_ints(seed, 3, -300, 300, OC).astype(np.int32) if given_sums else None
    za, zb = (int(v) for v in wl.rand_ints(seed, 4, 0, 15, 2))
    rq = ((1 << 30) + 987654321 % (1 << 30), shift, 3, 1, 14)
    want = oracle.conv2d(X, Wt, bias, do, za, zb, oracle.Requant(*rq))
    Xd = torch.zeros((X.size + 31) // 16 * 16, dtype=torch.uint8, device="cuda")
    Xd[:X.size] = dev(X)
    ws = torch.empty(q4.q4_conv2d_workspace_bytes(dq), dtype=torch.uint8, device="cuda")
    Y = torch.full((dq.M + 64, OC // 2), 0xA5, dtype=torch.uint8, device="cuda")
    colsum = None
    if given_sums:
        colsum = dev(oracle.unpack_rows(Wt, K).astype(np.int64).sum(axis=1).astype(np.int32))
    n0 = q4.q4_launch_count()
    q4.q4_conv2d(Xd[:X.size], dev(Wt), dq, za, zb, q4.Requant(*rq), Y[:dq.M], ws,
                 None if bias is None else dev(bias), colsum)
    assert q4.q4_launch_count() - n0 == 1            # one fused kernel, no unrolled matrix
    assert q4.q4_last_device_status() == q4.Q4_OK
    out = Y.cpu().numpy()
    assert (out[:dq.M] == want).all()
    assert (out[dq.M:] == 0xA5).all()                # nothing written past the last pixel
    # the warp-level fused kernels (variant 4) give the same bytes
    q4.q4_set_variant(4)
    try:
        Y2 = torch.full((dq.M, OC // 2), 0x5A, dtype=torch.uint8, device="cuda")
        q4.q4_conv2d(Xd[:X.size], dev(Wt), dq, za, zb, q4.Requant(*rq), Y2, ws,
                     None if bias is None else dev(bias), colsum)
        assert (Y2.cpu().numpy() == want).all()
    finally:
        q4.q4_set_variant(0)
    check_prepared_weights(q4, Xd[:X.size], Wt, dq, za, zb, rq, bias, colsum, want)


WIDE_LAYERS = [  # N, H, W, C, OC, KH, KW, sh, sw, ph, pw, shift
    (2, 12, 12, 32, 32, 3, 3, 1, 1, 1, 1, 6),       # 32 -> 32
    (3, 9, 11, 32, 64, 3, 3, 1, 1, 1, 1, 6),        # odd sizes
    (2, 16, 16, 64, 64, 3, 3, 1, 1, 1, 1, 7),       # 64 -> 64
    (2, 16, 16, 64, 128, 3, 3, 1, 1, 1, 1, 7),      # 64 -> 128: 128 columns
    (2, 8, 8, 128, 256, 3, 3, 1, 1, 1, 1, 8),       # 128 -> 256: channels split over two CTAs
    (3, 10, 14, 32, 96, 5, 5, 2, 1, 2, 2, 1),       # 5x5, mixed strides, padding 2, 64-bit rounding
    (5, 7, 9, 64, 32, 1, 1, 1, 1, 0, 0, 5),         # 1x1
    (2, 13, 10, 32, 64, 3, 2, 3, 2, 0, 1, 5),       # rectangular filter, stride 3 / 2
    (40, 4, 4, 32, 64, 3, 3, 1, 1, 1, 1, 6),        # many images per tile
    (1, 40, 36, 32, 160, 3, 3, 1, 1, 1, 1, 6),      # 160 channels: not two halves of whole 32-column chunks, explicit path
    (1, 24, 20, 96, 192, 3, 3, 2, 2, 1, 1, 7),      # 192 channels: two CTAs of 96 where shared memory has the room
]


@pytest.mark.parametrize("g", WIDE_LAYERS)
@pytest.mark.parametrize("given_sums", [False, True])
def test_run_time_geometry_kernel_for_wide_layers(q4, g, given_sums):
    """Layers with C a multiple of 32 through q4_conv2d: the tensor-memory kernel with
    run-time geometry where it applies (one launch), the explicit path elsewhere; both
    against the oracle."""
    import torch
    N, H, W, C, OC, KH, KW, sh, sw, ph, pw, shift = g
    seed = 9500 + sum(g)
    args = (N, H, W, C, OC, KH, KW, sh, sw, ph, pw)
    dq, do = q4.ConvDesc(*args), oracle.ConvDesc(*args)
    K = KH * KW * C
    X = wl.rand_flat_nibbles(seed, 1, N * H * W * C)
    Wt = wl.rand_packed(seed, 2, OC, K)
    bias = wl.rand_ints(seed, 3, -300, 300, OC).astype(np.int32) if given_sums else None
    za, zb = (int(v) for v in wl.rand_ints(seed, 4, 0, 15, 2))
    rq = ((1 << 30) + 987654321 % (1 << 30), shift, 3, 1, 14)
    want = oracle.conv2d(X, Wt, bias, do, za, zb, oracle.Requant(*rq))
    ws = torch.empty(q4.q4_conv2d_workspace_bytes(dq), dtype=torch.uint8, device="cuda")
    Y = torch.full((dq.M + 8, OC // 2), 0xA5, dtype=torch.uint8, device="cuda")
    colsum = None
    if given_sums:
        colsum = dev(oracle.unpack_rows(Wt, K).astype(np.int64).sum(axis=1).astype(np.int32))
    n0 = q4.q4_launch_count()
    q4.q4_conv2d(dev(X), dev(Wt), dq, za, zb, q4.Requant(*rq), Y[:dq.M], ws,
                 None if bias is None else dev(bias), colsum)
    launches = q4.q4_launch_count() - n0
    assert q4.q4_last_device_status() == q4.Q4_OK
    out = Y.cpu().numpy()
    assert (out[:dq.M] == want).all()
    assert (out[dq.M:] == 0xA5).all()
    if (C, OC) in ((32, 32), (32, 64), (64, 64), (64, 128), (128, 256), (64, 32), (32, 96)):
        assert launches == 1             # the tensor-memory kernel took it: no unrolled matrix
    if launches == 1:
        check_prepared_weights(q4, dev(X), Wt, dq, za, zb, rq, bias, colsum, want)
    else:
        assert q4.q4_conv2d_weights_bytes(dq) == 0       # no tensor-memory kernel, no image


@pytest.mark.parametrize("g", [(3, 48, 48, 8, 16, 3, 3, 2, 2, 1, 1), (2, 8, 8, 1, 8, 3, 3, 1, 1, 1, 1),
                               (3, 32, 32, 16, 32, 3, 3, 1, 1, 1, 1), (2, 16, 16, 64, 128, 3, 3, 1, 1, 1, 1)])
@pytest.mark.parametrize("big", [200_000, 3_000_000, -40_000_000])
def test_large_per_channel_constants(q4, g, big):
    """The kernels carry Eq. 3's per-channel constant into the product as signed-byte digits
    of an extra depth step; a bias that pushes it beyond the digits' range (about 226 000 with
    one spare word, a million with a whole step) switches to preloaded accumulators.  Both
    routes against the oracle.  Every channel's bias (a quarter of |big| up to |big|) is placed
    so that its accumulators straddle a rounding boundary of the re-quantizer: an error in the
    constant far smaller than one code step then flips output values."""
    import torch
    args = g
    N, H, W, C, OC = g[:5]
    dq, do = q4.ConvDesc(*args), oracle.ConvDesc(*args)
    K = 9 * C
    seed = 9900 + sum(g)
    X = wl.rand_flat_nibbles(seed, 1, N * H * W * C)
    Wt = wl.rand_packed(seed, 2, OC, K)
    za, zb = 6, 9
    shift = max(2, int(np.ceil(np.log2(abs(big) / 6.0))))
    mult = (1 << 30) + 12345
    real = mult / 2.0 ** (31 + shift)
    acc0 = oracle.conv2d_direct(X, Wt, do, za, zb).reshape(-1, OC).astype(np.int64)
    j = 1 + np.arange(OC) % 6
    sign = 1 if big > 0 else -1
    bias = (sign * np.round((j + 0.5) / real) - np.median(acc0, axis=0)).astype(np.int64)
    assert np.abs(bias).max() < 2 ** 30 and np.abs(bias).min() > abs(big) / 8
    bias = bias.astype(np.int32)
    rq = (mult, shift, 7, 0, 15)
    want = oracle.conv2d(X, Wt, bias, do, za, zb, oracle.Requant(*rq))
    codes = oracle.unpack_rows(want, OC)
    # most channels produce both codes next to their boundary
    assert sum(len(np.unique(codes[:, n])) >= 2 for n in range(OC)) >= OC // 2
    ws = torch.empty(q4.q4_conv2d_workspace_bytes(dq), dtype=torch.uint8, device="cuda")
    Y = torch.full((dq.M, OC // 2), 0xA5, dtype=torch.uint8, device="cuda")
    n0 = q4.q4_launch_count()
    q4.q4_conv2d(dev(X), dev(Wt), dq, za, zb, q4.Requant(*rq), Y, ws, dev(bias))
    assert q4.q4_launch_count() - n0 == 1
    assert q4.q4_last_device_status() == q4.Q4_OK
    assert (Y.cpu().numpy() == want).all()
    check_prepared_weights(q4, dev(X), Wt, dq, za, zb, rq, bias, None, want)     # both routes from an image too


def test_which_layers_take_the_tensor_memory_kernel(q4, capfd):
    """The kernel's instances are chosen by layer class; everything else keeps its path."""
    import os
    import subprocess
    import sys
    code = (
        "import torch\n"
        "from paper_2009_06488_b200 import binding as q4\n"
        "def run(*a):\n"
        "    d = q4.ConvDesc(*a)\n"
        "    X = torch.zeros(d.N*d.H*d.W*d.C//2 + 16, dtype=torch.uint8, device='cuda')\n"
        "    Wt = torch.zeros((d.OC, (d.K + 1)//2), dtype=torch.uint8, device='cuda')\n"
        "    Y = torch.zeros((d.M, d.OC//2), dtype=torch.uint8, device='cuda')\n"
        "    ws = torch.empty(q4.q4_conv2d_workspace_bytes(d), dtype=torch.uint8, device='cuda')\n"
        "    q4.q4_conv2d(X, Wt, d, 1, 2, q4.Requant(1 << 30, 4, 0, 0, 15), Y, ws)\n"
        "run(2, 32, 32, 16, 32, 3, 3, 1, 1, 1, 1)\n"     # c3 class
        "run(2, 32, 31, 16, 32, 3, 3, 1, 1, 1, 1)\n"     # output rows not whole groups of pixels
        "run(2, 32, 32, 16, 24, 3, 3, 1, 1, 1, 1)\n"     # another channel count
        "torch.cuda.synchronize()\n")
    env = dict(os.environ, Q4_LOG="1")
    root = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
    r = subprocess.run([sys.executable, "-c", code], capture_output=True, text=True, env=env, cwd=root)
    assert r.returncode == 0, r.stderr
    lines = [l for l in r.stderr.splitlines() if l.startswith("[q4] q4_conv2d")]
    assert len(lines) == 3
    assert "tcgen05" in lines[0]
    assert "tcgen05" not in lines[1] and "tcgen05" not in lines[2]


def _random_layers(count, seed):
    """Seeded layer geometries: half of them from the tensor-memory kernels' layer classes with
    enough rows for several tiles per CTA, half anything the entry points accept."""
    rng = np.random.default_rng(seed)
    out = []
    while len(out) < count:
        if len(out) % 2 == 0:
            C = int(rng.choice([1, 8, 16, 32, 64])); OC = int(rng.choice([8, 16, 32, 64, 128]))
            KH = KW = 3; s = int(rng.choice([1, 2])); p = 1
            H = int(rng.choice([8, 12, 16, 24, 32])); W = H if rng.random() < 0.7 else int(rng.integers(6, 40))
            Nb = int(rng.integers(1, 60)) if C * OC <= 512 else int(rng.integers(1, 8))
        else:
            C = int(rng.choice([1, 2, 3, 4, 8, 16, 24])); OC = int(rng.choice([2, 6, 8, 16, 24, 32, 72]))
            KH = int(rng.choice([1, 2, 3, 5])); KW = KH if rng.random() < 0.7 else int(rng.choice([1, 2, 3]))
            s = int(rng.choice([1, 1, 2])); p = int(rng.integers(0, (min(KH, KW) + 1) // 2 + 1))
            H = int(rng.integers(max(KH, 4), 30)); W = int(rng.integers(max(KW, 4), 30))
            Nb = int(rng.integers(1, 12))
        if (Nb * H * W * C) % 2:
            Nb += 1
        if (Nb * H * W * C) % 2 == 0:
            out.append((Nb, H, W, C, OC, KH, KW, s, s, p, p))
    return out


@pytest.mark.parametrize("g", _random_layers(28, 20260102))
def test_random_layers_through_every_convolution_entry_point(q4, g):
    """q4_conv2d (automatic choice and the explicit unroll + GEMM route), q4_conv2d_channels and,
    where the layer has one, the prepared weight image: the oracle's bytes from each."""
    import torch
    Nb, H, W, C, OC, KH, KW, s, _, p, _ = g
    dq, do = q4.ConvDesc(*g), oracle.ConvDesc(*g)
    K = KH * KW * C
    seed = 7000 + sum(g)
    X = wl.rand_flat_nibbles(seed, 1, Nb * H * W * C)
    Wt = wl.rand_packed(seed, 2, OC, K)
    bias = wl.rand_ints(seed, 3, -400, 400, OC).astype(np.int32)
    za, zb = 5, 11
    rq = ((1 << 30) + 12345 * (seed % 97), 4 + seed % 5, 3, 1, 14)
    want = oracle.conv2d(X, Wt, bias, do, za, zb, oracle.Requant(*rq))
    Xd = torch.zeros((X.size + 31) // 16 * 16, dtype=torch.uint8, device="cuda")
    Xd[:X.size] = dev(X)
    ws = torch.full((max(q4.q4_conv2d_workspace_bytes(dq), 16),), 0xA5, dtype=torch.uint8, device="cuda")
    try:
        for variant in (0, 4):
            q4.q4_set_variant(variant)
            Y = torch.full((dq.M, OC // 2), 0xA5, dtype=torch.uint8, device="cuda")
            q4.q4_conv2d(Xd, dev(Wt), dq, za, zb, q4.Requant(*rq), Y, ws, dev(bias))
            assert q4.q4_last_device_status() == q4.Q4_OK
            assert (Y.cpu().numpy() == want).all(), variant
    finally:
        q4.q4_set_variant(0)
    if q4.q4_conv2d_weights_bytes(dq):
        check_prepared_weights(q4, Xd, Wt, dq, za, zb, rq, bias, None, want)
    # per-channel weights: zero points, multipliers and shifts of their own
    zbc = wl.rand_ints(seed, 4, 0, 15, OC).astype(np.int32)
    mult = wl.rand_ints(seed, 5, 1 << 30, (1 << 31) - 1, OC).astype(np.int32)
    shift = wl.rand_ints(seed, 6, 0 if seed % 3 == 0 else 2, 12, OC).astype(np.int32)
    Ao, _ = oracle.im2col(X, do, za, (K + 1) // 2)
    wantc = oracle.requant_channels(oracle.gemm_channels(Ao, Wt, dq.M, OC, K, za, zbc, bias), mult, shift, 2, 1, 14)
    Y = torch.full((dq.M, OC // 2), 0xA5, dtype=torch.uint8, device="cuda")
    try:
        q4.q4_conv2d_channels(Xd, dev(Wt), dq, za, dev(zbc), dev(mult), dev(shift), 2, 1, 14, Y, dev(bias))
    except q4.Q4Error as e:
        assert e.status == q4.Q4_ERR_UNSUPPORTED      # layers the fused kernels do not take
        return
    assert q4.q4_last_device_status() == q4.Q4_OK
    assert (Y.cpu().numpy() == wantc).all()
