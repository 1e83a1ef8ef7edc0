"""GPU parity: q4_gemm_u8 (the 8-bit product of the paper's comparison) against the oracle,
bit for bit: full comparison at sizes the oracle finishes in seconds, sampled rows plus an
exact integer Freivalds check at the benchmark shape."""
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


def case(M, N, K, seed, ld_pad=0):
    ld = (K + 15) // 16 * 16 + ld_pad
    A = np.zeros((M, ld), np.uint8)
    Bt = np.zeros((N, ld), np.uint8)
    A[:, :K] = wl.rand_bytes(seed, 1, M * K).reshape(M, K)
    Bt[:, :K] = wl.rand_bytes(seed, 2, N * K).reshape(N, K)
    A[:, K:] = 0xEE                                     # pitch padding must not be read as data
    Bt[:, K:] = 0x77
    z = wl.rand_ints(seed, 3, 0, 255, 2)
    return A, Bt, int(z[0]), int(z[1])


def run(q4, A, Bt, M, N, K, za, zb, sums=False, ldc_pad=0):
    import torch
    C = torch.full((M, N + ldc_pad), -77, dtype=torch.int32, device="cuda")
    Ad, Bd = dev(A), dev(Bt)
    ra = cb = ws = None
    if sums:
        ra = dev(A[:, :K].astype(np.int64).sum(axis=1).astype(np.int32))
        cb = dev(Bt[:, :K].astype(np.int64).sum(axis=1).astype(np.int32))
    else:
        ws = torch.empty(q4.q4_gemm_u8_workspace_bytes(M, N), dtype=torch.uint8, device="cuda")
    q4.q4_gemm_u8(Ad, Bd, C[:, :N] if ldc_pad else C, M, N, K, za, zb, ra, cb, ws)
    assert q4.q4_last_device_status() == q4.Q4_OK
    out = C.cpu().numpy()
    assert (out[:, N:] == -77).all()
    return out[:, :N]


SHAPES = [(1, 1, 1), (64, 64, 256), (130, 70, 100), (128, 256, 128), (300, 264, 1000), (257, 129, 33),
          (1000, 520, 777), (384, 1024, 4096), (5, 300, 33024),
          # at least 74 tiles of 256 x 256: the CTA-pair kernel, ragged in every dimension
          (2321, 2344, 200), (2560, 2304, 640), (4100, 1290, 96)]


@pytest.mark.parametrize("shape", SHAPES)
def test_u8_gemm_matches_oracle(q4, shape):
    M, N, K = shape
    A, Bt, za, zb = case(M, N, K, seed=sum(shape), ld_pad=16 if M % 2 else 0)
    got = run(q4, A, Bt, M, N, K, za, zb, ldc_pad=4 if N % 8 else 0)
    assert (got == oracle.gemm_u8(A[:, :K], Bt[:, :K], za, zb)).all()


def test_u8_supplied_sums_and_extreme_zero_points(q4):
    M, N, K = 200, 136, 520
    A, Bt, _, _ = case(M, N, K, seed=9)
    for za, zb in ((0, 0), (255, 255), (0, 255), (255, 0)):
        want = oracle.gemm_u8(A[:, :K], Bt[:, :K], za, zb)
        assert (run(q4, A, Bt, M, N, K, za, zb, sums=True) == want).all()
        assert (run(q4, A, Bt, M, N, K, za, zb, sums=False) == want).all()


def test_u8_all_255_reaches_the_accumulator_bound(q4):
    M, N, K = 128, 64, 33024
    A = np.full((M, K), 255, np.uint8)
    Bt = np.full((N, K), 255, np.uint8)
    assert (run(q4, A, Bt, M, N, K, 0, 0) == 255 * 255 * K).all()


def test_u8_argument_checks(q4):
    import torch
    A = torch.zeros((16, 64), dtype=torch.uint8, device="cuda")
    C = torch.zeros((16, 16), dtype=torch.int32, device="cuda")
    with pytest.raises(q4.Q4Error) as e:
        q4.q4_gemm_u8(A, A, C, 16, 16, 64, 0, 256)
    assert e.value.status == q4.Q4_ERR_RANGE
    with pytest.raises(q4.Q4Error) as e:
        q4.q4_gemm_u8(A, A, C, 16, 16, 64, 0, 0)        # sums wanted, no workspace
    assert e.value.status == q4.Q4_ERR_WORKSPACE
    with pytest.raises(q4.Q4Error) as e:
        q4.q4_gemm_u8(A[:, 1:], A, C, 16, 16, 48, 0, 0)
    assert e.value.status == q4.Q4_ERR_ALIGNMENT


def test_u8_benchmark_shape_sampled_rows_and_freivalds(q4):
    """8192^3: rows sampled across every row tile against the oracle, plus exact integer
    Freivalds on the whole matrix (C r == A' (B' r) and l C == (l A') B' in int64)."""
    n = 8192
    A, Bt, za, zb = case(n, n, n, seed=8192)
    got = run(q4, A, Bt, n, n, n, za, zb)
    rows = np.unique(np.concatenate([np.arange(0, n, 128) + (np.arange(n // 128) * 37) % 128, [0, n - 1]]))
    assert (got[rows] == oracle.gemm_u8(A[rows], Bt, za, zb)).all()
    rng = np.random.default_rng(1)
    a, b = A.astype(np.int64) - za, Bt.astype(np.int64) - zb
    r = rng.integers(1, 1 << 10, size=n).astype(np.int64)
    assert (got.astype(np.int64) @ r == a @ (b.T @ r)).all()
    l = rng.integers(1, 1 << 10, size=n).astype(np.int64)
    assert (l @ got.astype(np.int64) == (l @ a) @ b.T).all()
