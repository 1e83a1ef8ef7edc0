"""Pins of the 8-bit product oracle (oracle/q8.py): brute force, the independently pinned
4-bit C oracle on values below 16, Eq. 2's identity, range and degenerate cases."""
import numpy as np
import pytest

import oracle


def test_brute_force_on_tiny_inputs():
    rng = np.random.default_rng(0)
    for _ in range(20):
        M, N, K = rng.integers(1, 5, size=3)
        A = rng.integers(0, 256, size=(M, K)).astype(np.uint8)
        Bt = rng.integers(0, 256, size=(N, K)).astype(np.uint8)
        za, zb = int(rng.integers(0, 256)), int(rng.integers(0, 256))
        want = [[sum((int(A[m, k]) - za) * (int(Bt[n, k]) - zb) for k in range(K)) for n in range(N)]
                for m in range(M)]
        assert oracle.gemm_u8(A, Bt, za, zb).tolist() == want


def test_hand_computed_example():
    # (1-1)(3-2) + (2-1)(4-2) = 2 ; (1-1)(5-2) + (2-1)(6-2) = 4 ; (255-1)(3-2) + 0 = 254 ; 254*3 = 762
    A = np.array([[1, 2], [255, 1]], dtype=np.uint8)
    Bt = np.array([[3, 4], [5, 6]], dtype=np.uint8)
    assert oracle.gemm_u8(A, Bt, 1, 2).tolist() == [[2, 4], [254, 762]]


@pytest.mark.parametrize("seed", range(4))
def test_agrees_with_the_4bit_oracle_on_small_values(seed):
    rng = np.random.default_rng(seed)
    M, N, K = 9, 7, 2 * int(rng.integers(1, 40))
    A = rng.integers(0, 16, size=(M, K)).astype(np.uint8)
    Bt = rng.integers(0, 16, size=(N, K)).astype(np.uint8)
    za, zb = int(rng.integers(0, 16)), int(rng.integers(0, 16))
    pack = lambda X: (X[:, 0::2] | (X[:, 1::2] << 4)).astype(np.uint8)
    assert (oracle.gemm_u8(A, Bt, za, zb) == oracle.gemm(pack(A), pack(Bt), M, N, K, za, zb)).all()


@pytest.mark.parametrize("seed", range(4))
def test_eq2_identity(seed):
    rng = np.random.default_rng(100 + seed)
    A = rng.integers(0, 256, size=(13, 77)).astype(np.uint8)
    Bt = rng.integers(0, 256, size=(11, 77)).astype(np.uint8)
    za, zb = int(rng.integers(0, 256)), int(rng.integers(0, 256))
    assert (oracle.gemm_u8(A, Bt, za, zb) == oracle.gemm_u8_fourterm(A, Bt, za, zb)).all()


def test_range_and_degenerate_cases():
    K = 300
    full = np.full((3, K), 255, np.uint8)
    assert (oracle.gemm_u8(full, full, 0, 0) == 255 * 255 * K).all()
    assert (oracle.gemm_u8(full, full, 255, 0) == 0).all()           # A == za everywhere
    assert (oracle.gemm_u8(full, np.full((2, K), 9, np.uint8), 3, 9) == 0).all()
    # additivity over the depth
    rng = np.random.default_rng(5)
    A = rng.integers(0, 256, size=(4, 60)).astype(np.uint8)
    Bt = rng.integers(0, 256, size=(5, 60)).astype(np.uint8)
    whole = oracle.gemm_u8(A, Bt, 17, 200)
    parts = oracle.gemm_u8(A[:, :25], Bt[:, :25], 17, 200) + oracle.gemm_u8(A[:, 25:], Bt[:, 25:], 17, 200)
    assert (whole == parts).all()
    # transposition symmetry
    assert (oracle.gemm_u8(A, Bt, 17, 200).T == oracle.gemm_u8(Bt, A, 200, 17)).all()
