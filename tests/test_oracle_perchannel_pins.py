"""Pins of the per-channel oracle (oracle/perchannel.py): with one zero point and one
multiplier for all channels it must equal the separately pinned C oracle; brute force and
arbitrary-precision rounding on tiny inputs; channels are independent."""
import numpy as np
import pytest

import oracle
from paper_2009_06488_b200 import workloads as wl


def case(M, N, K, seed):
    A = wl.rand_packed(seed, 1, M, K)
    Bt = wl.rand_packed(seed, 2, N, K)
    bias = wl.rand_ints(seed, 3, -512, 512, N).astype(np.int32)
    zb = wl.rand_ints(seed, 4, 0, 15, N)
    mult = wl.rand_ints(seed, 5, 1 << 30, (1 << 31) - 1, N)
    shift = wl.rand_ints(seed, 6, 0, 12, N)
    return A, Bt, bias, zb, mult, shift


@pytest.mark.parametrize("seed", range(4))
def test_uniform_channels_equal_the_per_tensor_oracle(seed):
    M, N, K = 11, 10, 37 + seed
    A, Bt, bias, _, _, _ = case(M, N, K, seed)
    za, zb, mult, shift = 5, 9, (1 << 30) + 12345 * (seed + 1), 3 + seed
    acc = oracle.gemm_channels(A, Bt, M, N, K, za, [zb] * N)
    assert (acc == oracle.gemm(A, Bt, M, N, K, za, zb)).all()
    got = oracle.requant_channels(oracle.gemm_channels(A, Bt, M, N, K, za, [zb] * N, bias),
                                  [mult] * N, [shift] * N, 2, 1, 14)
    want = oracle.gemm_requant(A, Bt, M, N, K, za, zb, bias, oracle.Requant(mult, shift, 2, 1, 14))
    assert (got == want).all()


def test_brute_force_with_python_integers():
    M, N, K = 3, 4, 9
    A, Bt, bias, zb, mult, shift = case(M, N, K, 77)
    a, b = oracle.unpack_rows(A, K).astype(int), oracle.unpack_rows(Bt, K).astype(int)
    acc = oracle.gemm_channels(A, Bt, M, N, K, 7, zb, bias)
    y = oracle.requant_channels(acc, mult, shift, 3, 0, 15)
    for m in range(M):
        for n in range(N):
            s = sum((int(a[m, k]) - 7) * (int(b[n, k]) - int(zb[n])) for k in range(K)) + int(bias[n])
            assert acc[m, n] == s
            t = 31 + int(shift[n])
            q = (s * int(mult[n]) + (1 << (t - 1))) >> t          # arbitrary precision
            want = min(max(q + 3, 0), 15)
            got = (y[m, n // 2] >> (4 * (n % 2))) & 0x0F
            assert got == want


def test_channels_are_independent():
    M, N, K = 6, 8, 50
    A, Bt, bias, zb, mult, shift = case(M, N, K, 5)
    full = oracle.gemm_channels(A, Bt, M, N, K, 4, zb, bias)
    for n in range(N):
        one = oracle.gemm(A, Bt[n:n + 1], M, 1, K, 4, int(zb[n]))[:, 0] + bias[n]
        assert (full[:, n] == one).all()
    # changing one channel's zero point changes only that column
    zb2 = zb.copy(); zb2[3] = (zb2[3] + 5) % 16
    other = oracle.gemm_channels(A, Bt, M, N, K, 4, zb2, bias)
    assert (np.delete(other, 3, axis=1) == np.delete(full, 3, axis=1)).all()


def test_ties_round_up_per_channel():
    acc = np.array([[4, -4, 6, -6]], dtype=np.int32)       # mult 2^30: q = floor(acc / 2^(shift+1) + 1/2)
    y = oracle.requant_channels(acc, [1 << 30] * 4, [2, 2, 1, 1], 8, 0, 15)
    # 4/8 = .5 -> 1 ; -4/8 = -.5 -> 0 ; 6/4 = 1.5 -> 2 ; -6/4 = -1.5 -> -1 ; plus zo = 8
    assert [(y[0, 0] & 15), (y[0, 0] >> 4), (y[0, 1] & 15), (y[0, 1] >> 4)] == [9, 8, 10, 7]
