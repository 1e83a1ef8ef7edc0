"""CPU oracle for per-output-channel weight quantization -- TEST INFRASTRUCTURE ONLY.

The paper quantizes each weight matrix with one scale and one zero point (Eq. 1 over the whole
matrix, Section II-A/III-B).  Giving every output channel n (a row of the weight matrix the
paper writes on the left, a column of B here) its own zero point zb[n] and its own
re-quantization multiplier leaves Eq. 2 unchanged column by column:
    acc[m][n] = sum_k (a[m][k] - za) * (b[k][n] - zb[n]) + bias[n]
    q[m][n]   = floor((acc * mult[n] + 2^(30 + shift[n])) / 2^(31 + shift[n]))     (one rounding, ties up)
    y[m][n]   = clamp(q + zo, lo, hi), packed two per byte along n.
Plain numpy int64 on unpacked values; Python integers for the rounding shift.
"""
from __future__ import annotations

import numpy as np


def _unpack(P: np.ndarray, K: int) -> np.ndarray:
    P = np.asarray(P, dtype=np.uint8)
    V = np.empty((P.shape[0], 2 * P.shape[1]), dtype=np.int64)
    V[:, 0::2] = P & 0x0F
    V[:, 1::2] = P >> 4
    return V[:, :K]


def gemm_channels(A, Bt, M: int, N: int, K: int, za: int, zb, bias=None) -> np.ndarray:
    """int32 accumulators with a zero point per output channel (zb: N values in 0..15)."""
    a = _unpack(np.asarray(A)[:M], K)
    b = _unpack(np.asarray(Bt)[:N], K)
    zb = np.asarray(zb, dtype=np.int64).reshape(N)
    assert 0 <= za <= 15 and zb.min(initial=0) >= 0 and zb.max(initial=0) <= 15
    acc = (a - za) @ (b - zb[:, None]).T
    if bias is not None:
        acc = acc + np.asarray(bias, dtype=np.int64).reshape(1, N)
    assert np.abs(acc).max(initial=0) < 2 ** 31
    return acc.astype(np.int32)


def requant_channels(acc, mult, shift, zo: int, lo: int, hi: int) -> np.ndarray:
    """Packed uint4 [M, N/2] from int32 accumulators [M, N] with a multiplier in [2^30, 2^31) and
    a shift in 0..31 per channel."""
    acc = np.asarray(acc, dtype=np.int64)
    M, N = acc.shape
    assert N % 2 == 0
    y = np.empty((M, N), dtype=np.uint8)
    for n in range(N):
        m_n, t = int(mult[n]), 31 + int(shift[n])
        assert (1 << 30) <= m_n < (1 << 31) and 31 <= t <= 62
        q = (acc[:, n] * m_n + (1 << (t - 1))) >> t        # int64: |acc * mult| < 2^62; >> floors
        y[:, n] = np.clip(q + zo, lo, hi)
    return (y[:, 0::2] | (y[:, 1::2] << 4)).astype(np.uint8)
