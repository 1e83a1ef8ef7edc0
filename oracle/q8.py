"""CPU oracle for the 8-bit quantized matrix product -- TEST INFRASTRUCTURE ONLY.

The paper's comparison system: the same quantized product (Section II-B, Eq. 2) with 8-bit
values in 0..255 and 32-bit accumulators instead of 4-bit values and 16-bit ones.  This is
the plain definition (the middle expression of Eq. 2 without the scale factors),
    C[m][n] = sum_k (A[m][k] - za) * (B[k][n] - zb),
on unpacked uint8 arrays, written as one int64 matrix product; B is given as Bt (N x K,
depth-contiguous, the layout weights are prepared in once).  `gemm_u8_fourterm` evaluates
the last line of Eq. 2 term by term instead.
"""
from __future__ import annotations

import numpy as np

MAX_DEPTH = 33024      # 255 * 255 * K stays below 2^31: the raw product fits the 32-bit accumulator


def _check(A, Bt, za, zb):
    A, Bt = np.asarray(A), np.asarray(Bt)
    assert A.dtype == np.uint8 and Bt.dtype == np.uint8 and A.ndim == 2 and Bt.ndim == 2
    assert A.shape[1] == Bt.shape[1] and 1 <= A.shape[1] <= MAX_DEPTH
    assert 0 <= za <= 255 and 0 <= zb <= 255
    return A.astype(np.int64), Bt.astype(np.int64)


def gemm_u8(A, Bt, za: int, zb: int) -> np.ndarray:
    a, b = _check(A, Bt, za, zb)
    C = (a - za) @ (b - zb).T
    assert np.abs(C).max(initial=0) <= 255 * 255 * a.shape[1]
    return C.astype(np.int32)


def gemm_u8_fourterm(A, Bt, za: int, zb: int) -> np.ndarray:
    """Last line of Eq. 2: raw product, minus zb * (sums over the depth of A's rows), minus
    za * (sums over the depth of B's columns), plus K * za * zb."""
    a, b = _check(A, Bt, za, zb)
    K = a.shape[1]
    raw = a @ b.T
    C = raw - zb * a.sum(axis=1)[:, None] - za * b.sum(axis=1)[None, :] + K * za * zb
    return C.astype(np.int32)
