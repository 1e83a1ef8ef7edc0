"""CPU oracle for the float boundary of a quantized layer -- TEST INFRASTRUCTURE ONLY.

The linear quantization of Eq. 1 (Section II-A) that turns a floating-point tensor into
4-bit codes at the input of a quantized layer (the F -> Q case of Section III-B), and the
conversion of an integer result back to floating point by its scale factor (Eq. 4; the
Q -> F case).  numpy, one array operation per step of the equations, no blocking.

Precision: the paper's floating-point values are 32-bit, and a quantized code is an integer
decided by floating-point arithmetic, so every operation below is an IEEE binary32 operation
(numpy float32 scalars and arrays: correctly rounded subtraction, division and
multiplication).

Reading of Eq. 1.  As printed, the zero point z = min(min w, 0) is in real units while the
code is floor(w / s) - z and Eq. 2 de-quantizes as s * (code - z); the two only agree when z
is counted in steps of s.  Taken here:
    s   = (max(max w, 0) - min(min w, 0)) / (2^p - 1),  p = 4   (s := 1 for an all-zero tensor)
    z_q = -floor(min(min w, 0) / s)                         (an integer in 0..15)
    code = clamp(floor(w / s) + z_q, 0, 15)
    w  ~= s * (code - z_q)
so that non-negative data gets z_q = 0 (Section III-A takes z = 0 for such data) and the
integer zero point is what Eq. 2's correction terms use.
"""
from __future__ import annotations

import numpy as np

LEVELS = 15          # 2^p - 1 for p = 4 (Eq. 1)


def quant_params(X: np.ndarray) -> tuple[np.float32, int]:
    """Scale factor and integer zero point of Eq. 1 for the finite float32 array X."""
    X = np.asarray(X, dtype=np.float32)
    lo = np.float32(min(np.float32(X.min()) if X.size else np.float32(0), np.float32(0)))
    hi = np.float32(max(np.float32(X.max()) if X.size else np.float32(0), np.float32(0)))
    s = np.float32(np.float32(hi - lo) / np.float32(LEVELS))
    if s == 0:
        s = np.float32(1)
    z = int(-np.floor(np.float32(lo / s)))
    return s, min(max(z, 0), LEVELS)


def quantize(X: np.ndarray, scale, zero: int, ldq: int | None = None) -> np.ndarray:
    """Codes of Eq. 1 for a rows x cols float32 matrix, packed two per byte along a row
    (low nibble = even column), row pitch ldq bytes (default: the packed row), pad bytes and
    an odd row's last high nibble 0."""
    X = np.asarray(X, dtype=np.float32)
    rows, cols = X.shape
    kb = (cols + 1) // 2
    ldq = kb if ldq is None else ldq
    t = np.floor(X / np.float32(scale))                    # float32 division, then floor
    codes = np.clip(t.astype(np.int64) + int(zero), 0, LEVELS).astype(np.uint8)
    if cols % 2:
        codes = np.concatenate([codes, np.zeros((rows, 1), np.uint8)], axis=1)
    Q = np.zeros((rows, ldq), dtype=np.uint8)
    Q[:, :kb] = codes[:, 0::2] | (codes[:, 1::2] << 4)
    return Q


def dequantize(C: np.ndarray, scale) -> np.ndarray:
    """Eq. 4: r = s * r_hat for an int32 matrix of results with zero point 0 (s = s_w * s_x, or
    the running product of Section III-B); the integer is converted to float32 (round to
    nearest even) and multiplied once."""
    return np.asarray(C, dtype=np.int32).astype(np.float32) * np.float32(scale)
