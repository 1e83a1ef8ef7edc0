"""CPU oracle for the 4-bit quantized GEMM / convolution path -- TEST INFRASTRUCTURE ONLY.

Thin ctypes access to ``q4ref.c`` (plain C, 64-bit accumulation).  The oracle is the
plain definition of what the path computes (Eq. 2 / Eq. 3 of the paper and the
GEMM-based convolution it describes); it shares no code with the CUDA library and
must never be imported by the product package.  Only tests, the smoke check and the
benchmark's CPU-baseline leg may use it.

Arrays are numpy: packed uint4 data as ``uint8`` (two values per byte, low nibble =
even index, rows K-contiguous), sums / accumulators / bias as ``int32``.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from dataclasses import dataclass

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_LIB_PATH = os.path.join(_HERE, "libq4ref.so")
_SOURCES = [os.path.join(_HERE, "q4ref.c"), os.path.join(_HERE, "q4ref.h")]

OK, E_ARG, E_RANGE, E_PAD = 0, -1, -2, -4


class OracleError(RuntimeError):
    def __init__(self, code: int, where: str):
        super().__init__(f"{where}: oracle returned {code}")
        self.code = code


def build(force: bool = False) -> str:
    """Compile q4ref.c into libq4ref.so (gcc -O2 -fopenmp) if missing or stale."""
    stale = force or not os.path.exists(_LIB_PATH) or any(
        os.path.getmtime(s) > os.path.getmtime(_LIB_PATH) for s in _SOURCES)
    if stale:
        tmp = _LIB_PATH + f".tmp{os.getpid()}"
        subprocess.check_call(["gcc", "-O2", "-std=c11", "-fopenmp", "-fPIC", "-shared",
                               "-Wall", "-Wextra", "-o", tmp, _SOURCES[0]])
        os.replace(tmp, _LIB_PATH)
    return _LIB_PATH


class _ConvDesc(ctypes.Structure):
    _fields_ = [(n, ctypes.c_int32) for n in
                ("N", "H", "W", "C", "OC", "KH", "KW", "stride_h", "stride_w", "pad_h", "pad_w")]


class _Requant(ctypes.Structure):
    _fields_ = [(n, ctypes.c_int32) for n in ("mult", "shift", "zo", "clamp_lo", "clamp_hi")]


@dataclass(frozen=True)
class ConvDesc:
    N: int
    H: int
    W: int
    C: int
    OC: int
    KH: int
    KW: int
    stride_h: int = 1
    stride_w: int = 1
    pad_h: int = 0
    pad_w: int = 0

    def _c(self) -> _ConvDesc:
        return _ConvDesc(self.N, self.H, self.W, self.C, self.OC, self.KH, self.KW,
                         self.stride_h, self.stride_w, self.pad_h, self.pad_w)


@dataclass(frozen=True)
class Requant:
    mult: int
    shift: int
    zo: int = 0
    clamp_lo: int = 0
    clamp_hi: int = 15

    def _c(self) -> _Requant:
        return _Requant(self.mult, self.shift, self.zo, self.clamp_lo, self.clamp_hi)


_lib = None


def lib() -> ctypes.CDLL:
    global _lib
    if _lib is None:
        L = ctypes.CDLL(build())
        u8p, i32p = ctypes.c_void_p, ctypes.c_void_p
        i32, i64 = ctypes.c_int32, ctypes.c_int64
        L.q4ref_num_threads.restype = ctypes.c_int
        L.q4ref_set_num_threads.argtypes = [ctypes.c_int]
        L.q4ref_set_num_threads.restype = None
        L.q4ref_unpack_row.argtypes = [u8p, i64, u8p]
        L.q4ref_unpack_row.restype = None
        L.q4ref_pack_row.argtypes = [u8p, i64, u8p]
        L.q4ref_gemm.argtypes = [u8p, i64, u8p, i64, i32p, i64, i32, i32, i32, i32, i32]
        L.q4ref_gemm_fourterm.argtypes = [u8p, i64, u8p, i64, i32p, i64, i32, i32, i32, i32, i32,
                                          i32p, i32p]
        L.q4ref_requant_value.argtypes = [i64, ctypes.POINTER(_Requant)]
        L.q4ref_requant_value.restype = i32
        L.q4ref_requant_matrix.argtypes = [i32p, i64, i32, i32, i32p, ctypes.POINTER(_Requant),
                                           u8p, i64]
        L.q4ref_gemm_requant.argtypes = [u8p, i64, u8p, i64, i32, i32, i32, i32, i32, i32p,
                                         ctypes.POINTER(_Requant), u8p, i64]
        L.q4ref_conv_out.argtypes = [i32, i32, i32, i32]
        L.q4ref_conv_out.restype = i32
        L.q4ref_im2col.argtypes = [u8p, ctypes.POINTER(_ConvDesc), i32, u8p, i64, i32p]
        L.q4ref_conv2d_direct.argtypes = [u8p, u8p, i64, ctypes.POINTER(_ConvDesc), i32, i32, i32p]
        L.q4ref_conv2d.argtypes = [u8p, u8p, i64, i32p, ctypes.POINTER(_ConvDesc), i32, i32,
                                   ctypes.POINTER(_Requant), u8p]
        L.q4ref_pack_bt.argtypes = [u8p, i64, u8p, i64, i32, i32]
        _lib = L
    return _lib


def _p(a):
    return None if a is None else a.ctypes.data_as(ctypes.c_void_p)


def _u8(a, name):
    a = np.ascontiguousarray(a)
    if a.dtype != np.uint8:
        raise TypeError(f"{name} must be uint8")
    return a


def _i32(a, name):
    if a is None:
        return None
    a = np.ascontiguousarray(a)
    if a.dtype != np.int32:
        raise TypeError(f"{name} must be int32")
    return a


def _check(rc, where):
    if rc != OK:
        raise OracleError(rc, where)


def num_threads() -> int:
    return lib().q4ref_num_threads()


def set_num_threads(n: int) -> None:
    lib().q4ref_set_num_threads(n)


def unpack(packed: np.ndarray, count: int) -> np.ndarray:
    """Flat packed nibble array -> one value per byte (``count`` values)."""
    packed = _u8(packed, "packed")
    assert packed.size * 2 >= count
    out = np.empty(count, np.uint8)
    lib().q4ref_unpack_row(_p(packed), count, _p(out))
    return out


def pack(values: np.ndarray) -> np.ndarray:
    """One value per byte (0..15) -> flat packed nibble array."""
    values = _u8(values, "values").reshape(-1)
    out = np.empty((values.size + 1) // 2, np.uint8)
    _check(lib().q4ref_pack_row(_p(values), values.size, _p(out)), "pack")
    return out


def unpack_rows(P: np.ndarray, K: int) -> np.ndarray:
    """Packed matrix [rows, ld] -> values [rows, K]."""
    P = _u8(P, "P")
    return np.stack([unpack(P[r], K) for r in range(P.shape[0])]) if P.shape[0] else \
        np.empty((0, K), np.uint8)


def pack_rows(V: np.ndarray, ld: int | None = None) -> np.ndarray:
    """Values [rows, K] -> packed matrix [rows, ld] (pad bytes zero)."""
    V = _u8(V, "V")
    rows, K = V.shape
    ld = (K + 1) // 2 if ld is None else ld
    out = np.zeros((rows, ld), np.uint8)
    for r in range(rows):
        out[r, :(K + 1) // 2] = pack(V[r])
    return out


def gemm(A, Bt, M, N, K, za, zb, lda=None, ldb=None) -> np.ndarray:
    A, Bt = _u8(A, "A"), _u8(Bt, "Bt")
    lda = A.shape[1] if lda is None else lda
    ldb = Bt.shape[1] if ldb is None else ldb
    C = np.empty((M, N), np.int32)
    _check(lib().q4ref_gemm(_p(A), lda, _p(Bt), ldb, _p(C), N, M, N, K, za, zb), "gemm")
    return C


def gemm_fourterm(A, Bt, M, N, K, za, zb, lda=None, ldb=None):
    """Returns (C, rowsum_a, colsum_b) through the four terms of Eq. 2."""
    A, Bt = _u8(A, "A"), _u8(Bt, "Bt")
    lda = A.shape[1] if lda is None else lda
    ldb = Bt.shape[1] if ldb is None else ldb
    C = np.empty((M, N), np.int32)
    ra = np.empty(M, np.int32)
    cb = np.empty(N, np.int32)
    _check(lib().q4ref_gemm_fourterm(_p(A), lda, _p(Bt), ldb, _p(C), N, M, N, K, za, zb,
                                     _p(ra), _p(cb)), "gemm_fourterm")
    return C, ra, cb


def requant_value(acc: int, rq: Requant) -> int:
    c = rq._c()
    return int(lib().q4ref_requant_value(int(acc), ctypes.byref(c)))


def requant_matrix(C, bias, rq: Requant) -> np.ndarray:
    C = _i32(C, "C")
    bias = _i32(bias, "bias")
    M, N = C.shape
    Cq = np.zeros((M, N // 2), np.uint8)
    c = rq._c()
    _check(lib().q4ref_requant_matrix(_p(C), N, M, N, _p(bias), ctypes.byref(c), _p(Cq), N // 2),
           "requant_matrix")
    return Cq


def gemm_requant(A, Bt, M, N, K, za, zb, bias, rq: Requant, lda=None, ldb=None) -> np.ndarray:
    A, Bt = _u8(A, "A"), _u8(Bt, "Bt")
    bias = _i32(bias, "bias")
    lda = A.shape[1] if lda is None else lda
    ldb = Bt.shape[1] if ldb is None else ldb
    Cq = np.zeros((M, N // 2), np.uint8)
    c = rq._c()
    _check(lib().q4ref_gemm_requant(_p(A), lda, _p(Bt), ldb, M, N, K, za, zb, _p(bias),
                                    ctypes.byref(c), _p(Cq), N // 2), "gemm_requant")
    return Cq


def conv_out(inp: int, k: int, stride: int, pad: int) -> int:
    return int(lib().q4ref_conv_out(inp, k, stride, pad))


def conv_gemm_shape(d: ConvDesc):
    """(M, K, OH, OW) of the GEMM a convolution unrolls to."""
    OH = conv_out(d.H, d.KH, d.stride_h, d.pad_h)
    OW = conv_out(d.W, d.KW, d.stride_w, d.pad_w)
    return d.N * OH * OW, d.KH * d.KW * d.C, OH, OW


def im2col(X, d: ConvDesc, za: int, lda: int | None = None):
    """Returns (A [M, lda] packed, rowsum_a [M])."""
    X = _u8(X, "X")
    M, K, _, _ = conv_gemm_shape(d)
    lda = (K + 1) // 2 if lda is None else lda
    A = np.full((M, lda), 0xA5, np.uint8)
    ra = np.empty(M, np.int32)
    c = d._c()
    _check(lib().q4ref_im2col(_p(X), ctypes.byref(c), za, _p(A), lda, _p(ra)), "im2col")
    return A, ra


def conv2d_direct(X, Wt, d: ConvDesc, za: int, zb: int, ldw=None) -> np.ndarray:
    """int32 NHWC result [N, OH, OW, OC] of the direct convolution sum."""
    X, Wt = _u8(X, "X"), _u8(Wt, "Wt")
    ldw = Wt.shape[1] if ldw is None else ldw
    _, _, OH, OW = conv_gemm_shape(d)
    Y = np.empty((d.N, OH, OW, d.OC), np.int32)
    c = d._c()
    _check(lib().q4ref_conv2d_direct(_p(X), _p(Wt), ldw, ctypes.byref(c), za, zb, _p(Y)),
           "conv2d_direct")
    return Y


def conv2d(X, Wt, bias, d: ConvDesc, za: int, zb: int, rq: Requant, ldw=None) -> np.ndarray:
    """Packed uint4 NHWC output, flat [N*OH*OW, OC/2]."""
    X, Wt = _u8(X, "X"), _u8(Wt, "Wt")
    bias = _i32(bias, "bias")
    ldw = Wt.shape[1] if ldw is None else ldw
    M, _, _, _ = conv_gemm_shape(d)
    Y = np.zeros((M, d.OC // 2), np.uint8)
    c, r = d._c(), rq._c()
    _check(lib().q4ref_conv2d(_p(X), _p(Wt), ldw, _p(bias), ctypes.byref(c), za, zb,
                              ctypes.byref(r), _p(Y)), "conv2d")
    return Y


def pack_bt(B_kn, K: int, N: int, ldb: int | None = None) -> np.ndarray:
    B_kn = _u8(B_kn, "B_kn")
    ldb = (K + 1) // 2 if ldb is None else ldb
    Bt = np.full((N, ldb), 0xA5, np.uint8)
    _check(lib().q4ref_pack_bt(_p(B_kn), B_kn.shape[1], _p(Bt), ldb, K, N), "pack_bt")
    return Bt


# The float boundary of a quantized layer (Eq. 1 quantizer, Eq. 4 scale-back), numpy float32.
from .qfloat import dequantize, quant_params, quantize  # noqa: E402,F401

# The 8-bit product of the paper's comparison (Eq. 2 with 8-bit values), numpy int64.
from .q8 import gemm_u8, gemm_u8_fourterm  # noqa: E402,F401

# Per-output-channel weight zero points and re-quantization multipliers, numpy int64.
from .perchannel import gemm_channels, requant_channels  # noqa: E402,F401
