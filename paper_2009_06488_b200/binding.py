"""ctypes binding of the q4 CUDA library: same names as the C ABI in ``include/q4.h``.

Argument marshalling only -- tensors in, pointers and sizes out.  Every step of the
path runs in the library's kernels; there is no CPU fallback, and importing this
module without the built library raises.

Tensors are torch CUDA tensors: packed uint4 data as ``torch.uint8`` (two values per
byte, low nibble = even index), int32 for sums / bias / accumulators.  Pitches are
taken from the tensors' strides.  Calls enqueue on the current torch CUDA stream.
"""
from __future__ import annotations

import ctypes
import os
from dataclasses import dataclass

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libq4.so")

if not os.path.exists(LIB_PATH):
    raise ImportError(
        f"{LIB_PATH} is missing: build the CUDA library first "
        "(python -m paper_2009_06488_b200.build); there is no CPU fallback")

_lib = ctypes.CDLL(LIB_PATH)

(Q4_OK, Q4_ERR_INVALID_ARG, Q4_ERR_ALIGNMENT, Q4_ERR_RANGE, Q4_ERR_WORKSPACE,
 Q4_ERR_UNSUPPORTED, Q4_ERR_CUDA, Q4_ERR_DEVICE_TIMEOUT, Q4_ERR_STATIC_SCRATCH, Q4_ERR_WEIGHT_IMAGE) = range(10)
Q4_STATIC_SCRATCH_BYTES = 8 << 20

EXPORTS = ["q4_gemm", "q4_gemm_requant", "q4_im2col", "q4_conv2d", "q4_conv2d_static",
           "q4_gemm_workspace_bytes",
           "q4_conv2d_workspace_bytes", "q4_pack_bt", "q4_row_sums", "q4_gemm_host",
           "q4_gemm_host_staging_bytes", "q4_last_device_status", "q4_set_variant",
           "q4_launch_count", "q4_status_string", "q4_version", "q4_measure_mma_peak",
           "q4_quant_params", "q4_quantize", "q4_dequantize", "q4_gemm_u8",
           "q4_gemm_u8_workspace_bytes", "q4_selftest_wait_timeout", "q4_requant_channels", "q4_conv2d_channels",
           "q4_gemm_requant_channels", "q4_conv2d_weights_bytes", "q4_conv2d_prepare_weights",
           "q4_conv2d_prepared"]


class Q4Error(RuntimeError):
    def __init__(self, status: int, where: str):
        super().__init__(f"{where}: {q4_status_string(status)} (status {status})")
        self.status = status


class _Requant(ctypes.Structure):
    _fields_ = [(n, ctypes.c_int32) for n in ("mult", "shift", "zo", "clamp_lo", "clamp_hi")]


class _ConvDesc(ctypes.Structure):
    _fields_ = [(n, ctypes.c_int32) for n in
                ("N", "H", "W", "C", "OC", "KH", "KW", "stride_h", "stride_w", "pad_h", "pad_w")]


@dataclass(frozen=True)
class Requant:
    mult: int
    shift: int
    zo: int = 0
    clamp_lo: int = 0
    clamp_hi: int = 15

    def _c(self):
        return _Requant(self.mult, self.shift, self.zo, self.clamp_lo, self.clamp_hi)


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

    def _c(self):
        return _ConvDesc(self.N, self.H, self.W, self.C, self.OC, self.KH, self.KW,
                         self.stride_h, self.stride_w, self.pad_h, self.pad_w)

    @property
    def OH(self):
        return (self.H + 2 * self.pad_h - self.KH) // self.stride_h + 1

    @property
    def OW(self):
        return (self.W + 2 * self.pad_w - self.KW) // self.stride_w + 1

    @property
    def M(self):
        return self.N * self.OH * self.OW

    @property
    def K(self):
        return self.KH * self.KW * self.C


_vp, _i32, _i64, _sz = ctypes.c_void_p, ctypes.c_int32, ctypes.c_int64, ctypes.c_size_t
_lib.q4_gemm.argtypes = [_vp, _i64, _vp, _i64, _vp, _i64, _i32, _i32, _i32, _i32, _i32,
                         _vp, _vp, _vp, _sz, _vp]
_lib.q4_gemm_requant.argtypes = [_vp, _i64, _vp, _i64, _i32, _i32, _i32, _i32, _i32, _vp, _vp, _vp,
                                 ctypes.POINTER(_Requant), _vp, _i64, _vp, _sz, _vp]
_lib.q4_im2col.argtypes = [_vp, ctypes.POINTER(_ConvDesc), _i32, _vp, _i64, _vp, _vp]
_lib.q4_conv2d.argtypes = [_vp, _vp, _i64, _vp, _vp, ctypes.POINTER(_ConvDesc), _i32, _i32,
                           ctypes.POINTER(_Requant), _vp, _vp, _sz, _vp]
_lib.q4_conv2d_static.argtypes = [_vp, _vp, _i64, _vp, _vp, ctypes.POINTER(_ConvDesc), _i32, _i32,
                                  ctypes.POINTER(_Requant), _vp, _vp]
_lib.q4_conv2d_weights_bytes.argtypes = [ctypes.POINTER(_ConvDesc)]
_lib.q4_conv2d_weights_bytes.restype = _sz
_lib.q4_conv2d_prepare_weights.argtypes = [_vp, _i64, _vp, _vp, ctypes.POINTER(_ConvDesc), _i32, _i32, _vp, _sz, _vp]
_lib.q4_conv2d_prepared.argtypes = [_vp, _vp, _sz, ctypes.POINTER(_ConvDesc), _i32, ctypes.POINTER(_Requant), _vp, _vp]
_lib.q4_gemm_workspace_bytes.argtypes = [_i32, _i32, _i32]
_lib.q4_gemm_workspace_bytes.restype = _sz
_lib.q4_conv2d_workspace_bytes.argtypes = [ctypes.POINTER(_ConvDesc)]
_lib.q4_conv2d_workspace_bytes.restype = _sz
_lib.q4_pack_bt.argtypes = [_vp, _i64, _vp, _i64, _i32, _i32, _vp]
_lib.q4_row_sums.argtypes = [_vp, _i64, _i32, _i32, _vp, _vp]
_lib.q4_gemm_host.argtypes = [_vp, _i64, _vp, _i64, _vp, _i64, _i32, _i32, _i32, _i32, _i32,
                              _vp, _sz, _vp]
_lib.q4_gemm_host_staging_bytes.argtypes = [_i32, _i32, _i32, _i64, _i64, _i64]
_lib.q4_gemm_host_staging_bytes.restype = _sz
_lib.q4_measure_mma_peak.argtypes = [ctypes.c_int, ctypes.c_int, ctypes.c_int, _vp, ctypes.c_int, _vp]
_lib.q4_gemm_u8.argtypes = [_vp, _i64, _vp, _i64, _vp, _i64, _i32, _i32, _i32, _i32, _i32,
                            _vp, _vp, _vp, _sz, _vp]
_lib.q4_gemm_u8_workspace_bytes.argtypes = [_i32, _i32]
_lib.q4_gemm_u8_workspace_bytes.restype = _sz
_lib.q4_quant_params.argtypes = [_vp, _i64, _i32, _i32, _vp, _vp]
_lib.q4_quantize.argtypes = [_vp, _i64, _i32, _i32, _vp, _vp, _i64, _vp]
_lib.q4_dequantize.argtypes = [_vp, _i64, _i32, _i32, ctypes.c_float, _vp, _i64, _vp]
_lib.q4_selftest_wait_timeout.argtypes = [_vp, _vp]
_lib.q4_requant_channels.argtypes = [_vp, _i64, _i32, _i32, _i32, _i32, _vp, _vp, _vp, _vp, _vp,
                                     _i32, _i32, _i32, _vp, _i64, _vp]
_lib.q4_gemm_requant_channels.argtypes = [_vp, _i64, _vp, _i64, _i32, _i32, _i32, _i32, _vp, _vp, _vp, _vp, _vp, _vp,
                                          _i32, _i32, _i32, _vp, _i64, _vp, _sz, _vp]
_lib.q4_conv2d_channels.argtypes = [_vp, _vp, _i64, _vp, _vp, ctypes.POINTER(_ConvDesc), _i32, _vp, _vp, _vp,
                                    _i32, _i32, _i32, _vp, _vp]
_lib.q4_last_device_status.argtypes = [_vp]
_lib.q4_set_variant.argtypes = [ctypes.c_int]
_lib.q4_launch_count.restype = ctypes.c_uint64
_lib.q4_status_string.argtypes = [ctypes.c_int]
_lib.q4_status_string.restype = ctypes.c_char_p


def _ptr(t: torch.Tensor | None):
    return None if t is None else ctypes.c_void_p(t.data_ptr())


def _stream():
    return ctypes.c_void_p(torch.cuda.current_stream().cuda_stream)


def _dev(t: torch.Tensor | None, dtype, name: str):
    if t is None:
        return
    if not t.is_cuda:
        raise ValueError(f"{name} must be a CUDA tensor")
    if t.dtype != dtype:
        raise TypeError(f"{name} must be {dtype}")


def _rows(t: torch.Tensor, name: str) -> int:
    """Row pitch (in elements) of a 2-D tensor whose rows are contiguous."""
    if t.dim() != 2 or (t.shape[1] > 1 and t.stride(1) != 1):
        raise ValueError(f"{name} must be 2-D with contiguous rows")
    return t.stride(0) if t.shape[0] > 1 else max(t.shape[1], t.stride(0))


def _check(status: int, where: str):
    if status != Q4_OK:
        raise Q4Error(status, where)


def q4_status_string(status: int) -> str:
    return _lib.q4_status_string(status).decode()


def q4_version() -> int:
    return _lib.q4_version()


def q4_set_variant(variant: int) -> int:
    return _lib.q4_set_variant(variant)


def q4_launch_count() -> int:
    return int(_lib.q4_launch_count())


def q4_last_device_status() -> int:
    return _lib.q4_last_device_status(_stream())


def q4_measure_mma_peak(kind: int, n: int = 256, iters: int = 2048, num_ctas: int | None = None):
    """Multiply-accumulates per clock per SM of back-to-back tcgen05.mma (median over
    CTAs); kind 0 = i8, 1 = bf16, 2 = e4m3, 3 = i8 issued by CTA pairs.  Returns (mac_per_clk_per_sm, cycles_median)."""
    if num_ctas is None:
        num_ctas = torch.cuda.get_device_properties(torch.cuda.current_device()).multi_processor_count
    if kind == 3:
        num_ctas -= num_ctas % 2
    cycles = torch.zeros(num_ctas // 2 if kind == 3 else num_ctas, dtype=torch.int64, device="cuda")
    _check(_lib.q4_measure_mma_peak(kind, n, iters, _ptr(cycles), num_ctas, _stream()),
           "q4_measure_mma_peak")
    torch.cuda.synchronize()
    med = float(cycles.double().median().item())
    k = 16 if kind == 1 else 32
    return 4.0 * iters * 128 * n * k / med, med      # per SM: a pair instruction is 128 rows per SM


def q4_gemm_workspace_bytes(M: int, N: int, K: int) -> int:
    return int(_lib.q4_gemm_workspace_bytes(M, N, K))




def q4_conv2d_workspace_bytes(d: ConvDesc) -> int:
    c = d._c()
    return int(_lib.q4_conv2d_workspace_bytes(ctypes.byref(c)))


def q4_gemm(A, Bt, C, M, N, K, za, zb, rowsum_a=None, colsum_b=None, ws=None):
    _dev(A, torch.uint8, "A"); _dev(Bt, torch.uint8, "Bt"); _dev(C, torch.int32, "C")
    _dev(rowsum_a, torch.int32, "rowsum_a"); _dev(colsum_b, torch.int32, "colsum_b")
    _check(_lib.q4_gemm(_ptr(A), _rows(A, "A"), _ptr(Bt), _rows(Bt, "Bt"), _ptr(C), _rows(C, "C"),
                        M, N, K, za, zb, _ptr(rowsum_a), _ptr(colsum_b), _ptr(ws),
                        0 if ws is None else ws.numel() * ws.element_size(), _stream()), "q4_gemm")
    return C


def q4_gemm_requant(A, Bt, Cq, M, N, K, za, zb, rq: Requant, bias=None, rowsum_a=None,
                    colsum_b=None, ws=None):
    _dev(A, torch.uint8, "A"); _dev(Bt, torch.uint8, "Bt"); _dev(Cq, torch.uint8, "Cq")
    _dev(bias, torch.int32, "bias")
    _dev(rowsum_a, torch.int32, "rowsum_a"); _dev(colsum_b, torch.int32, "colsum_b")
    c = rq._c()
    _check(_lib.q4_gemm_requant(_ptr(A), _rows(A, "A"), _ptr(Bt), _rows(Bt, "Bt"), M, N, K, za, zb,
                                _ptr(rowsum_a), _ptr(colsum_b), _ptr(bias), ctypes.byref(c),
                                _ptr(Cq), _rows(Cq, "Cq"), _ptr(ws),
                                0 if ws is None else ws.numel() * ws.element_size(), _stream()),
           "q4_gemm_requant")
    return Cq


def q4_im2col(X, d: ConvDesc, za: int, A, rowsum_a=None):
    _dev(X, torch.uint8, "X"); _dev(A, torch.uint8, "A"); _dev(rowsum_a, torch.int32, "rowsum_a")
    c = d._c()
    _check(_lib.q4_im2col(_ptr(X), ctypes.byref(c), za, _ptr(A), _rows(A, "A"), _ptr(rowsum_a),
                          _stream()), "q4_im2col")
    return A


def q4_conv2d(X, Wt, d: ConvDesc, za: int, zb: int, rq: Requant, Y, ws, bias=None, colsum_w=None):
    _dev(X, torch.uint8, "X"); _dev(Wt, torch.uint8, "Wt"); _dev(Y, torch.uint8, "Y")
    _dev(bias, torch.int32, "bias"); _dev(colsum_w, torch.int32, "colsum_w")
    if ws is not None and not ws.is_cuda:
        raise ValueError("ws must be a CUDA tensor")
    c, r = d._c(), rq._c()
    _check(_lib.q4_conv2d(_ptr(X), _ptr(Wt), _rows(Wt, "Wt"), _ptr(colsum_w), _ptr(bias),
                          ctypes.byref(c), za, zb, ctypes.byref(r), _ptr(Y), _ptr(ws),
                          0 if ws is None else ws.numel() * ws.element_size(), _stream()),
           "q4_conv2d")
    return Y


def q4_conv2d_static(X, Wt, d: ConvDesc, za: int, zb: int, rq: Requant, Y, bias=None, colsum_w=None):
    """q4_conv2d for callers that cannot allocate: the workspace is the library's own
    fixed device array (Q4_STATIC_SCRATCH_BYTES).  Layers that need more are rejected
    with Q4_ERR_STATIC_SCRATCH.  One array per device: do not overlap calls."""
    _dev(X, torch.uint8, "X"); _dev(Wt, torch.uint8, "Wt"); _dev(Y, torch.uint8, "Y")
    _dev(bias, torch.int32, "bias"); _dev(colsum_w, torch.int32, "colsum_w")
    c, r = d._c(), rq._c()
    _check(_lib.q4_conv2d_static(_ptr(X), _ptr(Wt), _rows(Wt, "Wt"), _ptr(colsum_w), _ptr(bias),
                                 ctypes.byref(c), za, zb, ctypes.byref(r), _ptr(Y), _stream()),
           "q4_conv2d_static")
    return Y


def q4_conv2d_weights_bytes(d: ConvDesc) -> int:
    """Bytes of the layer's prepared weight image, 0 if the layer has no tensor-memory kernel."""
    c = d._c()
    return int(_lib.q4_conv2d_weights_bytes(ctypes.byref(c)))


def q4_conv2d_prepare_weights(Wt, d: ConvDesc, za: int, zb: int, prepared, bias=None, colsum_w=None):
    """The layer's weight-side work, once: writes the opaque image q4_conv2d_prepared runs from
    into ``prepared`` (uint8 CUDA tensor of q4_conv2d_weights_bytes(d) bytes); see include/q4.h."""
    _dev(Wt, torch.uint8, "Wt"); _dev(prepared, torch.uint8, "prepared")
    _dev(bias, torch.int32, "bias"); _dev(colsum_w, torch.int32, "colsum_w")
    c = d._c()
    _check(_lib.q4_conv2d_prepare_weights(_ptr(Wt), _rows(Wt, "Wt"), _ptr(colsum_w), _ptr(bias), ctypes.byref(c),
                                          za, zb, _ptr(prepared), prepared.numel(), _stream()),
           "q4_conv2d_prepare_weights")
    return prepared


def q4_conv2d_prepared(X, prepared, d: ConvDesc, za: int, rq: Requant, Y):
    """q4_conv2d from a prepared weight image (same output bytes, no workspace); see include/q4.h."""
    _dev(X, torch.uint8, "X"); _dev(prepared, torch.uint8, "prepared"); _dev(Y, torch.uint8, "Y")
    c, r = d._c(), rq._c()
    _check(_lib.q4_conv2d_prepared(_ptr(X), _ptr(prepared), prepared.numel(), ctypes.byref(c), za,
                                   ctypes.byref(r), _ptr(Y), _stream()), "q4_conv2d_prepared")
    return Y


def q4_pack_bt(B_kn, Bt, K: int, N: int):
    _dev(B_kn, torch.uint8, "B_kn"); _dev(Bt, torch.uint8, "Bt")
    _check(_lib.q4_pack_bt(_ptr(B_kn), _rows(B_kn, "B_kn"), _ptr(Bt), _rows(Bt, "Bt"), K, N,
                           _stream()), "q4_pack_bt")
    return Bt


def q4_gemm_u8_workspace_bytes(M: int, N: int) -> int:
    return int(_lib.q4_gemm_u8_workspace_bytes(M, N))


def q4_gemm_u8(A, Bt, C, M: int, N: int, K: int, za: int, zb: int, rowsum_a=None, colsum_b=None,
               ws=None):
    """8-bit product (one byte per value); see include/q4.h."""
    _dev(A, torch.uint8, "A"); _dev(Bt, torch.uint8, "Bt"); _dev(C, torch.int32, "C")
    for t, n in ((rowsum_a, "rowsum_a"), (colsum_b, "colsum_b")):
        if t is not None:
            _dev(t, torch.int32, n)
    if ws is not None:
        _dev(ws, torch.uint8, "ws")
    _check(_lib.q4_gemm_u8(_ptr(A), _rows(A, "A"), _ptr(Bt), _rows(Bt, "Bt"), _ptr(C), _rows(C, "C"),
                           M, N, K, za, zb, _ptr(rowsum_a), _ptr(colsum_b), _ptr(ws),
                           0 if ws is None else ws.numel(), _stream()), "q4_gemm_u8")
    return C


def _pitch_elems(t, name: str) -> int:
    if t.dim() == 1:
        return t.numel()
    if t.dim() != 2 or t.stride(1) != 1:
        raise ValueError(f"{name}: expected a 2-D tensor with contiguous rows")
    return t.stride(0)


def q4_quant_params(X, qp):
    """Eq. 1's scale and zero point of the float matrix X into ``qp``: a CUDA tensor of two
    32-bit words (``torch.int32``, shape [2]; word 0 holds the scale's float bits)."""
    _dev(X, torch.float32, "X"); _dev(qp, torch.int32, "qp")
    rows, cols = (1, X.numel()) if X.dim() == 1 else X.shape
    _check(_lib.q4_quant_params(_ptr(X), _pitch_elems(X, "X"), rows, cols, _ptr(qp), _stream()),
           "q4_quant_params")
    return qp


def q4_quantize(X, qp, Q):
    _dev(X, torch.float32, "X"); _dev(qp, torch.int32, "qp"); _dev(Q, torch.uint8, "Q")
    rows, cols = (1, X.numel()) if X.dim() == 1 else X.shape
    _check(_lib.q4_quantize(_ptr(X), _pitch_elems(X, "X"), rows, cols, _ptr(qp), _ptr(Q),
                            _rows(Q, "Q") if Q.dim() == 2 else Q.numel(), _stream()), "q4_quantize")
    return Q


def q4_dequantize(C, scale: float, R):
    _dev(C, torch.int32, "C"); _dev(R, torch.float32, "R")
    rows, cols = (1, C.numel()) if C.dim() == 1 else C.shape
    _check(_lib.q4_dequantize(_ptr(C), _pitch_elems(C, "C"), rows, cols, float(scale), _ptr(R),
                              _pitch_elems(R, "R"), _stream()), "q4_dequantize")
    return R


def q4_selftest_wait_timeout(outcome=None):
    """Launches the diagnostic kernel whose bounded wait runs out (see include/q4.h);
    ``outcome`` is an optional CUDA int32 tensor of one element."""
    _dev(outcome, torch.int32, "outcome")
    _check(_lib.q4_selftest_wait_timeout(_ptr(outcome), _stream()), "q4_selftest_wait_timeout")


def q4_requant_channels(C0, M: int, N: int, K: int, za: int, rowsum_a, zb, bias, mult, shift,
                        zo: int, clamp_lo: int, clamp_hi: int, Cq):
    """Finishes a product taken with zb = 0 for per-channel weight zero points and
    multipliers; see include/q4.h."""
    _dev(C0, torch.int32, "C0"); _dev(Cq, torch.uint8, "Cq")
    for t, n in ((rowsum_a, "rowsum_a"), (zb, "zb"), (bias, "bias"), (mult, "mult"), (shift, "shift")):
        _dev(t, torch.int32, n)
    _check(_lib.q4_requant_channels(_ptr(C0), _rows(C0, "C0"), M, N, K, za, _ptr(rowsum_a), _ptr(zb),
                                    _ptr(bias), _ptr(mult), _ptr(shift), zo, clamp_lo, clamp_hi,
                                    _ptr(Cq), _rows(Cq, "Cq"), _stream()), "q4_requant_channels")
    return Cq


def q4_gemm_requant_channels(A, Bt, Cq, M: int, N: int, K: int, za: int, zb, mult, shift, zo: int,
                             clamp_lo: int, clamp_hi: int, bias=None, rowsum_a=None, colsum_b=None, ws=None):
    """4-bit product with per-output-channel weight zero points, multipliers and shifts
    (CUDA int32 tensors of N elements) finished in the GEMM's epilogue; see include/q4.h."""
    _dev(A, torch.uint8, "A"); _dev(Bt, torch.uint8, "Bt"); _dev(Cq, torch.uint8, "Cq")
    for t, n in ((zb, "zb"), (mult, "mult"), (shift, "shift"), (bias, "bias"), (rowsum_a, "rowsum_a"),
                 (colsum_b, "colsum_b")):
        _dev(t, torch.int32, n)
    _check(_lib.q4_gemm_requant_channels(_ptr(A), _rows(A, "A"), _ptr(Bt), _rows(Bt, "Bt"), M, N, K, za,
                                         _ptr(zb), _ptr(rowsum_a), _ptr(colsum_b), _ptr(bias), _ptr(mult),
                                         _ptr(shift), zo, clamp_lo, clamp_hi, _ptr(Cq), _rows(Cq, "Cq"),
                                         _ptr(ws), 0 if ws is None else ws.numel() * ws.element_size(),
                                         _stream()), "q4_gemm_requant_channels")
    return Cq


def q4_conv2d_channels(X, Wt, d: ConvDesc, za: int, zb, mult, shift, zo: int, clamp_lo: int,
                       clamp_hi: int, Y, bias=None, colsum_w=None):
    """Fused convolution layer with per-output-channel weight zero points, multipliers and
    shifts (CUDA int32 tensors of OC elements); see include/q4.h."""
    _dev(X, torch.uint8, "X"); _dev(Wt, torch.uint8, "Wt"); _dev(Y, torch.uint8, "Y")
    for t, n in ((zb, "zb"), (mult, "mult"), (shift, "shift"), (bias, "bias"), (colsum_w, "colsum_w")):
        _dev(t, torch.int32, n)
    c = d._c()
    _check(_lib.q4_conv2d_channels(_ptr(X), _ptr(Wt), _rows(Wt, "Wt"), _ptr(colsum_w), _ptr(bias),
                                   ctypes.byref(c), za, _ptr(zb), _ptr(mult), _ptr(shift), zo, clamp_lo,
                                   clamp_hi, _ptr(Y), _stream()), "q4_conv2d_channels")
    return Y


def q4_row_sums(P, rows: int, K: int, sums):
    _dev(P, torch.uint8, "P"); _dev(sums, torch.int32, "sums")
    _check(_lib.q4_row_sums(_ptr(P), _rows(P, "P"), rows, K, _ptr(sums), _stream()), "q4_row_sums")
    return sums


def q4_gemm_host_staging_bytes(M, N, K, lda, ldb, ldc) -> int:
    return int(_lib.q4_gemm_host_staging_bytes(M, N, K, lda, ldb, ldc))


def q4_gemm_host(hA, hBt, hC, M, N, K, za, zb, dev_staging):
    """Host tensors in and out (pinned for asynchronous copies); ``dev_staging`` is a
    CUDA uint8 tensor of at least q4_gemm_host_staging_bytes bytes."""
    for t, n in ((hA, "hA"), (hBt, "hBt"), (hC, "hC")):
        if t.is_cuda:
            raise ValueError(f"{n} must be a host tensor")
    _check(_lib.q4_gemm_host(_ptr(hA), _rows(hA, "hA"), _ptr(hBt), _rows(hBt, "hBt"), _ptr(hC),
                             _rows(hC, "hC"), M, N, K, za, zb, _ptr(dev_staging),
                             dev_staging.numel(), _stream()), "q4_gemm_host")
    return hC
