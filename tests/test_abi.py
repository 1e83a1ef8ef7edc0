"""The C-ABI library loads without a GPU, exports every symbol the header declares,
and validates arguments on the host before touching the device."""
import ctypes
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    from paper_2009_06488_b200 import build
    return ctypes.CDLL(build.build())


def declared_symbols():
    text = open(os.path.join(ROOT, "include", "q4.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(q4_[a-z0-9_]+)\s*\(", text)))


def test_header_declares_the_four_calls():
    syms = declared_symbols()
    for name in ("q4_gemm", "q4_gemm_requant", "q4_im2col", "q4_conv2d"):
        assert name in syms


def test_library_exports_every_declared_symbol(lib):
    for name in declared_symbols():
        assert hasattr(lib, name), name


def test_binding_lists_the_same_symbols():
    from paper_2009_06488_b200 import binding
    assert sorted(binding.EXPORTS) == declared_symbols()
    for name in binding.EXPORTS:
        assert hasattr(binding, name) or name in ("q4_gemm_workspace_bytes",)


def test_status_strings_and_version(lib):
    lib.q4_status_string.restype = ctypes.c_char_p
    assert lib.q4_status_string(0) == b"ok"
    assert len({lib.q4_status_string(i) for i in range(8)}) == 8
    assert lib.q4_version() >= 100


class RQ(ctypes.Structure):
    _fields_ = [(n, ctypes.c_int32) for n in ("mult", "shift", "zo", "lo", "hi")]


class CD(ctypes.Structure):
    _fields_ = [(n, ctypes.c_int32) for n in
                ("N", "H", "W", "C", "OC", "KH", "KW", "sh", "sw", "ph", "pw")]


def test_host_side_validation_needs_no_device(lib):
    vp, i32, i64, sz = ctypes.c_void_p, ctypes.c_int32, ctypes.c_int64, ctypes.c_size_t
    lib.q4_gemm.argtypes = [vp, i64, vp, i64, vp, i64, i32, i32, i32, i32, i32, vp, vp, vp, sz, vp]
    fake = 0x1000   # never dereferenced: every call below is rejected before any launch
    INVALID, ALIGN, RANGE, WORKSPACE = 1, 2, 3, 4
    g = lambda **kw: lib.q4_gemm(kw.get("A", fake), kw.get("lda", 64), kw.get("B", fake),
                                 kw.get("ldb", 64), kw.get("C", fake), kw.get("ldc", 8),
                                 kw.get("M", 8), kw.get("N", 8), kw.get("K", 128),
                                 kw.get("za", 0), kw.get("zb", 0), None, None, None, 0, None)
    assert g(K=0) == INVALID
    assert g(M=-1) == INVALID
    assert g(A=None) == INVALID
    assert g(C=None) == INVALID
    assert g(lda=63) == INVALID            # pitch shorter than a row of 128 nibbles
    assert g(ldc=7) == INVALID
    assert g(za=16) == RANGE
    assert g(zb=-1) == RANGE
    assert g(K=(1 << 22) + 1, lda=1 << 22, ldb=1 << 22) == RANGE
    assert g(C=fake + 2) == ALIGN
    assert g(M=0) == 0 and g(N=0) == 0      # empty problems are no-ops

    lib.q4_gemm_requant.argtypes = [vp, i64, vp, i64, i32, i32, i32, i32, i32, vp, vp, vp,
                                    ctypes.POINTER(RQ), vp, i64, vp, sz, vp]
    def r(rq, N=8, ldcq=4):
        return lib.q4_gemm_requant(fake, 64, fake, 64, 8, N, 128, 0, 0, None, None, None,
                                   ctypes.byref(rq) if rq else None, fake, ldcq, None, 0, None)
    assert r(None) == INVALID
    assert r(RQ(1 << 29, 8, 0, 0, 15)) == RANGE
    assert r(RQ(1 << 30, 32, 0, 0, 15)) == RANGE
    assert r(RQ(1 << 30, 8, 16, 0, 15)) == RANGE
    assert r(RQ(1 << 30, 8, 0, 9, 8)) == RANGE
    assert r(RQ(1 << 30, 8, 0, 0, 15), N=7) == INVALID
    assert r(RQ(1 << 30, 8, 0, 0, 15), ldcq=3) == INVALID

    lib.q4_conv2d.argtypes = [vp, vp, i64, vp, vp, ctypes.POINTER(CD), i32, i32,
                              ctypes.POINTER(RQ), vp, vp, sz, vp]
    lib.q4_conv2d_workspace_bytes.argtypes = [ctypes.POINTER(CD)]
    lib.q4_conv2d_workspace_bytes.restype = sz
    d = CD(2, 8, 8, 16, 32, 3, 3, 1, 1, 1, 1)
    rq = RQ(1 << 30, 8, 0, 0, 15)
    need = lib.q4_conv2d_workspace_bytes(ctypes.byref(d))
    assert need >= 2 * 8 * 8 * (80 + 4)     # unrolled matrix at a 16-byte-multiple pitch + row sums
    c = lambda d, ws, wsb: lib.q4_conv2d(fake, fake, 72, None, None, ctypes.byref(d), 0, 0,
                                         ctypes.byref(rq), fake, ws, wsb, None)
    assert c(d, None, 0) == WORKSPACE
    assert c(d, 0x10000, need - 1) == WORKSPACE
    assert c(d, 0x10010, need) == ALIGN
    assert c(CD(2, 2, 2, 16, 32, 3, 3, 1, 1, 0, 0), 0x10000, 1 << 20) == INVALID   # kernel larger than image
    assert c(CD(2, 8, 8, 16, 31, 3, 3, 1, 1, 1, 1), 0x10000, 1 << 20) == INVALID   # odd channel count out

    # the entry point with built-in scratch checks its arguments like q4_conv2d, before its size
    # test and before it looks up the array: none of these calls needs a device
    lib.q4_conv2d_static.argtypes = [vp, vp, i64, vp, vp, ctypes.POINTER(CD), i32, i32, ctypes.POINTER(RQ), vp, vp]
    st = lambda d, **kw: lib.q4_conv2d_static(kw.get("X", fake), fake, kw.get("ldw", 72), None, None, ctypes.byref(d),
                                              kw.get("za", 0), kw.get("zb", 0),
                                              ctypes.byref(kw.get("rq", rq)) if kw.get("rq", rq) else None, fake, None)
    big = CD(256, 32, 32, 16, 32, 3, 3, 1, 1, 1, 1)                 # needs ~21 MB of scratch
    assert st(big) == 8                                              # Q4_ERR_STATIC_SCRATCH
    assert st(big, rq=None) == INVALID and st(big, zb=16) == RANGE and st(big, ldw=71) == INVALID
    assert st(big, rq=RQ(1 << 29, 8, 0, 0, 15)) == RANGE and st(big, X=None) == INVALID
    assert st(CD(256, 32, 32, 16, 31, 3, 3, 1, 1, 1, 1)) == INVALID
    assert st(CD(0, 32, 32, 16, 32, 3, 3, 1, 1, 1, 1)) == 0         # empty: no-op, no lookup


def test_compute_call_without_a_device_fails_loudly(lib):
    import torch
    if torch.cuda.is_available():
        pytest.skip("a device is present")
    vp, i32, i64, sz = ctypes.c_void_p, ctypes.c_int32, ctypes.c_int64, ctypes.c_size_t
    lib.q4_gemm.argtypes = [vp, i64, vp, i64, vp, i64, i32, i32, i32, i32, i32, vp, vp, vp, sz, vp]
    assert lib.q4_gemm(0x1000, 64, 0x1000, 64, 0x1000, 8, 8, 8, 128, 0, 0, None, None, None, 0,
                       None) == 6   # Q4_ERR_CUDA: no silent CPU path


def test_validation_of_the_float_boundary_and_the_8bit_product(lib):
    vp, i32, i64, sz = ctypes.c_void_p, ctypes.c_int32, ctypes.c_int64, ctypes.c_size_t
    fake = 0x1000
    INVALID, ALIGN, RANGE, WORKSPACE = 1, 2, 3, 4
    lib.q4_gemm_u8.argtypes = [vp, i64, vp, i64, vp, i64, i32, i32, i32, i32, i32, vp, vp, vp, sz, vp]
    lib.q4_gemm_u8_workspace_bytes.argtypes = [i32, i32]
    lib.q4_gemm_u8_workspace_bytes.restype = sz
    u = lambda **kw: lib.q4_gemm_u8(kw.get("A", fake), kw.get("lda", 128), fake, 128, kw.get("C", fake), 8,
                                    kw.get("M", 8), 8, kw.get("K", 128), kw.get("za", 0), kw.get("zb", 0),
                                    kw.get("ra", fake), kw.get("cb", fake), kw.get("ws"), kw.get("wsb", 0), None)
    assert u(K=0) == INVALID and u(M=-1) == INVALID and u(A=None) == INVALID
    assert u(lda=127) == INVALID                     # pitch shorter than a row
    assert u(za=256) == RANGE and u(zb=-1) == RANGE
    assert u(K=33025, lda=33040) == INVALID          # ldb (128) is shorter than the row
    assert lib.q4_gemm_u8(fake, 33040, fake, 33040, fake, 8, 8, 8, 33025, 0, 0, fake, fake, None, 0, None) == RANGE
    assert u(A=fake + 8) == ALIGN and u(lda=136) == ALIGN and u(C=fake + 2) == ALIGN
    assert u(ra=None) == WORKSPACE                   # sums wanted, no workspace given
    assert u(ra=None, ws=0x2000, wsb=lib.q4_gemm_u8_workspace_bytes(8, 8) - 1) == WORKSPACE
    assert u(M=0) == 0
    assert lib.q4_gemm_u8_workspace_bytes(1000, 10) >= 4 * 1010

    lib.q4_quant_params.argtypes = [vp, i64, i32, i32, vp, vp]
    lib.q4_quantize.argtypes = [vp, i64, i32, i32, vp, vp, i64, vp]
    lib.q4_dequantize.argtypes = [vp, i64, i32, i32, ctypes.c_float, vp, i64, vp]
    assert lib.q4_quant_params(fake, 7, 4, 8, fake, None) == INVALID       # pitch shorter than a row
    assert lib.q4_quant_params(fake, 8, 4, 8, None, None) == INVALID
    assert lib.q4_quant_params(fake + 2, 8, 4, 8, fake, None) == ALIGN
    assert lib.q4_quantize(fake, 8, 4, 8, fake, fake, 3, None) == INVALID  # 8 codes need 4 bytes
    assert lib.q4_quantize(fake, 8, 4, 9, fake, fake, 4, None) == INVALID  # 9 codes need 5 bytes
    assert lib.q4_quantize(fake, 8, 0, 8, fake, fake, 4, None) == 0        # empty: no-op
    assert lib.q4_quantize(None, 8, 4, 8, fake, fake, 4, None) == INVALID
    assert lib.q4_dequantize(fake, 7, 4, 8, 1.0, fake, 8, None) == INVALID
    assert lib.q4_dequantize(fake, 8, 4, 8, 1.0, fake + 1, 8, None) == ALIGN
    assert lib.q4_dequantize(fake, 8, 4, 0, 1.0, fake, 8, None) == 0


def test_validation_of_the_per_channel_entry_points(lib):
    vp, i32, i64 = ctypes.c_void_p, ctypes.c_int32, ctypes.c_int64
    fake = 0x1000
    INVALID, ALIGN, RANGE = 1, 2, 3
    lib.q4_requant_channels.argtypes = [vp, i64, i32, i32, i32, i32, vp, vp, vp, vp, vp, i32, i32, i32, vp, i64, vp]
    r = lambda **kw: lib.q4_requant_channels(kw.get("C0", fake), kw.get("ldc", 8), kw.get("M", 4), kw.get("N", 8),
                                             kw.get("K", 16), kw.get("za", 0), kw.get("ra", fake), None, None,
                                             kw.get("mult", fake), fake, kw.get("zo", 0), kw.get("lo", 0),
                                             kw.get("hi", 15), fake, kw.get("ldcq", 4), None)
    assert r(N=7) == INVALID and r(ldc=7) == INVALID and r(ldcq=3) == INVALID and r(K=0) == INVALID
    assert r(za=16) == RANGE and r(zo=-1) == RANGE and r(lo=9, hi=8) == RANGE
    assert r(mult=None) == INVALID and r(ra=None) == INVALID
    assert r(C0=fake + 2) == ALIGN
    assert r(M=0) == 0

    lib.q4_conv2d_channels.argtypes = [vp, vp, i64, vp, vp, ctypes.POINTER(CD), i32, vp, vp, vp, i32, i32, i32, vp, vp]
    c = lambda d, **kw: lib.q4_conv2d_channels(fake, fake, kw.get("ldw", 72), None, None, ctypes.byref(d),
                                               kw.get("za", 0), kw.get("zb", fake), fake, fake, 0, 0,
                                               kw.get("hi", 15), kw.get("Y", fake), None)
    d = CD(2, 8, 8, 16, 32, 3, 3, 1, 1, 1, 1)
    assert c(d, ldw=71) == INVALID and c(d, zb=None) == INVALID
    assert c(d, za=16) == RANGE and c(d, hi=16) == RANGE
    assert c(d, zb=fake + 2) == ALIGN
    assert c(CD(2, 8, 8, 16, 72, 3, 3, 1, 1, 1, 1), ldw=72) == 5            # unsupported: 72 output channels
    assert c(d, Y=fake + 4) == 5                                            # unsupported: Y not 8-byte aligned
    assert c(CD(0, 8, 8, 16, 32, 3, 3, 1, 1, 1, 1)) == 0


def test_prepared_weight_entry_points_validate_without_a_device(lib):
    vp, i32, i64, sz = ctypes.c_void_p, ctypes.c_int32, ctypes.c_int64, ctypes.c_size_t
    INVALID, ALIGN, RANGE, WORKSPACE = 1, 2, 3, 4
    lib.q4_conv2d_weights_bytes.argtypes = [ctypes.POINTER(CD)]
    lib.q4_conv2d_weights_bytes.restype = sz
    lib.q4_conv2d_prepare_weights.argtypes = [vp, i64, vp, vp, ctypes.POINTER(CD), i32, i32, vp, sz, vp]
    lib.q4_conv2d_prepared.argtypes = [vp, vp, sz, ctypes.POINTER(CD), i32, ctypes.POINTER(RQ), vp, vp]
    lib.q4_status_string.restype = ctypes.c_char_p
    UNSUPPORTED = next(c for c in range(1, 16) if b"unsupported" in lib.q4_status_string(c).lower()
                       or b"not supported" in lib.q4_status_string(c).lower())
    fake = 0x1000       # never dereferenced
    c3 = CD(2, 32, 32, 16, 32, 3, 3, 1, 1, 1, 1)          # a layer class of the tensor-memory kernels
    wide = CD(2, 16, 16, 128, 256, 3, 3, 1, 1, 1, 1)       # two CTAs' shares
    odd = CD(2, 9, 11, 3, 6, 5, 5, 1, 1, 2, 2)             # no tensor-memory kernel
    nb = lib.q4_conv2d_weights_bytes(ctypes.byref(c3))
    # B: 64 columns x 7 depth steps of 32 bytes in two 128-byte blocks, 64 constants, 16 bytes of flag
    assert nb == 2 * 64 * 128 + 64 * 4 + 16
    nw = lib.q4_conv2d_weights_bytes(ctypes.byref(wide))
    assert nw == 2 * (10 * 128 * 128 + 128 * 4 + 16)       # 36 + 1 steps -> ten blocks of 128 columns
    assert lib.q4_conv2d_weights_bytes(ctypes.byref(odd)) == 0
    assert lib.q4_conv2d_weights_bytes(None) == 0
    rq = RQ(1 << 30, 8, 0, 0, 15)
    prep = lambda d, **kw: lib.q4_conv2d_prepare_weights(kw.get("Wt", fake), kw.get("ldw", 72), None, None, ctypes.byref(d),
                                                         kw.get("za", 0), kw.get("zb", 0), kw.get("out", fake),
                                                         kw.get("nbytes", nb), None)
    assert prep(c3, Wt=None) == INVALID
    assert prep(c3, out=None) == INVALID
    assert prep(c3, ldw=71) == INVALID
    assert prep(c3, zb=16) == RANGE
    assert prep(c3, za=-1) == RANGE
    assert prep(c3, nbytes=nb - 1) == WORKSPACE
    assert prep(c3, out=fake + 8) == ALIGN
    assert prep(odd, ldw=38) == UNSUPPORTED
    run = lambda d, **kw: lib.q4_conv2d_prepared(kw.get("X", fake), kw.get("img", fake), kw.get("nbytes", nb), ctypes.byref(d),
                                                 kw.get("za", 0), ctypes.byref(kw.get("rq", rq)), kw.get("Y", fake), None)
    assert run(c3, img=None) == INVALID
    assert run(c3, X=None) == INVALID
    assert run(c3, Y=None) == INVALID
    assert run(c3, nbytes=nb - 16) == WORKSPACE
    assert run(c3, img=fake + 4) == ALIGN
    assert run(c3, rq=RQ(1 << 29, 8, 0, 0, 15)) == RANGE
    assert run(c3, Y=fake + 8) == UNSUPPORTED               # output rows not 16-byte aligned: use q4_conv2d
    assert run(odd) == UNSUPPORTED
    assert run(CD(0, 32, 32, 16, 32, 3, 3, 1, 1, 1, 1)) == 0    # empty batch: a no-op
