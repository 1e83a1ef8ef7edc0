"""Pins for the CPU oracle: it is checked against things other than itself --
library routines on special cases, closed forms, constants the paper prints,
arbitrary-precision arithmetic and brute force on tiny inputs."""
import itertools
import os

import numpy as np
import pytest
from hypothesis import given, settings, strategies as st

import oracle
from oracle import ConvDesc, Requant
from paper_2009_06488_b200 import workloads as wl

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def paper_constants():
    out = {}
    with open(os.path.join(GOLDEN, "paper_constants.txt")) as f:
        for line in f:
            line = line.split("#")[0].strip()
            if line:
                k, v = line.split("=")
                out[k.strip()] = int(v)
    return out


def rand_vals(rng, rows, K):
    return rng.integers(0, 16, size=(rows, K), dtype=np.uint8)


# ---------------------------------------------------------------- packing

def test_packing_hand_written_bytes():
    # low nibble = even index: values 1,2,3,4 -> bytes 0x21, 0x43
    assert oracle.pack(np.array([1, 2, 3, 4], np.uint8)).tolist() == [0x21, 0x43]
    assert oracle.pack(np.array([15, 0, 0, 15, 7], np.uint8)).tolist() == [0x0F, 0xF0, 0x07]
    assert oracle.unpack(np.array([0x21, 0x43], np.uint8), 4).tolist() == [1, 2, 3, 4]
    assert oracle.unpack(np.array([0xAB], np.uint8), 2).tolist() == [0xB, 0xA]


def test_packing_round_trip_and_numpy_bit_ops():
    rng = np.random.default_rng(1)
    for count in (1, 2, 3, 16, 17, 255):
        v = rng.integers(0, 16, count, dtype=np.uint8)
        p = oracle.pack(v)
        assert oracle.unpack(p, count).tolist() == v.tolist()
        # same bytes from numpy bit operations on the even / odd elements
        vv = np.concatenate([v, np.zeros(count & 1, np.uint8)])
        assert p.tolist() == (vv[0::2] | (vv[1::2] << 4)).tolist()


def test_pack_rejects_values_above_15():
    with pytest.raises(oracle.OracleError):
        oracle.pack(np.array([16], np.uint8))


def test_generator_bytes_are_packed_uniform_nibbles():
    P = wl.rand_packed(7, 1, 64, 255)
    assert P.shape == (64, 128)
    assert (P[:, -1] >> 4 == 0).all()          # odd K: last high nibble is zero
    V = oracle.unpack_rows(P, 255)
    hist = np.bincount(V.reshape(-1), minlength=16)
    assert hist.min() > 0.8 * V.size / 16 and hist.max() < 1.2 * V.size / 16
    # counter-based: same stream twice, different stream differs
    assert (wl.rand_packed(7, 1, 64, 255) == P).all()
    assert (wl.rand_packed(7, 2, 64, 255) != P).any()


# ---------------------------------------------------------------- GEMM value

def test_gemm_brute_force_depth_one_exhaustive():
    # M = all 16 values of a, N = all 16 values of b, K = 1, every zero-point pair.
    a = np.arange(16, dtype=np.uint8).reshape(16, 1)
    A = oracle.pack_rows(a)
    for za, zb in itertools.product(range(16), range(16)):
        C = oracle.gemm(A, A, 16, 16, 1, za, zb)
        for i in range(16):
            for j in range(16):
                assert C[i, j] == (i - za) * (j - zb)


def test_gemm_brute_force_depth_two():
    pairs = np.array(list(itertools.product(range(16), range(16))), np.uint8)  # 256 x 2
    P = oracle.pack_rows(pairs)
    for za, zb in [(0, 0), (7, 8), (15, 0), (0, 15), (15, 15), (3, 12)]:
        C = oracle.gemm(P, P, 256, 256, 2, za, zb)
        for m in range(0, 256, 7):
            for n in range(0, 256, 5):
                a0, a1 = int(pairs[m, 0]), int(pairs[m, 1])
                b0, b1 = int(pairs[n, 0]), int(pairs[n, 1])
                assert C[m, n] == (a0 - za) * (b0 - zb) + (a1 - za) * (b1 - zb)


# the paper's Table I shapes: left matrix H x D, right matrix D x W
TABLE1 = [(h, w, d) for h in (8, 24) for w in (100, 400, 1600) for d in (10, 40, 100)]


@pytest.mark.parametrize("shape", TABLE1 + [(1, 1, 1), (3, 5, 7), (65, 33, 129), (130, 70, 255)])
def test_gemm_matches_numpy_matmul_of_shifted_operands(shape):
    M, N, K = shape
    rng = np.random.default_rng(M * 1000003 + N * 101 + K)
    a, b = rand_vals(rng, M, K), rand_vals(rng, N, K)
    A, Bt = oracle.pack_rows(a, (K + 1) // 2 + 3), oracle.pack_rows(b)
    # zero points 0: plain non-negative integer matrix product (library routine)
    C0 = oracle.gemm(A, Bt, M, N, K, 0, 0)
    assert (C0 == a.astype(np.int64) @ b.astype(np.int64).T).all()
    # any zero points: library product of the shifted operands
    za, zb = int(rng.integers(0, 16)), int(rng.integers(0, 16))
    C = oracle.gemm(A, Bt, M, N, K, za, zb)
    assert (C == (a.astype(np.int64) - za) @ (b.astype(np.int64) - zb).T).all()


def test_gemm_four_term_identity_eq2():
    rng = np.random.default_rng(5)
    for M, N, K in [(8, 100, 10), (24, 40, 100), (17, 9, 33), (64, 64, 256)]:
        a, b = rand_vals(rng, M, K), rand_vals(rng, N, K)
        A, Bt = oracle.pack_rows(a), oracle.pack_rows(b)
        for za, zb in [(0, 0), (7, 8), (15, 15), (0, 15), (11, 2)]:
            C = oracle.gemm(A, Bt, M, N, K, za, zb)
            C4, ra, cb = oracle.gemm_fourterm(A, Bt, M, N, K, za, zb)
            assert (C == C4).all()
            assert (ra == a.sum(1, dtype=np.int64)).all()
            assert (cb == b.sum(1, dtype=np.int64)).all()


def test_gemm_invariants():
    rng = np.random.default_rng(6)
    M, N, K1, K2 = 13, 11, 21, 10
    za, zb = 5, 9
    a, b = rand_vals(rng, M, K1 + K2), rand_vals(rng, N, K1 + K2)
    C = oracle.gemm(oracle.pack_rows(a), oracle.pack_rows(b), M, N, K1 + K2, za, zb)
    # operand identically equal to its zero point -> result identically zero
    Az = oracle.pack_rows(np.full((M, K1), za, np.uint8))
    assert (oracle.gemm(Az, oracle.pack_rows(b[:, :K1]), M, N, K1, za, zb) == 0).all()
    Bz = oracle.pack_rows(np.full((N, K1), zb, np.uint8))
    assert (oracle.gemm(oracle.pack_rows(a[:, :K1]), Bz, M, N, K1, za, zb) == 0).all()
    # additivity in the depth
    Ca = oracle.gemm(oracle.pack_rows(a[:, :K1]), oracle.pack_rows(b[:, :K1]), M, N, K1, za, zb)
    Cb = oracle.gemm(oracle.pack_rows(a[:, K1:]), oracle.pack_rows(b[:, K1:]), M, N, K2, za, zb)
    assert (C == Ca + Cb).all()
    # transposition symmetry
    Ct = oracle.gemm(oracle.pack_rows(b), oracle.pack_rows(a), N, M, K1 + K2, zb, za)
    assert (C.T == Ct).all()
    # the same depth permutation applied to both operands changes nothing
    perm = rng.permutation(K1 + K2)
    Cp = oracle.gemm(oracle.pack_rows(a[:, perm]), oracle.pack_rows(b[:, perm]), M, N, K1 + K2, za, zb)
    assert (C == Cp).all()


def test_range_constants_printed_in_the_paper():
    pc = paper_constants()
    assert pc["max_product"] == 15 * 15
    # all-15 operands, zero points 0: every output is 225 * K
    for K in (1, pc["depth_bound_signed16"], pc["depth_bound_unsigned16"], 1000):
        P = oracle.pack_rows(np.full((3, K), 15, np.uint8))
        C = oracle.gemm(P, P, 3, 3, K, 0, 0)
        assert (C == pc["max_product"] * K).all()
    D16 = pc["depth_bound_signed16"]
    assert pc["max_product"] * D16 <= 2 ** 15 - 1 < pc["max_product"] * (D16 + 1)
    U16 = pc["depth_bound_unsigned16"]
    assert pc["max_product"] * U16 <= 2 ** 16 - 1 < pc["max_product"] * (U16 + 1)
    # Eq. 5: channels for 1x1 / 3x3 / 5x5 kernels; depth D = kh*kw*c
    assert D16 // 1 == pc["channels_1x1"]
    assert D16 // 9 == pc["channels_3x3"]
    assert D16 // 25 == pc["channels_5x5"]
    for k, c in ((1, pc["channels_1x1"]), (3, pc["channels_3x3"]), (5, pc["channels_5x5"])):
        d = ConvDesc(1, 7, 7, c, 2, k, k)
        assert oracle.conv_gemm_shape(d)[1] == k * k * c <= D16
    # op-count convention: 24 widening multiply-accumulates of 8 lanes, times 2 depth steps
    assert pc["big_kernel_muladds"] == 24 * 8 * 2


def test_worst_case_correction_magnitude_c5_zero_points():
    # za = 0, zb = 15: C = sum a (b - 15) lies in [-225 K, 0]
    K = 16384
    a = np.full((1, K), 15, np.uint8)
    b = np.zeros((1, K), np.uint8)
    C = oracle.gemm(oracle.pack_rows(a), oracle.pack_rows(b), 1, 1, K, 0, 15)
    assert C[0, 0] == -225 * K == -3686400
    rng = np.random.default_rng(9)
    a, b = rand_vals(rng, 4, K), rand_vals(rng, 4, K)
    C = oracle.gemm(oracle.pack_rows(a), oracle.pack_rows(b), 4, 4, K, 0, 15)
    assert (C <= 0).all() and (C >= -225 * K).all()


def test_odd_depth_pad_nibble_contract():
    a = np.array([[1, 2, 3]], np.uint8)
    A = oracle.pack_rows(a)
    assert oracle.gemm(A, A, 1, 1, 3, 0, 0)[0, 0] == 14
    A_bad = A.copy()
    A_bad[0, 1] |= 0x50
    with pytest.raises(oracle.OracleError) as e:
        oracle.gemm(A_bad, A, 1, 1, 3, 0, 0)
    assert e.value.code == oracle.E_PAD


def test_pack_bt_is_a_transpose():
    rng = np.random.default_rng(10)
    for K, N in [(1, 2), (7, 5), (32, 64), (33, 17)]:
        b_kn = rng.integers(0, 16, (K, N), dtype=np.uint8)
        Bt = oracle.pack_bt(oracle.pack_rows(b_kn), K, N, (K + 1) // 2 + 2)
        assert (oracle.unpack_rows(Bt, K) == b_kn.T).all()
        assert (Bt[:, (K + 1) // 2:] == 0).all()
        if K & 1:
            assert (Bt[:, K // 2] >> 4 == 0).all()


# ---------------------------------------------------------------- requantization

@settings(max_examples=400, deadline=None)
@given(acc=st.integers(-2 ** 31, 2 ** 31 - 1), mult=st.integers(2 ** 30, 2 ** 31 - 1),
       shift=st.integers(0, 31), zo=st.integers(0, 15), lo=st.integers(0, 15), hi=st.integers(0, 15))
def test_requant_against_arbitrary_precision(acc, mult, shift, zo, lo, hi):
    lo, hi = min(lo, hi), max(lo, hi)
    t = 31 + shift
    q = (acc * mult + (1 << (t - 1))) >> t       # Python ints: exact, >> floors
    want = min(max(q + zo, lo), hi)
    assert oracle.requant_value(acc, Requant(mult, shift, zo, lo, hi)) == want


def test_requant_power_of_two_multiplier_is_textbook_rounding():
    # mult = 2^30 -> q = floor(acc / 2^(shift+1) + 1/2)
    from fractions import Fraction
    import math
    for shift in (0, 1, 5, 8, 16):
        rq = Requant(1 << 30, shift, 0, 0, 15)
        for acc in list(range(-40, 41)) + [2 ** shift, -(2 ** shift), 3 * 2 ** shift, 5 * 2 ** shift - 1]:
            want = math.floor(Fraction(acc, 2 ** (shift + 1)) + Fraction(1, 2))
            assert oracle.requant_value(acc, rq) == min(max(want, 0), 15)


def test_requant_ties_go_toward_plus_infinity():
    # acc / 2^(shift+1) = +-1/2 exactly
    for shift in (3, 8):
        rq_pos = Requant(1 << 30, shift, 0, 0, 15)
        assert oracle.requant_value(2 ** shift, rq_pos) == 1           #  0.5 ->  1
        rq_neg = Requant(1 << 30, shift, 8, 0, 15)
        assert oracle.requant_value(-(2 ** shift), rq_neg) == 8        # -0.5 ->  0
        assert oracle.requant_value(-3 * 2 ** shift, rq_neg) == 7      # -1.5 -> -1
        assert oracle.requant_value(5 * 2 ** shift, rq_neg) == 11      #  2.5 ->  3


def test_requant_monotone_and_saturating():
    rq = Requant((1 << 30) + 12345, 9, 3, 3, 12)
    prev = -1
    for acc in range(-30000, 30000, 7):
        y = oracle.requant_value(acc, rq)
        assert 3 <= y <= 12 and y >= prev
        prev = y
    assert oracle.requant_value(-2 ** 31, rq) == 3
    assert oracle.requant_value(2 ** 31 - 1, rq) == 12


def test_requant_matrix_packs_along_n_and_adds_bias():
    C = np.array([[0, 1024, 2048, 4096], [-1024, 512, 511, 100000]], np.int32)
    rq = Requant(1 << 30, 9, 0, 0, 15)            # divide by 1024, round half up
    Cq = oracle.requant_matrix(C, None, rq)
    assert oracle.unpack_rows(Cq, 4).tolist() == [[0, 1, 2, 4], [0, 1, 0, 15]]
    assert Cq.tolist() == [[0x10, 0x42], [0x10, 0xF0]]
    bias = np.array([1024, -1024, 1, 0], np.int32)
    Cq = oracle.requant_matrix(C, bias, rq)
    assert oracle.unpack_rows(Cq, 4).tolist() == [[1, 0, 2, 4], [0, 0, 1, 15]]


def test_gemm_requant_is_gemm_then_requant():
    c = wl.gemm_case("t", 37, 18, 75, seed=11, with_bias=True)
    rq = Requant(c.mult, 4, 2, 2, 15)
    C = oracle.gemm(c.A, c.Bt, c.M, c.N, c.K, c.za, c.zb)
    want = oracle.requant_matrix(C, c.bias, rq)
    got = oracle.gemm_requant(c.A, c.Bt, c.M, c.N, c.K, c.za, c.zb, c.bias, rq)
    assert (got == want).all()
    assert len(np.unique(oracle.unpack_rows(got, c.N))) > 4   # not degenerate


# ---------------------------------------------------------------- convolution

CONVS = [
    ConvDesc(2, 6, 7, 3, 4, 3, 3, 1, 1, 1, 1),
    ConvDesc(1, 9, 8, 1, 2, 3, 3, 2, 2, 1, 1),      # single channel: nibble-granular pixels
    ConvDesc(2, 33, 25, 1, 8, 5, 5, 1, 1, 0, 0),    # Table II layer 1 shape, no padding
    ConvDesc(1, 10, 11, 8, 16, 3, 3, 2, 1, 0, 1),   # mixed strides / pads
    ConvDesc(3, 5, 5, 16, 6, 1, 1, 1, 1, 0, 0),
    ConvDesc(1, 4, 4, 2, 2, 3, 3, 1, 1, 2, 2),      # pad wider than needed
]


def conv_inputs(d, seed):
    rng = np.random.default_rng(seed)
    x = rng.integers(0, 16, (d.N, d.H, d.W, d.C), dtype=np.uint8)
    w = rng.integers(0, 16, (d.OC, d.KH, d.KW, d.C), dtype=np.uint8)
    return x, w, oracle.pack(x.reshape(-1)), oracle.pack_rows(w.reshape(d.OC, -1))


@pytest.mark.parametrize("d", CONVS)
def test_conv_direct_matches_float64_library_convolution(d):
    import torch
    x, w, X, Wt = conv_inputs(d, 20)
    za, zb = 6, 11
    Y = oracle.conv2d_direct(X, Wt, d, za, zb)
    # out-of-image taps read the zero point, i.e. contribute (za - za) = 0: zero padding of x - za
    xs = torch.from_numpy(x.astype(np.float64) - za).permute(0, 3, 1, 2)
    ws = torch.from_numpy(w.astype(np.float64) - zb).permute(0, 3, 1, 2)
    ref = torch.nn.functional.conv2d(xs, ws, stride=(d.stride_h, d.stride_w),
                                     padding=(d.pad_h, d.pad_w)).permute(0, 2, 3, 1)
    assert Y.shape == tuple(ref.shape)
    assert (Y == ref.numpy().astype(np.int64)).all()


@pytest.mark.parametrize("d", CONVS)
def test_im2col_then_gemm_equals_direct_convolution(d):
    x, w, X, Wt = conv_inputs(d, 21)
    za, zb = 9, 4
    M, K, OH, OW = oracle.conv_gemm_shape(d)
    lda = (K + 1) // 2 + 5
    A, ra = oracle.im2col(X, d, za, lda)
    assert (A[:, (K + 1) // 2:] == 0).all()
    if K & 1:
        assert (A[:, K // 2] >> 4 == 0).all()
    assert (ra == oracle.unpack_rows(A, K).sum(1, dtype=np.int64)).all()
    C = oracle.gemm(A, Wt, M, d.OC, K, za, zb)
    Y = oracle.conv2d_direct(X, Wt, d, za, zb)
    assert (C.reshape(d.N, OH, OW, d.OC) == Y).all()


def test_im2col_hand_written_example():
    # 1 x 2 x 2 x 1 image [[1,2],[3,4]], 3x3 window, pad 1, stride 1, zero point 9.
    X = oracle.pack(np.array([1, 2, 3, 4], np.uint8))
    d = ConvDesc(1, 2, 2, 1, 1, 3, 3, 1, 1, 1, 1)
    A, ra = oracle.im2col(X, d, 9)
    rows = oracle.unpack_rows(A, 9).tolist()
    assert rows[0] == [9, 9, 9, 9, 1, 2, 9, 3, 4]       # output (0,0): top and left taps outside
    assert rows[3] == [1, 2, 9, 3, 4, 9, 9, 9, 9]       # output (1,1)
    assert ra.tolist()[0] == 9 * 5 + 10


def test_pointwise_convolution_is_a_gemm():
    d = ConvDesc(2, 5, 3, 16, 6, 1, 1)
    x, w, X, Wt = conv_inputs(d, 22)
    Y = oracle.conv2d_direct(X, Wt, d, 3, 12)
    A = X.reshape(d.N * d.H * d.W, d.C // 2)
    C = oracle.gemm(A, Wt, A.shape[0], d.OC, d.C, 3, 12)
    assert (Y.reshape(-1, d.OC) == C).all()


def test_padding_equals_explicit_zero_point_border():
    d = ConvDesc(1, 6, 5, 4, 4, 3, 3, 2, 1, 1, 1)
    x, w, X, Wt = conv_inputs(d, 23)
    za, zb = 13, 2
    Y = oracle.conv2d_direct(X, Wt, d, za, zb)
    xb = np.full((d.N, d.H + 2, d.W + 2, d.C), za, np.uint8)
    xb[:, 1:-1, 1:-1, :] = x
    d2 = ConvDesc(1, d.H + 2, d.W + 2, 4, 4, 3, 3, 2, 1, 0, 0)
    Y2 = oracle.conv2d_direct(oracle.pack(xb.reshape(-1)), Wt, d2, za, zb)
    assert (Y == Y2).all()


def test_conv2d_is_direct_plus_bias_plus_requant():
    d = ConvDesc(2, 7, 6, 8, 10, 3, 3, 2, 2, 1, 1)
    x, w, X, Wt = conv_inputs(d, 24)
    bias = np.arange(-5, 5, dtype=np.int32) * 100
    rq = Requant((1 << 30) + 99, 4, 5, 5, 15)
    Y32 = oracle.conv2d_direct(X, Wt, d, 7, 8)
    want = oracle.requant_matrix(Y32.reshape(-1, d.OC), bias, rq)
    got = oracle.conv2d(X, Wt, bias, d, 7, 8, rq)
    assert (got == want).all()


def test_table2_layer_sizes():
    pc = paper_constants()
    net = wl.paper_table2_net(batch=1)
    assert (net.layers[0].H, net.layers[0].W) == (pc["table2_input_h"], pc["table2_input_w"])
    params = sum(l.OC * l.K for l in net.layers)
    assert params == pc["table2_conv_params"]


def test_c4_chain_shapes():
    net = wl.c4(batch=2)
    assert [(l.M // 2, l.K, l.OC) for l in net.layers] == \
        [(48 * 48, 9, 8), (24 * 24, 72, 16), (12 * 12, 144, 32), (6 * 6, 288, 64), (1, 2304, 256)]
