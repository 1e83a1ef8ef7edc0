"""Pins of the float-boundary oracle (oracle/qfloat.py): Eq. 1's quantizer under the reading
stated there, and Eq. 4's scale-back.  Each test fixes the oracle to something other than
itself: hand-computed codes, closed forms, exact rational arithmetic, invariants."""
from fractions import Fraction

import numpy as np
import pytest

import oracle


def unpack(Q, cols):
    lo, hi = Q & 0x0F, Q >> 4
    out = np.empty((Q.shape[0], 2 * Q.shape[1]), dtype=np.int64)
    out[:, 0::2], out[:, 1::2] = lo, hi
    return out[:, :cols]


def test_lattice_values_get_their_own_index():
    # w = 0.25 * (j - 4), j = 0..15: min -1, max 2.75, s = 3.75 / 15 = 0.25, z_q = 4, code = j
    X = (0.25 * (np.arange(16) - 4)).astype(np.float32).reshape(2, 8)
    s, z = oracle.quant_params(X)
    assert s == np.float32(0.25) and z == 4
    Q = oracle.quantize(X, s, z)
    assert Q.tolist() == [[0x10, 0x32, 0x54, 0x76], [0x98, 0xBA, 0xDC, 0xFE]]


def test_hand_computed_codes_off_the_lattice():
    # s = 0.25, z_q = 4 as above; floor(0.45/0.25) = 1, floor(0.3/0.25) = 1, floor(-0.1/0.25) = -1
    X = np.array([[-1.0, 2.75, 0.45, 0.3, -0.1]], dtype=np.float32)
    s, z = oracle.quant_params(X)
    assert (s, z) == (np.float32(0.25), 4)
    assert unpack(oracle.quantize(X, s, z), 5).tolist() == [[0, 15, 5, 5, 3]]
    # odd row: the last high nibble is 0
    assert oracle.quantize(X, s, z)[0, 2] == 0x03


def test_non_negative_data_has_zero_point_zero():
    # Section III-A: z = 0 for non-negative data; the maximum maps to the top code
    X = np.array([[0.5, 3.0, 1.5, 6.0]], dtype=np.float32)
    s, z = oracle.quant_params(X)
    assert z == 0 and s == np.float32(6.0) / np.float32(15)
    assert unpack(oracle.quantize(X, s, z), 4).tolist() == [[1, 7, 3, 15]]


def test_all_negative_data_puts_zero_at_the_top_code():
    X = np.array([[-7.5, -0.5, -3.0, -0.25]], dtype=np.float32)
    s, z = oracle.quant_params(X)                     # max(max, 0) = 0: s = 7.5 / 15 = 0.5
    assert (s, z) == (np.float32(0.5), 15)
    assert unpack(oracle.quantize(X, s, z), 4).tolist() == [[0, 14, 9, 14]]
    assert unpack(oracle.quantize(np.zeros((1, 2), np.float32), s, z), 2).tolist() == [[15, 15]]


def test_all_zero_tensor():
    s, z = oracle.quant_params(np.zeros((3, 4), np.float32))
    assert (s, z) == (np.float32(1), 0)
    assert not oracle.quantize(np.zeros((3, 4), np.float32), s, z).any()


@pytest.mark.parametrize("seed", range(6))
def test_codes_against_exact_rational_arithmetic(seed):
    rng = np.random.default_rng(seed)
    X = (rng.standard_normal((7, 33)) * rng.uniform(0.01, 50)).astype(np.float32)
    if seed % 3 == 1:
        X = np.abs(X)
    s, z = oracle.quant_params(X)
    # scale and zero point from exact rationals of the float32 inputs, rounded once where Eq. 1 divides
    lo = min(Fraction(float(X.min())), Fraction(0))
    hi = max(Fraction(float(X.max())), Fraction(0))
    exact_s = (hi - lo) / 15
    assert abs(Fraction(float(s)) - exact_s) <= exact_s / (1 << 22)      # two float32 roundings
    assert z == min(max(-((lo / Fraction(float(s))).__floor__()), 0), 15) or \
        abs(lo / Fraction(float(s)) - round(lo / Fraction(float(s)))) < Fraction(1, 1 << 18)
    got = unpack(oracle.quantize(X, s, z), 33)
    fs = Fraction(float(s))
    for (i, j), w in np.ndenumerate(X):
        q = Fraction(float(w)) / fs                    # the exact quotient
        exact = min(max(q.__floor__() + z, 0), 15)
        if abs(q - round(q)) > Fraction(1, 1 << 18) * max(1, abs(q)):
            assert got[i, j] == exact                  # away from an integer boundary: no freedom
        else:
            assert abs(int(got[i, j]) - exact) <= 1    # float32 division may round across it


def test_reconstruction_error_is_below_one_step():
    rng = np.random.default_rng(11)
    X = rng.uniform(-3, 9, size=(5, 64)).astype(np.float32)
    s, z = oracle.quant_params(X)
    codes = unpack(oracle.quantize(X, s, z), 64)
    err = X.astype(np.float64) - float(s) * (codes - z)
    assert (err > -1e-5).all() and (err < float(s) * (1 + 1e-5)).all()     # floor: 0 <= err < s
    assert codes.min() == 0 and codes.max() == 15


def test_monotone_and_pitch_padding():
    X = np.sort(np.random.default_rng(3).uniform(-2, 2, size=(1, 101)).astype(np.float32))
    s, z = oracle.quant_params(X)
    Q = oracle.quantize(X, s, z, ldq=64)
    assert Q.shape == (1, 64) and not Q[:, 51:].any()
    codes = unpack(Q, 101)
    assert (np.diff(codes[0]) >= 0).all()


def test_dequantize_examples():
    C = np.array([[3, -5, 0], [1 << 24, (1 << 24) + 1, -7]], dtype=np.int32)
    R = oracle.dequantize(C, 0.5)
    assert R.dtype == np.float32
    # 2^24 + 1 is not a float32: it rounds to 2^24 before the multiplication
    assert R.tolist() == [[1.5, -2.5, 0.0], [8388608.0, 8388608.0, -3.5]]


def test_quantize_then_scale_back_gives_the_lattice():
    # Eq. 2's reading of a code: s * (code - z_q)
    X = (0.25 * (np.arange(16) - 4)).astype(np.float32).reshape(1, 16)
    s, z = oracle.quant_params(X)
    codes = unpack(oracle.quantize(X, s, z), 16)
    assert (oracle.dequantize((codes - z).astype(np.int32), s) == X).all()
