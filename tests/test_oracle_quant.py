"""Pins for the oracle's quantiser, packing, integer GEMM and dequantisation (CPU only)."""
import os

import numpy as np
import pytest

from oracle import singlequant_oracle as ora
from paper_2511_22316_b200 import workloads as wl

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def _cases():
    out = []
    with open(os.path.join(GOLDEN, "quantiser_cases.txt")) as f:
        for line in f:
            line = line.strip()
            if line and not line.startswith("#"):
                a, b = line.split()
                out.append((float(a), int(b)))
    return out


# ---------------------------------------------------------------- Q_Delta (P10)
@pytest.mark.parametrize("decision", ["f64", "f32"])
@pytest.mark.parametrize("delta", [1.0, 0.25, 3.0])
def test_quantiser_hand_cases(decision, delta):
    """Each hand case z/Delta sits in a row whose absmax is 7*Delta, so Delta_t = Delta exactly
    (0.25, 1 and 3 are fp16 numbers and 7*Delta/7 is exact)."""
    cases = _cases()
    Z = np.array([[c[0] * delta, 7.0 * delta] for c in cases])
    codes, d = ora.quantize_rows(Z, decision)
    assert np.all(d == np.float16(delta))
    assert [int(x) for x in codes[:, 0]] == [c[1] for c in cases]
    assert np.all(codes[:, 1] == 7)


@pytest.mark.parametrize("decision", ["f64", "f32"])
def test_quantiser_properties(decision):
    rng = np.random.default_rng(0)
    Z = rng.standard_normal((64, 256)) * rng.uniform(0.01, 50, size=(64, 1))
    Z[5] = 0.0
    codes, d = ora.quantize_rows(Z, decision)
    assert codes.dtype == np.int8 and d.dtype == np.float16
    assert codes.min() >= -8 and codes.max() <= 7
    assert np.all(codes[5] == 0) and d[5] == 0
    dd = d.astype(np.float64)
    amax = np.max(np.abs(Z), axis=1)
    # Delta is amax/7 rounded to fp16: relative error at most 2^-11
    nz = amax > 0
    assert np.all(np.abs(dd[nz] - amax[nz] / 7) <= amax[nz] / 7 * 2.0 ** -11)
    # |z - Q(z)| <= Delta/2 wherever the clamp is not active (fp16 rounding of Delta can push
    # the absmax entry itself just past 7.5 only if Delta shrank by > 6%; it cannot)
    err = np.abs(Z - codes * dd[:, None])
    assert np.all(err[nz] <= dd[nz, None] * (0.5 + 1e-6))
    # every non-zero row uses the full range: its absmax entry has a code of magnitude 7
    assert np.all(np.max(np.abs(codes[nz].astype(int)), axis=1) == 7)


def test_quantiser_f32_and_f64_decisions_agree_off_boundaries():
    w = wl.small("q", 32, 16, 32, 8, 7)
    X = wl.make_activations(w)
    R1, R2 = ora.build_rotation(X.astype(np.float32), w.n1, w.n2)
    Z = ora.rotate(X, R1, R2)
    c64, d64 = ora.quantize_rows(Z, "f64")
    c32, d32 = ora.quantize_rows(Z, "f32")
    assert np.mean(d64 != d32) <= 0.05
    diff = np.abs(c64.astype(int) - c32.astype(int))
    assert diff.max() <= 1
    assert np.mean(diff != 0) <= 1e-3


def test_half_goes_up_not_to_even():
    # 2.5 -> 3 and -2.5 -> -2 under floor(x + 1/2); round-half-even would give 2 and -2
    Z = np.array([[2.5, -2.5, 7.0]])
    codes, _ = ora.quantize_rows(Z, "f64")
    assert list(codes[0]) == [3, -2, 7]


# ---------------------------------------------------------------- packing (P10)
def test_pack_unpack_all_bytes():
    packed = np.arange(256, dtype=np.uint8).reshape(1, 256)
    codes = ora.unpack_int4(packed)
    assert codes.shape == (1, 512)
    assert codes.min() == -8 and codes.max() == 7
    assert np.array_equal(ora.pack_int4(codes), packed)
    # the low nibble is the even channel, two's complement
    assert list(ora.unpack_int4(np.array([[0x7F]], np.uint8))[0]) == [-1, 7]
    assert list(ora.unpack_int4(np.array([[0x80]], np.uint8))[0]) == [0, -8]
    assert ora.pack_int4(np.array([[-8, 7]], np.int8))[0, 0] == 0x78
    assert ora.pack_int4(np.array([[1, -2]], np.int8))[0, 0] == 0xE1


def test_pack_round_trip_random():
    rng = np.random.default_rng(1)
    codes = rng.integers(-8, 8, size=(7, 64)).astype(np.int8)
    assert np.array_equal(ora.unpack_int4(ora.pack_int4(codes)), codes)


# ---------------------------------------------------------------- integer GEMM (P12)
def test_gemm_i32_against_python_loops():
    rng = np.random.default_rng(2)
    for (T, C, K) in [(1, 1, 2), (3, 5, 8), (4, 7, 34)]:
        Xc = rng.integers(-8, 8, size=(T, K)).astype(np.int8)
        Wc = rng.integers(-8, 8, size=(C, K)).astype(np.int8)
        a = ora.gemm_i32(Xc, Wc)
        assert a.dtype == np.int32
        assert np.array_equal(a, ora.gemm_i32_loops(Xc, Wc))
        assert np.array_equal(a, Xc.astype(np.int64) @ Wc.astype(np.int64).T)


def test_gemm_i32_closed_forms():
    K = 28672
    ones = np.ones((2, K), np.int8)
    assert np.all(ora.gemm_i32(ones, ones) == K)
    lo = np.full((1, K), -8, np.int8)
    assert ora.gemm_i32(lo, lo)[0, 0] == 64 * K                   # 1,835,008 fits in int32
    hi = np.full((1, K), 7, np.int8)
    assert ora.gemm_i32(lo, hi)[0, 0] == -56 * K
    # not symmetric in its arguments' roles: rows of the second operand are output channels
    A = np.array([[1, 2]], np.int8)
    B = np.array([[3, 4], [5, 6], [-1, 0]], np.int8)
    assert ora.gemm_i32(A, B).tolist() == [[11, 17, -1]]


# ---------------------------------------------------------------- dequant + whole layer (P13)
def test_dequant():
    acc = np.array([[10, -3], [7, 0]], np.int32)
    sx = np.array([0.5, 2.0], np.float16)
    sw = np.array([0.25, 3.0], np.float16)
    y = ora.dequant(acc, sx, sw)
    assert y.dtype == np.float16
    assert y.tolist() == [[1.25, -4.5], [3.5, 0.0]]


def test_linear_on_grid_inputs_reduces_to_plain_matmul():
    """Identity rotation and inputs already on the INT4 grid: the quantiser is lossless, so the
    W4A4 layer must equal the float64 product X W^T up to the final fp16 rounding."""
    rng = np.random.default_rng(3)
    T, C, K = 9, 11, 64
    cx = rng.integers(-7, 8, size=(T, K))
    cw = rng.integers(-7, 8, size=(C, K))
    cx[:, 0] = 7
    cw[:, 1] = -7
    sx = 2.0 ** rng.integers(-6, 3, size=T)
    sw = 2.0 ** rng.integers(-9, -3, size=C)
    X = (cx * sx[:, None]).astype(np.float16)
    W = (cw * sw[:, None]).astype(np.float16)
    assert np.array_equal(X.astype(np.float64), cx * sx[:, None])
    Y = ora.linear(X, W, None, None)
    ref = ora.linear_fp(X, W)
    assert np.array_equal(Y, ref.astype(np.float16))
    Xq, dx, _ = ora.rotate_quant(X, None, None)
    assert np.array_equal(ora.unpack_int4(Xq), cx.astype(np.int8))
    assert np.array_equal(dx.astype(np.float64), sx)


def test_linear_with_rotation_beats_no_rotation_on_outlier_inputs():
    """Reported sanity of the method (ablation paragraph): with massive outliers the rotated
    W4A4 layer is closer to the full-precision layer than the unrotated one."""
    w = wl.TINY
    X, W = wl.make_layer(w)
    Y = ora.linear_fp(X, W)
    R1, R2 = ora.build_rotation(X.astype(np.float32), w.n1, w.n2)
    e_rot = np.linalg.norm(ora.linear(X, W, R1, R2).astype(np.float64) - Y) / np.linalg.norm(Y)
    e_none = np.linalg.norm(ora.linear(X, W, None, None).astype(np.float64) - Y) / np.linalg.norm(Y)
    assert e_rot < e_none
    assert e_rot < 0.5
