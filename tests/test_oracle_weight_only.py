"""Pins for the oracle's weight-only variant (Appendix "Weight-only Quantization", Table "wquant")
and for the grouped form of the layer: hand-worked values, closed forms, bounds and special cases
that reduce to a plain matrix product."""
import numpy as np
import pytest

from oracle import singlequant_oracle as ora


def test_three_bit_codes_of_a_hand_worked_row():
    # amax = 3, 2^(3-1) - 1 = 3 -> Delta = 1; floor(z + 1/2): 0 -> 0, 1.5 -> 2, -3 -> -3, 3 -> 3,
    # -0.5 -> 0 (floor(0) = 0), -0.51 -> -1, 2.49 -> 2, -2.5 -> -2
    Z = np.array([[0.0, 1.5, -3.0, 3.0, -0.5, -0.51, 2.49, -2.5]])
    codes, delta = ora.quantize_rows_bits(Z, 3)
    assert float(delta[0]) == 1.0
    assert codes.tolist() == [[0, 2, -3, 3, 0, -1, 2, -2]]
    # 4 bits on the same row: Delta = fp16(3/7) = 0.428466796875 exactly (fp16 has 11 significant bits)
    codes4, delta4 = ora.quantize_rows_bits(Z, 4)
    assert float(delta4[0]) == 0.428466796875
    # 1.5 / 0.4284668 = 3.5008 -> floor(4.0008) = 4; 3 / Delta = 7.0016 -> floor(7.5016) = 7;
    # -0.5 / Delta = -1.1669 -> floor(-0.6669) = -1; 2.49 / Delta = 5.811 -> 6; -2.5 / Delta = -5.835 -> -6
    assert codes4.tolist() == [[0, 4, -7, 7, -1, -1, 6, -6]]


def test_clamp_is_reached_only_through_the_rounding_of_delta():
    # amax / 3 = 1.00048828125 lies halfway between the fp16 neighbours 1.0 and 1.0009765625 and rounds
    # to even, 1.0: Delta is smaller than amax / 3 and the extreme entries give floor(3.00146 + 0.5) = 3.
    Z = np.array([[3.00146484375, -3.00146484375, 1.0]])
    codes, delta = ora.quantize_rows_bits(Z, 3)
    assert float(delta[0]) == 1.0 and codes.tolist() == [[3, -3, 1]]
    # amax / 3 = 1.16666.. rounds UP to fp16 1.1669921875: 3.5 / Delta = 2.9991 -> floor(3.4991) = 3
    Z2 = np.array([[3.5, -3.5]])
    c2, d2 = ora.quantize_rows_bits(Z2, 3)
    assert float(d2[0]) == 1.1669921875 and c2.tolist() == [[3, -3]]
    # codes stay inside the b-bit range on rows of any magnitude
    rng = np.random.default_rng(5)
    Z3 = rng.standard_normal((64, 256)) * rng.uniform(1e-3, 1e3, size=(64, 1))
    c3, _ = ora.quantize_rows_bits(Z3, 3)
    assert c3.min() >= -4 and c3.max() <= 3
    c4, _ = ora.quantize_rows_bits(Z3, 4)
    assert c4.min() >= -8 and c4.max() <= 7


@pytest.mark.parametrize("decision", ["f64", "f32"])
def test_four_bits_is_the_w4a4_quantiser(decision):
    rng = np.random.default_rng(11)
    Z = rng.standard_normal((40, 96)) * rng.uniform(1e-4, 1e4, size=(40, 1))
    Z[3] = 0.0
    a_codes, a_delta = ora.quantize_rows_bits(Z, 4, decision)
    b_codes, b_delta = ora.quantize_rows(Z, decision)
    assert np.array_equal(a_codes, b_codes)
    assert np.array_equal(a_delta.view(np.uint16), b_delta.view(np.uint16))


@pytest.mark.parametrize("bits", [3, 4])
def test_reconstruction_error_is_at_most_half_a_step(bits):
    rng = np.random.default_rng(12 + bits)
    Z = rng.standard_normal((32, 512)) * rng.uniform(0.01, 50.0, size=(32, 1))
    codes, delta = ora.quantize_rows_bits(Z, bits)
    d = delta.astype(np.float64)[:, None]
    qmax = 2 ** (bits - 1) - 1
    inside = np.abs(Z) <= (qmax + 0.5) * d            # not clamped
    err = np.abs(codes * d - Z)
    assert np.all(err[inside] <= 0.5 * d.repeat(Z.shape[1], 1)[inside] * (1 + 1e-12))
    # entries beyond the last level (possible only because fp16(amax/qmax) may round down) miss by
    # at most half a step plus that rounding: amax - qmax * Delta <= qmax * Delta * 2^-11
    assert np.all(err <= 0.5 * d + qmax * d * 2.0 ** -11 + 1e-300)


def test_interleaved_storage_order_by_hand():
    # channels 0..7 with codes 0..7: positions hold channels (0, 2, 4, 6, 1, 3, 5, 7) -> the word reads
    # 0x75316420, little-endian bytes 20 64 31 75
    codes = np.arange(8, dtype=np.int8)[None, :]
    packed = ora.pack_int4_interleaved(codes)
    assert packed.tolist() == [[0x20, 0x64, 0x31, 0x75]]
    # negative codes are two's-complement nibbles: -1 -> 0xF, -8 -> 0x8
    codes = np.array([[-1, -8, 0, 0, 0, 0, 0, 7]], dtype=np.int8)
    packed = ora.pack_int4_interleaved(codes)
    word = int.from_bytes(bytes(packed[0].tolist()), "little")
    # position 0 = channel 0 (-1 -> F), position 4 = channel 1 (-8 -> 8), position 7 = channel 7 (7)
    assert word == 0x7008000F


def test_interleaved_order_gives_channel_pairs_by_one_shift_and_mask():
    rng = np.random.default_rng(3)
    codes = rng.integers(-8, 8, size=(5, 64), dtype=np.int8)
    packed = ora.pack_int4_interleaved(codes)
    for r in range(5):
        for g in range(8):
            word = int.from_bytes(bytes(packed[r, 4 * g:4 * g + 4].tolist()), "little")
            for s in range(4):
                pair = (word >> (4 * s)) & 0x000F000F
                lo, hi = pair & 0xF, pair >> 16
                assert lo == int(codes[r, 8 * g + 2 * s]) & 15
                assert hi == int(codes[r, 8 * g + 2 * s + 1]) & 15
    assert np.array_equal(ora.unpack_int4_interleaved(packed), codes)


@pytest.mark.parametrize("bits", [3, 4])
def test_lossless_weights_give_the_plain_product(bits):
    """Identity rotation and weights that are integer multiples of a power-of-two step with the
    extreme level present: the codes are the integers, Delta is the step, and the layer is the
    fp16-rounded plain product of the fp16 activations with W."""
    rng = np.random.default_rng(20 + bits)
    qmax = 2 ** (bits - 1) - 1
    C, n, T = 24, 64, 9
    ints = rng.integers(-qmax, qmax + 1, size=(C, n))
    ints[:, 0] = qmax
    step = 2.0 ** rng.integers(-6, 3, size=(C, 1))
    W = (ints * step).astype(np.float16)
    X = rng.standard_normal((T, n)).astype(np.float16)
    Y = ora.linear_wo(X, W, None, None, bits)
    expect = (X.astype(np.float64) @ W.astype(np.float64).T).astype(np.float16)
    assert np.array_equal(Y.view(np.uint16), expect.view(np.uint16))
    Wq, sw, _ = ora.pack_weight_wo(W, None, None, bits)
    assert np.array_equal(ora.unpack_int4_interleaved(Wq), ints.astype(np.int8))
    assert np.array_equal(sw.astype(np.float64), step[:, 0])


@pytest.mark.parametrize("bits", [3, 4])
def test_weight_only_layer_is_within_the_quantisation_bound_of_the_exact_layer(bits):
    """(X R)(R^T W^T) = X W^T before quantisation; afterwards every output misses by at most
    ||z||_1 * Delta_c / 2 (half a step per weight) plus the fp16 roundings of z and of the result."""
    rng = np.random.default_rng(30 + bits)
    n1, n2, T, C = 8, 16, 12, 20
    X = rng.standard_normal((T, n1 * n2)).astype(np.float16)
    W = (0.02 * rng.standard_normal((C, n1 * n2))).astype(np.float16)
    R1, R2 = ora.build_rotation(X.astype(np.float32), n1, n2)
    Y = ora.linear_wo(X, W, R1, R2, bits).astype(np.float64)
    exact = ora.linear_fp(X, W)
    Z = ora.rotate(X, R1, R2)
    _, sw, Zw = ora.pack_weight_wo(W, R1, R2, bits)
    qmax = 2 ** (bits - 1) - 1
    half_step = 0.5 * sw.astype(np.float64) + qmax * sw.astype(np.float64) * 2.0 ** -11
    bound = np.abs(Z).sum(axis=1)[:, None] * half_step[None, :]
    bound += 2.0 ** -11 * np.abs(Z).sum(axis=1)[:, None] * np.abs(Zw).max(axis=1)[None, :]      # fp16(z)
    bound += 2.0 ** -10 * np.abs(exact) + 1e-6                                                  # fp16(y), fp32 factors
    assert np.all(np.abs(Y - exact) <= bound)
    # and the error is not trivially zero: the bound is exercised to within two orders of magnitude
    assert np.max(np.abs(Y - exact) / bound) > 0.01


def test_three_bits_lose_more_than_four():
    rng = np.random.default_rng(41)
    n1, n2, T, C = 8, 16, 32, 48
    X = rng.standard_normal((T, n1 * n2)).astype(np.float16)
    W = (0.02 * rng.standard_normal((C, n1 * n2))).astype(np.float16)
    R1, R2 = ora.build_rotation(X.astype(np.float32), n1, n2)
    exact = ora.linear_fp(X, W)
    e4 = np.linalg.norm(ora.linear_wo(X, W, R1, R2, 4).astype(np.float64) - exact)
    e3 = np.linalg.norm(ora.linear_wo(X, W, R1, R2, 3).astype(np.float64) - exact)
    # uniform rounding error scales with the step: 7/3 = 2.33 between the two (within a broad band)
    assert 1.6 < e3 / e4 < 3.2


def test_rotate_f16_is_the_rounded_rotation_and_keeps_norms():
    rng = np.random.default_rng(42)
    n1, n2 = 4, 8
    X = rng.standard_normal((6, n1 * n2)).astype(np.float16)
    R1, R2 = ora.build_rotation(X.astype(np.float32), n1, n2)
    Z16 = ora.rotate_f16(X, R1, R2)
    assert Z16.dtype == np.float16
    dense = X.astype(np.float64) @ ora.kron_dense(R1, R2)
    assert np.array_equal(Z16.view(np.uint16), dense.astype(np.float16).view(np.uint16)) or \
        np.max(np.abs(Z16.astype(np.float64) - dense)) <= 2.0 ** -11 * np.max(np.abs(dense)) * 1.01
    assert np.allclose(np.linalg.norm(Z16.astype(np.float64), axis=1), np.linalg.norm(X.astype(np.float64), axis=1),
                       rtol=2e-3)
    assert np.array_equal(ora.rotate_f16(X, None, None).view(np.uint16), X.view(np.uint16))


def test_grouped_layer_is_the_per_expert_layer():
    rng = np.random.default_rng(50)
    n1, n2, C = 4, 8, 10
    n = n1 * n2
    counts = [5, 0, 3, 1]
    offsets = np.concatenate([[0], np.cumsum(counts)])
    X = rng.standard_normal((offsets[-1], n)).astype(np.float16)
    Ws = [(0.05 * rng.standard_normal((C, n))).astype(np.float16) for _ in counts]
    rots = []
    for e in range(len(counts)):
        cal = rng.standard_normal((16, n)).astype(np.float32)
        rots.append(ora.build_rotation(cal, n1, n2, O=ora.haar_orthogonal(n1 - 2, np.random.default_rng(e))))
    Y = ora.linear_grouped(X, offsets, Ws, rots)
    assert Y.shape == (9, C)
    # one expert holding every token is the plain layer
    Y1 = ora.linear_grouped(X, [0, 9], [Ws[0]], [rots[0]])
    assert np.array_equal(Y1.view(np.uint16), ora.linear(X, Ws[0], *rots[0]).view(np.uint16))
    # a token's output depends on its own expert only: moving the other experts' tokens away changes nothing
    a, b = offsets[2], offsets[3]
    alone = ora.linear(X[a:b], Ws[2], *rots[2])
    assert np.array_equal(Y[a:b].view(np.uint16), alone.view(np.uint16))
    # swapping two experts' weights changes exactly those experts' rows
    Ws2 = [Ws[2], Ws[1], Ws[0], Ws[3]]
    Y2 = ora.linear_grouped(X, offsets, Ws2, rots)
    assert np.array_equal(Y2[offsets[3]:].view(np.uint16), Y[offsets[3]:].view(np.uint16))
    assert not np.array_equal(Y2[:offsets[1]].view(np.uint16), Y[:offsets[1]].view(np.uint16))
    # every row is within the W4A4 tolerance of the exact per-expert product
    for e, (a, b) in enumerate(zip(offsets[:-1], offsets[1:])):
        if b > a:
            exact = ora.linear_fp(X[a:b], Ws[e])
            assert np.linalg.norm(Y[a:b].astype(np.float64) - exact) <= 0.35 * np.linalg.norm(exact)
