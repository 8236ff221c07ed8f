"""GPU parity: every stage of the CUDA path, called through the C ABI, against the CPU oracle
on identical seeded inputs.  Tolerances:
  * rotated rows: relative Frobenius error and per-row max-norm error <= 1e-5 (fp32 vs float64);
  * INT4 codes: at most 1 LSB apart on <= 0.1% of the elements (rounding-boundary cases);
    steps equal except where the row absmax straddles an fp16 rounding boundary (<= 1 ulp);
  * GEMM accumulators: bit-exact int32 on identical codes;
  * fp16 outputs: relative Frobenius error <= 1e-2.
"""
import numpy as np
import pytest

from oracle import singlequant_oracle as ora
from paper_2511_22316_b200 import workloads as wl

from gpu_util import Guarded, dev, torch_mod

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def sq():
    from paper_2511_22316_b200 import binding, build
    build.build()
    binding.load()
    return binding


def _fp16_ulps_apart(a, b):
    ia = a.view(np.int16).astype(np.int32)
    ib = b.view(np.int16).astype(np.int32)
    return np.abs(ia - ib)


def run_rotate_quant(sq, rot, X, want_z=True):
    M, n = X.shape
    dX = dev(X)
    q = Guarded(M * n // 2)
    s = Guarded(M * 2)
    z = Guarded(M * n * 4) if want_z else None
    sq.sq_rotate_quant_act(rot, dX, M, q, s, z)
    torch_mod().cuda.synchronize()
    assert sq.sq_last_device_status() == sq.SQ_OK
    q.check(); s.check()
    if z is not None:
        z.check()
    return (q.numpy(np.uint8, (M, n // 2)), s.numpy(np.float16, (M,)),
            z.numpy(np.float32, (M, n)) if z is not None else None)


def check_rotate_quant(sq, X, R1, R2, rows=None, rot=None):
    """Compares the fused kernel with the oracle on the rows `rows` (default: all).  `rot`: the handle
    to run with (default: one made from the oracle's factors R1, R2)."""
    rot = sq.sq_rotation_from_factors(R1, R2) if rot is None else rot
    Xq, sx, Z = run_rotate_quant(sq, rot, X)
    sel = np.arange(X.shape[0]) if rows is None else np.asarray(rows)
    Zo = ora.rotate(X[sel], R1, R2)
    Zg = Z[sel].astype(np.float64)
    # step 1: rotated rows
    assert np.linalg.norm(Zg - Zo) <= 1e-5 * np.linalg.norm(Zo)
    rowmax = np.max(np.abs(Zo), axis=1)
    rowerr = np.max(np.abs(Zg - Zo), axis=1)
    assert np.all(rowerr <= 1e-5 * np.maximum(rowmax, 1e-30))
    # step 2: codes and steps, decision taken in fp32 on both sides
    co, do = ora.quantize_rows(Zo, "f32")
    cg = ora.unpack_int4(Xq[sel])
    ulps = _fp16_ulps_apart(sx[sel], do)
    assert ulps.max() <= 1
    assert np.count_nonzero(ulps) <= max(1, int(0.005 * len(sel)))
    diff = np.abs(cg.astype(np.int32) - co.astype(np.int32))
    assert diff.max() <= 1
    assert np.count_nonzero(diff) <= 1e-3 * diff.size
    # and against the paper's float64 form of the quantiser
    c64, _ = ora.quantize_rows(Zo, "f64")
    d64 = np.abs(cg.astype(np.int32) - c64.astype(np.int32))
    assert d64.max() <= 1 and np.count_nonzero(d64) <= 1e-3 * d64.size
    rot.close()
    return Xq, sx, Z


# ------------------------------------------------------------------ setup: sq_build_rotation
@pytest.mark.parametrize("w", [wl.TINY, wl.small("b1", 9, 12, 8, 8, 11), wl.small("b2", 4, 64, 64, 8, 12),
                               wl.small("b3", 3, 172, 64, 8, 13), wl.small("b4", 5, 3, 4, 8, 14)])
@pytest.mark.parametrize("flags", [7, 1, 2, 4, 0])
def test_build_rotation_matches_oracle(sq, w, flags):
    X = wl.make_activations(w).astype(np.float32)
    rng = np.random.default_rng(w.seed)
    O = ora.haar_orthogonal(w.n1 - 2, rng) if w.n1 > 2 else None
    R1o, R2o = ora.build_rotation(X, w.n1, w.n2, flags=flags, O=O)
    rot = sq.sq_build_rotation(X, w.n1, w.n2, flags=flags, O=O)
    assert rot.dims == (w.n1, w.n2)
    R1, R2 = rot.factors()
    assert np.max(np.abs(R1.astype(np.float64) - R1o)) <= 1e-6
    assert np.max(np.abs(R2.astype(np.float64) - R2o)) <= 1e-6
    rot.close()


@pytest.mark.parametrize("steps", [2, 5, 16])
def test_build_rotation_with_repeated_art_steps_matches_oracle(sq, steps):
    w = wl.small("arts", 6, 64, 64, 8, 17)
    X = wl.make_activations(w).astype(np.float32)
    O = ora.haar_orthogonal(w.n1 - 2, np.random.default_rng(5))
    R1o, R2o = ora.build_rotation(X, w.n1, w.n2, O=O, art_steps=steps)
    rot = sq.sq_build_rotation(X, w.n1, w.n2, flags=sq.SQ_ROT_DEFAULT | sq.SQ_ROT_ART_STEPS(steps), O=O)
    R1, R2 = rot.factors()
    assert np.max(np.abs(R1.astype(np.float64) - R1o)) <= 1e-6
    assert np.max(np.abs(R2.astype(np.float64) - R2o)) <= 1e-6
    one = sq.sq_build_rotation(X, w.n1, w.n2, O=O).factors()[0]
    assert not np.array_equal(one, R1)
    rot.close()


def test_build_rotation_own_generator_gives_orthogonal_factors(sq):
    w = wl.TINY
    X = wl.make_activations(w).astype(np.float32)
    for seed in (0, 1, 12345):
        rot = sq.sq_build_rotation(X, w.n1, w.n2, seed=seed)
        R1, R2 = (a.astype(np.float64) for a in rot.factors())
        assert np.allclose(R1.T @ R1, np.eye(w.n1), atol=1e-6)
        assert np.allclose(R2.T @ R2, np.eye(w.n2), atol=1e-6)
        Z = ora.rotate(X[:1], R1, R2)
        assert np.max(np.abs(Z)) < 800 / 2       # the massive outlier is smoothed
        rot.close()
    a = sq.sq_build_rotation(X, w.n1, w.n2, seed=5).factors()[0]
    b = sq.sq_build_rotation(X, w.n1, w.n2, seed=6).factors()[0]
    assert not np.array_equal(a, b)


# ------------------------------------------------------------------ steps 1+2
SMALL_ROT = [(2, 2, 1), (3, 4, 3), (5, 8, 2), (8, 2, 4), (12, 8, 5), (1, 8, 2), (7, 6, 3), (16, 32, 64),
             (20, 16, 9), (64, 64, 37), (172, 64, 5), (112, 128, 4), (64, 128, 6), (224, 128, 3), (256, 128, 2),
             # tensor-core kernel: 4, 2 and 1 tokens per accumulator, ragged n1, ragged token groups
             (8, 64, 9), (24, 64, 7), (32, 128, 5), (48, 64, 11), (100, 128, 3), (128, 64, 5), (128, 128, 3),
             (64, 64, 301),
             # CTA-pair tensor-core kernel (128 < n1 <= 256): 64- and 128-byte half tiles, ragged second block
             (129, 64, 3), (160, 64, 75), (172, 64, 9), (224, 128, 5), (256, 64, 4), (144, 128, 150)]


@pytest.mark.parametrize("n1,n2,M", SMALL_ROT)
def test_rotate_quant_small_and_ragged(sq, n1, n2, M):
    w = wl.small(f"r{n1}x{n2}", M, n1, n2, 8, seed=n1 * 7 + n2)
    X = wl.make_activations(w)
    if n2 & (n2 - 1) == 0:
        R1, R2 = ora.build_rotation(X.astype(np.float32), n1, n2, seed=1)
    else:
        R1, R2 = ora.build_rotation(X.astype(np.float32), n1, n2, flags=ora.ROT_ART | ora.ROT_URT, seed=1)
    check_rotate_quant(sq, X, R1, R2)


def test_rotate_quant_tiny_config(sq):
    w = wl.TINY
    X = wl.make_activations(w)
    R1, R2 = ora.build_rotation(X.astype(np.float32), w.n1, w.n2)
    check_rotate_quant(sq, X, R1, R2)


@pytest.mark.parametrize("w", [wl.L7B_QKVO, wl.L7B_DOWN, wl.decode_down(64), wl.decode_up(1), wl.decode_down(1)])
def test_rotate_quant_full_configs(sq, w):
    X = wl.make_activations(w)
    R1, R2 = ora.build_rotation(X.astype(np.float32), w.n1, w.n2)
    rng = np.random.default_rng(0)
    rows = np.unique(np.concatenate([[0, w.M - 1], rng.integers(0, w.M, size=min(w.M, 96))]))
    check_rotate_quant(sq, X, R1, R2, rows=rows)


@pytest.mark.parametrize("w", [wl.L70B_GATEUP, wl.L70B_DOWN])
def test_rotate_quant_70b_shapes_sampled_rows(sq, w):
    X = wl.make_activations(w)
    R1, R2 = ora.build_rotation(X.astype(np.float32), w.n1, w.n2)
    rng = np.random.default_rng(1)
    rows = np.unique(np.concatenate([[0, w.M - 1], rng.integers(0, w.M, size=32)]))
    check_rotate_quant(sq, X, R1, R2, rows=rows)


def test_rotate_quant_many_short_rows(sq):
    """More token rows than 16 bits can index, four tokens per accumulator, a ragged last group."""
    w = wl.small("many", 70001, 8, 64, 8, 77)
    X = wl.make_activations(w)
    R1, R2 = ora.build_rotation(X.astype(np.float32), w.n1, w.n2)
    rng = np.random.default_rng(2)
    rows = np.unique(np.concatenate([[0, 1, 2, 3, 65535, 65536, 69999, 70000], rng.integers(0, w.M, size=120)]))
    check_rotate_quant(sq, X, R1, R2, rows=rows)


def test_quantiser_is_bit_exact_under_identity_rotation(sq):
    """With R1 = R2 = I the rotated row equals the fp16 input exactly, so codes and steps must
    match the oracle's fp32-decision quantiser bit for bit (both the rotating kernel with
    identity factors and the no-handle weight path)."""
    w = wl.small("ident", 33, 16, 32, 8, 21)
    X = wl.make_activations(w)
    X[5] = 0                                  # all-zero row: step 0, codes 0
    X[6, :] = np.float16(6e-8)                # absmax/7 underflows fp16: step 0, codes 0
    co, do = ora.quantize_rows(X.astype(np.float32), "f32")
    rot = sq.sq_rotation_from_factors(np.eye(w.n1, dtype=np.float32), np.eye(w.n2, dtype=np.float32))
    Xq, sx, Z = run_rotate_quant(sq, rot, X)
    assert np.array_equal(Z, X.astype(np.float32))
    assert np.array_equal(sx.view(np.uint16), do.view(np.uint16))
    assert np.array_equal(ora.unpack_int4(Xq), co)
    assert sx[5] == 0 and not np.any(Xq[5])
    q = Guarded(X.shape[0] * w.n // 2)
    s = Guarded(X.shape[0] * 2)
    sq.sq_pack_weight(None, dev(X), X.shape[0], w.n, q, s)
    torch_mod().cuda.synchronize()
    q.check(); s.check()
    assert np.array_equal(q.numpy(np.uint8, Xq.shape), Xq)
    assert np.array_equal(s.numpy(np.float16, sx.shape).view(np.uint16), sx.view(np.uint16))
    rot.close()


def test_pack_weight_matches_oracle(sq):
    w = wl.small("pw", 8, 64, 64, 200, 31)
    X, W = wl.make_layer(w)
    R1, R2 = ora.build_rotation(X.astype(np.float32), w.n1, w.n2)
    rot = sq.sq_rotation_from_factors(R1, R2)
    q = Guarded(w.N * w.n // 2)
    s = Guarded(w.N * 2)
    sq.sq_pack_weight(rot, dev(W), w.N, w.n, q, s)
    torch_mod().cuda.synchronize()
    q.check(); s.check()
    Wq_o, sw_o, _ = ora.pack_weight(W, R1, R2, "f32")
    Wq = q.numpy(np.uint8, (w.N, w.n // 2))
    sw = s.numpy(np.float16, (w.N,))
    assert _fp16_ulps_apart(sw, sw_o).max() <= 1
    d = np.abs(ora.unpack_int4(Wq).astype(np.int32) - ora.unpack_int4(Wq_o).astype(np.int32))
    assert d.max() <= 1 and np.count_nonzero(d) <= 1e-3 * d.size
    rot.close()


def test_rotate_quant_is_deterministic(sq):
    w = wl.small("det", 50, 64, 64, 8, 41)
    X = wl.make_activations(w)
    R1, R2 = ora.build_rotation(X.astype(np.float32), w.n1, w.n2)
    rot = sq.sq_rotation_from_factors(R1, R2)
    a = run_rotate_quant(sq, rot, X)
    b = run_rotate_quant(sq, rot, X)
    for x, y in zip(a, b):
        assert np.array_equal(x.view(np.uint8), y.view(np.uint8))
    rot.close()


# ------------------------------------------------------------------ steps 1+2, R2 applied through its structure
ST_SHAPES = [(64, 64, 37), (64, 64, 301), (8, 64, 9), (24, 64, 7), (48, 64, 11), (128, 64, 5), (100, 64, 3),
             (32, 128, 5), (100, 128, 3), (112, 128, 4), (64, 128, 6), (128, 128, 3), (16, 128, 13)]


def _structured_pair(sq, X, n1, n2, flags, seed=3):
    """The oracle's factors and the library's handle for the same calibration batch and the same random
    block O; the handle applies R2 = H R2^U piece by piece, the oracle as the dense product."""
    O = ora.haar_orthogonal(n1 - 2, np.random.default_rng(seed)) if n1 > 2 else None
    R1, R2 = ora.build_rotation(X.astype(np.float32), n1, n2, flags=flags, O=O)
    rot = sq.sq_build_rotation(X.astype(np.float32), n1, n2, flags=flags | sq.SQ_ROT_APPLY_STRUCTURED, O=O)
    return R1, R2, rot


@pytest.mark.parametrize("n1,n2,M", ST_SHAPES)
def test_structured_rotation_matches_oracle(sq, n1, n2, M):
    w = wl.small(f"st{n1}x{n2}", M, n1, n2, 8, seed=n1 * 5 + n2)
    X = wl.make_activations(w)
    R1, R2, rot = _structured_pair(sq, X, n1, n2, ora.ROT_DEFAULT)
    assert rot.structured
    check_rotate_quant(sq, X, R1, R2, rot=rot)


@pytest.mark.parametrize("flags", [0, 1, 2, 3, 4, 5, 6])
@pytest.mark.parametrize("n1,n2,M", [(64, 64, 21), (112, 128, 5)])
def test_structured_rotation_with_components_switched_off(sq, n1, n2, M, flags):
    """Every subset of ART / URT / Hadamard: R2 is H R2^U, H alone, R2^U alone or the identity."""
    w = wl.small(f"stf{n1}x{n2}", M, n1, n2, 8, seed=n1 + n2 + flags)
    X = wl.make_activations(w)
    R1, R2, rot = _structured_pair(sq, X, n1, n2, flags)
    assert rot.structured
    check_rotate_quant(sq, X, R1, R2, rot=rot)


def test_structured_and_dense_application_agree(sq):
    """The same handle built without SQ_ROT_APPLY_STRUCTURED holds the same factors and rotates through
    the dense kernel; both are within the tolerance of the oracle, and their rotated rows within 2e-5
    of each other."""
    w = wl.small("stvsd", 70, 64, 64, 8, 91)
    X = wl.make_activations(w)
    R1, R2, rot = _structured_pair(sq, X, 64, 64, ora.ROT_DEFAULT)
    O = ora.haar_orthogonal(62, np.random.default_rng(3))
    dense = sq.sq_build_rotation(X.astype(np.float32), 64, 64, flags=sq.SQ_ROT_DEFAULT, O=O)
    assert rot.structured and not dense.structured
    for a, b in zip(rot.factors(), dense.factors()):
        assert np.array_equal(a, b)
    _, _, Zs = run_rotate_quant(sq, rot, X)
    _, _, Zd = run_rotate_quant(sq, dense, X)
    assert np.linalg.norm(Zs.astype(np.float64) - Zd) <= 2e-5 * np.linalg.norm(Zd)
    check_rotate_quant(sq, X, R1, R2, rot=dense)
    rot.close()


@pytest.mark.parametrize("w", [wl.L7B_QKVO, wl.L70B_GATEUP, wl.decode_up(1), wl.decode_up(64), wl.decode_down(1),
                               wl.decode_down(64)], ids=lambda w: w.name)
def test_structured_rotation_full_configs(sq, w):
    X = wl.make_activations(w)
    R1, R2, rot = _structured_pair(sq, X, w.n1, w.n2, ora.ROT_DEFAULT, seed=w.seed)
    assert rot.structured
    rng = np.random.default_rng(4)
    rows = np.unique(np.concatenate([[0, w.M - 1], rng.integers(0, w.M, size=min(w.M, 96))]))
    check_rotate_quant(sq, X, R1, R2, rows=rows, rot=rot)


def test_structured_rotation_many_short_rows_and_determinism(sq):
    w = wl.small("stmany", 70001, 8, 64, 8, 78)
    X = wl.make_activations(w)
    R1, R2, rot = _structured_pair(sq, X, w.n1, w.n2, ora.ROT_DEFAULT)
    a = run_rotate_quant(sq, rot, X, want_z=False)
    b = run_rotate_quant(sq, rot, X, want_z=False)
    assert np.array_equal(a[0], b[0]) and np.array_equal(a[1].view(np.uint16), b[1].view(np.uint16))
    rng = np.random.default_rng(2)
    rows = np.unique(np.concatenate([[0, 1, 2, 3, 65535, 65536, 69999, 70000], rng.integers(0, w.M, size=120)]))
    check_rotate_quant(sq, X, R1, R2, rows=rows, rot=rot)


# ------------------------------------------------------------------ step 3
def random_codes(rng, rows, K):
    c = rng.integers(-8, 8, size=(rows, K)).astype(np.int8)
    return c


def run_gemm(sq, Xc, Wc, sx, sw, want_acc=True):
    M, K = Xc.shape
    N = Wc.shape[0]
    Xq, Wq = ora.pack_int4(Xc), ora.pack_int4(Wc)
    y = Guarded(M * N * 2)
    a = Guarded(M * N * 4) if want_acc else None
    sq.sq_w4a4_gemm(dev(Xq), dev(sx), dev(Wq), dev(sw), M, N, K, y, a)
    torch_mod().cuda.synchronize()
    assert sq.sq_last_device_status() == sq.SQ_OK
    y.check()
    if a is not None:
        a.check()
    return y.numpy(np.float16, (M, N)), (a.numpy(np.int32, (M, N)) if a is not None else None)


GEMM_SHAPES = [
    # plain integer kernel (K % 128 != 0 or N % 8 != 0)
    (1, 1, 2), (3, 8, 34), (5, 24, 130), (7, 13, 256),
    # tensor-core kernel: single tile, ragged M and N, several k-blocks (more than the ring depth)
    (1, 8, 128), (4, 128, 128), (16, 136, 256), (64, 512, 512), (128, 256, 1152), (130, 264, 640),
    (300, 1000, 384), (257, 72, 2048), (64, 4096, 1024),
    # CTA-pair kernel (M > 128, N >= 128): one tile, ragged halves, odd k-block counts, several
    # tiles per pair and more k-blocks than the operand ring holds
    (129, 128, 128), (256, 256, 128), (200, 136, 384), (384, 520, 1664), (1000, 1288, 896),
    (513, 2304, 2176),
    # more CTA-pair shapes: N a multiple of 64 only, several bands with a ragged last one
    (300, 1024, 256), (520, 832, 384), (2048, 4096, 128), (1100, 1792, 640),
    # 65..128 tokens: the pair kernel with a half-empty tile (many channel tiles or short K) or the
    # decode kernel twice (few channels, long K), with one and with 63 rows in the second launch
    (100, 9608, 512), (96, 520, 8192), (65, 256, 6144), (127, 264, 4096),
    # decode kernel (M <= 64, weights as the A operand, K split over a cluster): all three
    # token-count classes, ragged channel tile, odd k-block count, the two decode layer shapes;
    # clusters of 2, 4 and 8, and more tiles than the device holds clusters (slots reused)
    (9, 264, 1280), (64, 640, 2560), (40, 136, 8192), (16, 5120, 14336), (33, 2432, 6144), (64, 5120, 14336),
    # dot-product kernel (M <= 2, and M <= 4 where the decode kernel does not take the shape): odd
    # channel counts, every token-count class
    (2, 1001, 2048), (2, 264, 14336), (3, 1001, 2048), (4, 7, 96), (3, 264, 14336),
    (1, 4096, 4096), (17, 1000, 2048), (33, 384, 1664), (64, 2048, 2304), (4, 14336, 4096), (16, 4096, 14336),
]


@pytest.mark.parametrize("M,N,K", GEMM_SHAPES)
def test_gemm_accumulators_bit_exact(sq, M, N, K):
    rng = np.random.default_rng(M * 1000003 + N * 101 + K)
    Xc, Wc = random_codes(rng, M, K), random_codes(rng, N, K)
    sx = rng.uniform(0.01, 2.0, size=M).astype(np.float16)
    sw = rng.uniform(0.001, 0.1, size=N).astype(np.float16)
    Y, acc = run_gemm(sq, Xc, Wc, sx, sw)
    acc_o = ora.gemm_i32(Xc, Wc)
    assert np.array_equal(acc, acc_o)
    Yo = ora.dequant(acc_o, sx, sw).astype(np.float64)
    err = np.linalg.norm(Y.astype(np.float64) - Yo) / max(np.linalg.norm(Yo), 1e-30)
    assert err <= 1e-3
    # the dequantised outputs are within one fp16 ulp of the float64 result
    assert _fp16_ulps_apart(Y, Yo.astype(np.float16)).max() <= 1


def test_gemm_random_shapes_bit_exact(sq):
    """Seeded random shapes across every kernel's range (token counts from each dispatch class, ragged
    channel counts, K a multiple of 128 or merely even): accumulators equal the oracle's bit for bit."""
    rng = np.random.default_rng(20251122)
    done = 0
    while done < 60:
        cls = done % 6
        M = int([rng.integers(1, 5), rng.integers(3, 17), rng.integers(17, 65), rng.integers(65, 129),
                 rng.integers(129, 300), rng.integers(1, 300)][cls])
        N = int(rng.integers(1, 200)) * 8 if rng.random() < 0.85 else int(rng.integers(1, 1500))
        K = int(rng.integers(1, 60)) * 128 if rng.random() < 0.85 else int(rng.integers(1, 2000)) * 2
        if M * N * K > 1.0e8:
            continue
        Xc, Wc = random_codes(rng, M, K), random_codes(rng, N, K)
        sx = rng.uniform(0.01, 2.0, size=M).astype(np.float16)
        sw = rng.uniform(0.001, 0.1, size=N).astype(np.float16)
        Y, acc = run_gemm(sq, Xc, Wc, sx, sw)
        acc_o = ora.gemm_i32(Xc, Wc)
        assert np.array_equal(acc, acc_o), (M, N, K)
        assert _fp16_ulps_apart(Y, ora.dequant(acc_o, sx, sw)).max() <= 1, (M, N, K)
        done += 1


def test_gemm_extreme_codes_do_not_overflow(sq):
    M, N, K = 4, 8, 28672
    Xc = np.full((M, K), -8, np.int8)
    Wc = np.full((N, K), -8, np.int8)
    Wc[1] = 7
    sx = np.full(M, 2.0 ** -10, np.float16)
    sw = np.full(N, 2.0 ** -10, np.float16)
    Y, acc = run_gemm(sq, Xc, Wc, sx, sw)
    assert np.all(acc[:, 0] == 64 * K) and np.all(acc[:, 1] == -56 * K)
    assert np.array_equal(acc, ora.gemm_i32(Xc, Wc))


@pytest.mark.parametrize("M,N", [(2, 8), (3, 136), (40, 256), (100, 128), (130, 128)])
def test_gemm_largest_k_and_largest_accumulator(sq, M, N):
    """K = 65536 is the largest supported contraction; with every code at -8 the accumulator reaches
    64 K = 2^22, the top of the range the exact int -> float step of the epilogues is built for."""
    K = 65536
    rng = np.random.default_rng(M * 31 + N)
    Xc, Wc = random_codes(rng, M, K), random_codes(rng, N, K)
    Xc[0] = -8
    Wc[0] = -8
    Wc[N - 1] = 7
    sx = np.full(M, 2.0 ** -12, np.float16)
    sw = np.full(N, 2.0 ** -12, np.float16)
    Y, acc = run_gemm(sq, Xc, Wc, sx, sw)
    acc_o = ora.gemm_i32(Xc, Wc)
    assert acc_o[0, 0] == 64 * K and acc_o[0, N - 1] == -56 * K
    assert np.array_equal(acc, acc_o)
    assert np.array_equal(Y.view(np.uint16), ora.dequant(acc_o, sx, sw).view(np.uint16))


def test_gemm_prefill_config_sampled_rows(sq):
    """LLaMA-2-7B q/k/v/o prefill shape at full size, in the configuration the benchmark times;
    the oracle checks every output channel of a sample of token rows."""
    M, N, K = 2048, 4096, 4096
    rng = np.random.default_rng(77)
    Xc, Wc = random_codes(rng, M, K), random_codes(rng, N, K)
    sx = rng.uniform(0.01, 2.0, size=M).astype(np.float16)
    sw = rng.uniform(0.001, 0.1, size=N).astype(np.float16)
    Y, acc = run_gemm(sq, Xc, Wc, sx, sw)
    rows = np.unique(np.concatenate([[0, 127, 128, M - 1], rng.integers(0, M, size=60)]))
    acc_o = ora.gemm_i32(Xc[rows], Wc)
    assert np.array_equal(acc[rows], acc_o)
    Yo = ora.dequant(acc_o, sx[rows], sw)
    assert _fp16_ulps_apart(Y[rows], Yo).max() <= 1


@pytest.mark.parametrize("M,N,K", [(200, 384, 1024), (40, 136, 8192), (16, 5120, 14336), (2, 264, 4096)])
def test_gemm_is_deterministic(sq, M, N, K):
    """Two calls give the same bits: the pair kernel, the decode kernel with K split over clusters
    (one tile per cluster, and several tiles per cluster with the reduce buffer reused), the
    dot-product kernel."""
    rng = np.random.default_rng(5)
    Xc, Wc = random_codes(rng, M, K), random_codes(rng, N, K)
    sx = rng.uniform(0.01, 2.0, size=M).astype(np.float16)
    sw = rng.uniform(0.001, 0.1, size=N).astype(np.float16)
    a = run_gemm(sq, Xc, Wc, sx, sw)
    b = run_gemm(sq, Xc, Wc, sx, sw)
    assert np.array_equal(a[0].view(np.uint16), b[0].view(np.uint16)) and np.array_equal(a[1], b[1])


# ------------------------------------------------------------------ whole layer
def run_linear(sq, w, X, W, R1, R2, host=False):
    torch = torch_mod()
    rot = sq.sq_rotation_from_factors(R1, R2)
    M, N, K = X.shape[0], W.shape[0], w.n
    wq = Guarded(N * K // 2)
    sw = Guarded(N * 2)
    sq.sq_pack_weight(rot, dev(W), N, K, wq, sw)
    if host:
        nbytes = sq.sq_linear_host_workspace_bytes(M, N, K)
        ws = torch.empty(nbytes + 256, dtype=torch.uint8, device="cuda")
        off = (-ws.data_ptr()) % 256
        Xh = torch.from_numpy(X).pin_memory()
        Yh = torch.empty((M, N), dtype=torch.float16).pin_memory()
        sq.sq_linear_host(rot, Xh, M, wq, sw, N, K, ws.data_ptr() + off, nbytes, Yh)
        Y = Yh.numpy().copy()
    else:
        nbytes = sq.sq_linear_workspace_bytes(M, K)
        ws = torch.empty(nbytes + 256, dtype=torch.uint8, device="cuda")
        off = (-ws.data_ptr()) % 256
        y = Guarded(M * N * 2)
        sq.sq_linear(rot, dev(X), M, wq, sw, N, K, ws.data_ptr() + off, nbytes, y)
        torch.cuda.synchronize()
        y.check()
        Y = y.numpy(np.float16, (M, N))
    assert sq.sq_last_device_status() == sq.SQ_OK
    wq.check(); sw.check()
    rot.close()
    return Y


@pytest.mark.parametrize("w", [wl.TINY, wl.small("lin1", 70, 64, 64, 264, 51), wl.small("lin2", 9, 12, 8, 24, 52),
                               wl.small("lin3", 5, 172, 64, 136, 53), wl.decode_up(4),
                               wl.small("lin_decode_split", 16, 112, 128, 512, 54),
                               wl.small("lin_mid_batch", 100, 64, 64, 520, 55)])
@pytest.mark.parametrize("host", [False, True])
def test_linear_matches_oracle(sq, w, host):
    X, W = wl.make_layer(w)
    flags = ora.ROT_DEFAULT if (w.n2 & (w.n2 - 1)) == 0 else (ora.ROT_ART | ora.ROT_URT)
    R1, R2 = ora.build_rotation(X.astype(np.float32), w.n1, w.n2, flags=flags)
    Y = run_linear(sq, w, X, W, R1, R2, host=host).astype(np.float64)
    Yo = ora.linear(X, W, R1, R2).astype(np.float64)
    assert np.linalg.norm(Y - Yo) <= 1e-2 * np.linalg.norm(Yo)


def test_linear_prefill_config_sampled(sq):
    """Full LLaMA-2-7B q/k/v/o prefill layer through sq_linear; the oracle recomputes a sample of
    token rows end to end (weights quantised by the oracle in full)."""
    w = wl.L7B_QKVO
    X, W = wl.make_layer(w)
    R1, R2 = ora.build_rotation(X.astype(np.float32), w.n1, w.n2)
    Y = run_linear(sq, w, X, W, R1, R2)
    rng = np.random.default_rng(3)
    rows = np.unique(np.concatenate([[0, w.M - 1], rng.integers(0, w.M, size=62)]))
    Yo = ora.linear(X[rows], W, R1, R2).astype(np.float64)
    Yg = Y[rows].astype(np.float64)
    assert np.linalg.norm(Yg - Yo) <= 1e-2 * np.linalg.norm(Yo)


def test_linear_host_chunked_equals_device_path(sq):
    """sq_linear_host cuts batches of 512 rows or more into row chunks whose copies and computation
    overlap.  Every row is treated on its own, so the outputs must equal those of one sq_linear call
    on the whole batch bit for bit -- here with a ragged last chunk (1100 = 2 x 512 + 76 rows) that
    takes a different GEMM kernel than the full chunks -- and twice in a row (the copy streams and
    events are reused)."""
    w = wl.small("host_chunks", 1100, 64, 64, 264, 77)
    X, W = wl.make_layer(w)
    R1, R2 = ora.build_rotation(X.astype(np.float32), w.n1, w.n2)
    Yd = run_linear(sq, w, X, W, R1, R2, host=False)
    for _ in range(2):
        Yh = run_linear(sq, w, X, W, R1, R2, host=True)
        assert np.array_equal(Yh.view(np.uint16), Yd.view(np.uint16))
    rows = np.array([0, 255, 256, 1023, 1024, 1099])
    Yo = ora.linear(X[rows], W, R1, R2).astype(np.float64)
    assert np.linalg.norm(Yd[rows].astype(np.float64) - Yo) <= 1e-2 * np.linalg.norm(Yo)


def test_empty_inputs_are_no_ops(sq):
    w = wl.TINY
    X = wl.make_activations(w)
    R1, R2 = ora.build_rotation(X.astype(np.float32), w.n1, w.n2)
    rot = sq.sq_rotation_from_factors(R1, R2)
    before = sq.sq_kernel_launch_count()
    sq.sq_rotate_quant_act(rot, None, 0, None, None)
    sq.sq_w4a4_gemm(None, None, None, None, 0, 0, 128, None)
    sq.sq_linear(rot, None, 0, None, None, 8, w.n, None, 0, None)
    assert sq.sq_kernel_launch_count() == before
    rot.close()
