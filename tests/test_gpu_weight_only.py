"""GPU parity of the weight-only variant (Appendix "Weight-only Quantization", Table "wquant") and of
the grouped layer, called through the C ABI, against the CPU oracle on identical seeded inputs.
Tolerances:
  * b-bit weight codes: at most 1 LSB apart on <= 0.1% of the elements (rounding-boundary cases; both
    sides take the decision in fp32), steps equal to within 1 fp16 ulp; bit-exact under the identity
    rotation;
  * fp16 rotated rows: |Z16 - fp16(Z)| <= 1e-5 * max|Z_t| + 1 fp16 ulp of the entry (the 1e-5 of the
    rotation, then one rounding on each side);
  * the product on identical fp16 rows and codes: bit-exact where fp32 accumulation is exact (small
    integers); otherwise relative Frobenius error <= 1e-3 (one fp16 rounding is 2.4e-4 rms) and, entry
    by entry, <= 1 fp16 ulp of the result + K * 2^-23 * sum_k |z_k code_k| * s_w (K fp32 additions, each
    off by at most one unit in the last place of a running sum that never exceeds the absolute sum);
  * the layer's fp16 outputs: relative Frobenius error <= 1e-2.
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


def _ulps(a, b):
    return np.abs(a.view(np.int16).astype(np.int32) - b.view(np.int16).astype(np.int32))


def _sync_ok(sq):
    torch_mod().cuda.synchronize()
    assert sq.sq_last_device_status() == sq.SQ_OK


# ------------------------------------------------------------------ offline weight path
@pytest.mark.parametrize("bits", [4, 3])
@pytest.mark.parametrize("n1,n2,N", [(16, 32, 40), (64, 64, 130), (172, 64, 24), (112, 128, 17), (12, 8, 9), (7, 8, 5)])
def test_pack_weight_wo_matches_oracle(sq, bits, n1, n2, N):
    w = wl.small(f"wo{n1}x{n2}", 16, n1, n2, N, seed=n1 + 3 * n2 + bits)
    X, W = wl.make_layer(w)
    R1, R2 = ora.build_rotation(X.astype(np.float32), n1, n2)
    rot = sq.sq_rotation_from_factors(R1, R2)
    K = n1 * n2
    q, s = Guarded(N * K // 2), Guarded(N * 2)
    sq.sq_pack_weight_wo(rot, dev(W), N, K, bits, q, s)
    _sync_ok(sq)
    q.check(); s.check()
    Zo = ora.rotate(W, R1, R2)
    co, do = ora.quantize_rows_bits(Zo, bits, "f32")
    cg = ora.unpack_int4_interleaved(q.numpy(np.uint8, (N, K // 2)))
    sg = s.numpy(np.float16, (N,))
    assert _ulps(sg, do).max() <= 1
    diff = np.abs(cg.astype(np.int32) - co.astype(np.int32))
    assert diff.max() <= 1 and np.count_nonzero(diff) <= max(1, 1e-3 * diff.size)
    assert cg.min() >= -(2 ** (bits - 1)) and cg.max() <= 2 ** (bits - 1) - 1
    rot.close()


@pytest.mark.parametrize("bits", [4, 3])
def test_pack_weight_wo_identity_rotation_is_bit_exact(sq, bits):
    rng = np.random.default_rng(90 + bits)
    N, K = 37, 264
    W = (rng.standard_normal((N, K)) * rng.uniform(1e-3, 30.0, size=(N, 1))).astype(np.float16)
    W[5] = 0
    q, s = Guarded(N * K // 2), Guarded(N * 2)
    sq.sq_pack_weight_wo(None, dev(W), N, K, bits, q, s)
    _sync_ok(sq)
    q.check(); s.check()
    Wq_o, sw_o, _ = ora.pack_weight_wo(W, None, None, bits, "f32")
    assert np.array_equal(q.numpy(np.uint8, (N, K // 2)), Wq_o)
    assert np.array_equal(s.numpy(np.float16, (N,)).view(np.uint16), sw_o.view(np.uint16))


def test_weight_only_argument_checks(sq):
    lib = sq.load()
    w = wl.small("woarg", 8, 8, 8, 16, 5)
    X, W = wl.make_layer(w)
    R1, R2 = ora.build_rotation(X.astype(np.float32), 8, 8)
    rot = sq.sq_rotation_from_factors(R1, R2)
    dW, q, s = dev(W), Guarded(16 * 32), Guarded(32)
    before = sq.sq_kernel_launch_count()
    assert lib.sq_pack_weight_wo(rot.handle, dW.data_ptr(), 16, 64, 5, q.data_ptr(), s.data_ptr(), None) == sq.SQ_ERR_INVALID_ARG
    assert lib.sq_pack_weight_wo(rot.handle, dW.data_ptr(), 16, 72, 4, q.data_ptr(), s.data_ptr(), None) == sq.SQ_ERR_SHAPE
    assert lib.sq_pack_weight_wo(None, dW.data_ptr(), 16, 60, 4, q.data_ptr(), s.data_ptr(), None) == sq.SQ_ERR_SHAPE
    assert lib.sq_w4a16_gemm(dW.data_ptr(), q.data_ptr(), s.data_ptr(), 4, 16, 60, q.data_ptr(), None) == sq.SQ_ERR_SHAPE
    assert lib.sq_w4a16_gemm(None, q.data_ptr(), s.data_ptr(), 4, 16, 64, q.data_ptr(), None) == sq.SQ_ERR_INVALID_ARG
    assert lib.sq_w4a16_gemm(dW.data_ptr() + 2, q.data_ptr(), s.data_ptr(), 4, 16, 64, q.data_ptr(), None) == sq.SQ_ERR_ALIGN
    assert lib.sq_rotate_act_f16(rot.handle, dW.data_ptr(), 4, dW.data_ptr(), None) == sq.SQ_ERR_INVALID_ARG
    assert lib.sq_linear_wo(rot.handle, dW.data_ptr(), 4, q.data_ptr(), s.data_ptr(), 16, 64, q.data_ptr(), 16,
                            q.data_ptr(), None) == sq.SQ_ERR_NOMEM
    # empty problems are no-ops
    assert lib.sq_w4a16_gemm(None, None, None, 0, 16, 64, None, None) == sq.SQ_OK
    assert lib.sq_rotate_act_f16(rot.handle, None, 0, None, None) == sq.SQ_OK
    assert lib.sq_pack_weight_wo(rot.handle, None, 0, 64, 4, None, None, None) == sq.SQ_OK
    assert sq.sq_kernel_launch_count() == before
    rot.close()


# ------------------------------------------------------------------ step 1 alone, fp16 rows
ROT_SHAPES = [(16, 32, 64), (64, 64, 37), (64, 64, 301), (8, 64, 9), (100, 128, 3), (112, 128, 4), (64, 128, 70),
              (129, 64, 3), (172, 64, 9), (224, 128, 5), (144, 128, 150), (12, 8, 5), (7, 6, 3)]


@pytest.mark.parametrize("n1,n2,M", ROT_SHAPES)
def test_rotate_act_f16_matches_oracle(sq, n1, n2, M):
    w = wl.small(f"rf{n1}x{n2}", M, n1, n2, 8, seed=5 * n1 + n2)
    X = wl.make_activations(w)
    flags = ora.ROT_DEFAULT if (n2 & (n2 - 1)) == 0 else (ora.ROT_ART | ora.ROT_URT)
    R1, R2 = ora.build_rotation(X.astype(np.float32), n1, n2, flags=flags)
    rot = sq.sq_rotation_from_factors(R1, R2)
    z = Guarded(M * n1 * n2 * 2)
    sq.sq_rotate_act_f16(rot, dev(X), M, z)
    _sync_ok(sq)
    z.check()
    Zg = z.numpy(np.float16, (M, n1 * n2))
    Zo = ora.rotate(X, R1, R2)
    Z16o = ora.rotate_f16(X, R1, R2)
    rowmax = np.max(np.abs(Zo), axis=1, keepdims=True)
    err = np.abs(Zg.astype(np.float64) - Z16o.astype(np.float64))
    assert np.all(err <= 1e-5 * rowmax + 2.0 ** -10 * np.abs(Zo) + 2.0 ** -24)
    assert np.count_nonzero(_ulps(Zg, Z16o) > 1) <= 0.02 * Zg.size          # small entries of rows with outliers
    assert np.linalg.norm(Zg.astype(np.float64) - Zo) <= 6e-4 * np.linalg.norm(Zo)
    rot.close()


# ------------------------------------------------------------------ the product
def _run_wo_gemm(sq, Z16, codes, sw):
    M, K = Z16.shape
    N = codes.shape[0]
    y = Guarded(M * N * 2)
    sq.sq_w4a16_gemm(dev(Z16), dev(ora.pack_int4_interleaved(codes)), dev(sw), M, N, K, y)
    _sync_ok(sq)
    y.check()
    return y.numpy(np.float16, (M, N))


WO_GEMM_SHAPES = [(1, 128, 64), (5, 136, 192), (64, 264, 256), (128, 128, 320), (130, 384, 1024), (200, 8, 4096),
                  (33, 5120, 512), (257, 16392, 128), (300, 16640, 448),
                  # two channel tiles per token tile: one tile pair; more tile pairs than SMs (a CTA's single
                  # accumulator set is handed back and reused), the last pair half empty
                  (129, 256, 64), (1300, 3592, 192),
                  # decode batches with few output channels: K split over clusters of 4 and of 2
                  (16, 264, 8192), (40, 1024, 4096), (64, 136, 2048),
                  # one or two tokens: the dot-product kernel (ragged row count, long rows)
                  (2, 134, 4096), (1, 263 * 8, 14336), (2, 5, 32),
                  # shapes the tensor-core path does not take: the plain kernel
                  (7, 5, 72), (3, 12, 8), (20, 130, 200)]


@pytest.mark.parametrize("M,N,K", WO_GEMM_SHAPES)
def test_wo_gemm_is_bit_exact_on_small_integers(sq, M, N, K):
    """Integer activations in [-8, 8], every code value, power-of-two steps: all partial sums are
    integers below 2^24, so fp32 accumulation is exact in any order and the result must be the
    oracle's, bit for bit (every channel, every k-block, the storage order, the ragged edges)."""
    rng = np.random.default_rng(M * 131 + N * 7 + K)
    Z16 = rng.integers(-8, 9, size=(M, K)).astype(np.float16)
    codes = rng.integers(-8, 8, size=(N, K), dtype=np.int8)
    codes[0] = -8
    Z16[0] = -8
    sw = (2.0 ** rng.integers(-12, -6, size=N)).astype(np.float16)
    Yg = _run_wo_gemm(sq, Z16, codes, sw)
    Yo = ora.gemm_w4a16(Z16, codes, sw)
    assert np.array_equal(Yg.view(np.uint16), Yo.view(np.uint16))


@pytest.mark.parametrize("M,N,K", [(2048, 4096, 4096), (2048, 4096, 11008), (4096, 28672, 8192)])
def test_wo_gemm_full_size_bit_exact_on_sampled_rows(sq, M, N, K):
    """The benchmark's prefill shapes (up to 24 tiles per CTA pair, 43 stages per tile, weights beyond
    L2): same integer construction as above (|partial sums| <= 64 K < 2^24), every channel of sampled
    token rows against the oracle, bit for bit."""
    rng = np.random.default_rng(M + N + K)
    Z16 = rng.integers(-8, 9, size=(M, K), dtype=np.int8).astype(np.float16)
    codes = rng.integers(-8, 8, size=(N, K), dtype=np.int8)
    sw = (2.0 ** rng.integers(-12, -6, size=N)).astype(np.float16)
    Yg = _run_wo_gemm(sq, Z16, codes, sw)
    rows = np.unique(np.concatenate([[0, 127, 128, 255, 256, M - 1], rng.integers(0, M, size=26)]))
    for c0 in range(0, N, 4096):                      # the oracle widens the codes to float64: in blocks of channels
        Yo = ora.gemm_w4a16(Z16[rows], codes[c0:c0 + 4096], sw[c0:c0 + 4096])
        assert np.array_equal(Yg[rows, c0:c0 + 4096].view(np.uint16), Yo.view(np.uint16))


def test_wo_gemm_random_shapes_bit_exact(sq):
    """Forty-eight seeded random shapes over every kernel of the product (dot products, the single-CTA
    form with and without the K split and with one or two channel tiles, the CTA-pair form, the plain
    kernel), small integers so that the result must equal the oracle's bit for bit."""
    rng = np.random.default_rng(20240607)
    for trial in range(48):
        kind = trial % 6
        if kind == 0:
            M, N, K = int(rng.integers(1, 3)), int(rng.integers(1, 400)), 32 * int(rng.integers(1, 200))
        elif kind == 1:
            M, N, K = int(rng.integers(3, 65)), 8 * int(rng.integers(16, 300)), 64 * int(rng.integers(1, 100))
        elif kind == 2:
            M, N, K = int(rng.integers(3, 65)), 8 * int(rng.integers(16, 40)), 64 * int(rng.integers(64, 200))
        elif kind == 3:
            M, N, K = int(rng.integers(65, 400)), 8 * int(rng.integers(1, 200)), 64 * int(rng.integers(1, 40))
        elif kind == 5:
            M, N, K = int(rng.integers(129, 1200)), 8 * int(rng.integers(32, 500)), 64 * int(rng.integers(1, 24))
        else:
            M, N, K = int(rng.integers(1, 40)), int(rng.integers(1, 150)), 8 * int(rng.integers(1, 60))
        Z16 = rng.integers(-8, 9, size=(M, K)).astype(np.float16)
        codes = rng.integers(-8, 8, size=(N, K), dtype=np.int8)
        sw = (2.0 ** rng.integers(-12, -6, size=N)).astype(np.float16)
        Yg = _run_wo_gemm(sq, Z16, codes, sw)
        Yo = ora.gemm_w4a16(Z16, codes, sw)
        assert np.array_equal(Yg.view(np.uint16), Yo.view(np.uint16)), (trial, M, N, K)


@pytest.mark.parametrize("M,N,K", [(70, 264, 4096), (16, 1024, 14336), (300, 512, 2048), (9, 130, 200), (1, 520, 14336),
                                   (2, 264, 4096)])
def test_wo_gemm_real_values_within_the_fp32_accumulation_bound(sq, M, N, K):
    rng = np.random.default_rng(M + N + K)
    Z16 = (rng.standard_normal((M, K)) * rng.uniform(0.1, 10.0, size=(M, 1))).astype(np.float16)
    codes = rng.integers(-8, 8, size=(N, K), dtype=np.int8)
    sw = rng.uniform(1e-3, 3e-2, size=N).astype(np.float16)
    Yg = _run_wo_gemm(sq, Z16, codes, sw).astype(np.float64)
    Yo = ora.gemm_w4a16(Z16, codes, sw).astype(np.float64)
    assert np.linalg.norm(Yg - Yo) <= 1e-3 * np.linalg.norm(Yo)
    S = np.abs(Z16.astype(np.float64)) @ np.abs(codes.astype(np.float64)).T
    bound = 2.0 ** -10 * np.abs(Yo) + K * 2.0 ** -23 * S * sw.astype(np.float64)[None, :] + 2.0 ** -24
    assert np.all(np.abs(Yg - Yo) <= bound)


def test_wo_gemm_three_bit_codes_and_determinism(sq):
    rng = np.random.default_rng(77)
    M, N, K = 48, 392, 1216
    Z16 = rng.standard_normal((M, K)).astype(np.float16)
    codes = rng.integers(-4, 4, size=(N, K), dtype=np.int8)
    sw = rng.uniform(1e-3, 3e-2, size=N).astype(np.float16)
    a = _run_wo_gemm(sq, Z16, codes, sw)
    b = _run_wo_gemm(sq, Z16, codes, sw)
    assert np.array_equal(a.view(np.uint16), b.view(np.uint16))
    Yo = ora.gemm_w4a16(Z16, codes, sw).astype(np.float64)
    assert np.linalg.norm(a.astype(np.float64) - Yo) <= 1e-3 * np.linalg.norm(Yo)


# ------------------------------------------------------------------ the weight-only layer
def _run_linear_wo(sq, rot, X, W, bits):
    torch = torch_mod()
    M, K = X.shape
    N = W.shape[0]
    wq, sw = Guarded(N * K // 2), Guarded(N * 2)
    sq.sq_pack_weight_wo(rot, dev(W), N, K, bits, wq, sw)
    nbytes = sq.sq_linear_wo_workspace_bytes(M, K)
    ws = torch.empty(nbytes + 256, dtype=torch.uint8, device="cuda")
    y = Guarded(M * N * 2)
    sq.sq_linear_wo(rot, dev(X), M, wq, sw, N, K, ws.data_ptr() + (-ws.data_ptr()) % 256, nbytes, y)
    _sync_ok(sq)
    y.check(); wq.check(); sw.check()
    return y.numpy(np.float16, (M, N))


@pytest.mark.parametrize("bits", [4, 3])
@pytest.mark.parametrize("w", [wl.TINY, wl.small("wl1", 70, 64, 64, 264, 51), wl.small("wl2", 9, 12, 8, 24, 52),
                               wl.small("wl3", 33, 172, 64, 136, 53), wl.small("wl4", 5, 112, 128, 512, 54),
                               wl.small("wl5", 150, 64, 128, 128, 55)], ids=lambda w: w.name)
def test_linear_wo_matches_oracle(sq, w, bits):
    X, W = wl.make_layer(w)
    R1, R2 = ora.build_rotation(X.astype(np.float32), w.n1, w.n2)
    rot = sq.sq_rotation_from_factors(R1, R2)
    Yg = _run_linear_wo(sq, rot, X, W, bits).astype(np.float64)
    Yo = ora.linear_wo(X, W, R1, R2, bits).astype(np.float64)
    assert np.linalg.norm(Yg - Yo) <= 1e-2 * np.linalg.norm(Yo)
    # and the variant does what it is for: closer to the unquantised layer than W4A4 on the same inputs
    exact = ora.linear_fp(X, W)
    e_wo = np.linalg.norm(Yg - exact)
    e_w4a4 = np.linalg.norm(ora.linear(X, W, R1, R2).astype(np.float64) - exact)
    if bits == 4:
        assert e_wo < e_w4a4
    rot.close()


@pytest.mark.parametrize("w", [wl.L7B_QKVO, wl.decode_up(16), wl.decode_down(4)], ids=lambda w: w.name)
def test_linear_wo_full_size_sampled_rows(sq, w):
    import dataclasses
    X = wl.make_activations(w)
    Xcal = wl.make_activations(dataclasses.replace(w, M=max(w.M, 64)) if w.M < 64 else w)
    W = wl.make_weights(w)
    R1, R2 = ora.build_rotation(Xcal.astype(np.float32), w.n1, w.n2)
    rot = sq.sq_rotation_from_factors(R1, R2)
    Yg = _run_linear_wo(sq, rot, X, W, 4)
    rows = np.unique(np.concatenate([[0, 1, w.M - 1], np.random.default_rng(w.seed).integers(0, w.M, size=24)]))
    rows = rows[rows < w.M]
    Wq_o = np.empty((w.N, w.K // 2), np.uint8)
    sw_o = np.empty((w.N,), np.float16)
    for r0 in range(0, w.N, 1024):
        Wq_o[r0:r0 + 1024], sw_o[r0:r0 + 1024], _ = ora.pack_weight_wo(W[r0:r0 + 1024], R1, R2, 4)
    Yo = ora.gemm_w4a16(ora.rotate_f16(X[rows], R1, R2), ora.unpack_int4_interleaved(Wq_o), sw_o).astype(np.float64)
    assert np.linalg.norm(Yg[rows].astype(np.float64) - Yo) <= 1e-2 * np.linalg.norm(Yo)
    rot.close()


# ------------------------------------------------------------------ the grouped W4A4 layer
@pytest.mark.parametrize("shared", [False, True], ids=["own_handles", "one_handle"])
@pytest.mark.parametrize("counts", [[5, 0, 3, 1], [64, 7, 130, 0, 0, 9, 1, 40], [0, 0, 12], [300],
                                    [64, 33, 17, 16, 1, 2, 0, 48], [3, 1, 4, 1, 5, 9, 2, 6, 5, 3, 5, 8, 9, 7, 9, 3, 2, 3],
                                    [300, 5, 0, 257, 64, 513, 129]])
def test_linear_grouped_matches_oracle_and_the_per_expert_calls(sq, counts, shared):
    """Each expert with a handle of its own, and all experts on one handle (then steps 1 and 2 run once
    over all rows and only step 3 per expert): against the oracle, and bit for bit against sq_linear on
    each expert's rows."""
    torch = torch_mod()
    n1, n2, N = 64, 64, 264
    K = n1 * n2
    E = len(counts)
    offsets = np.concatenate([[0], np.cumsum(counts)]).astype(np.int64)
    M = int(offsets[-1])
    rng = np.random.default_rng(sum(counts) + E)
    w = wl.small("grp", max(M, 64), n1, n2, N, seed=61)
    X = wl.make_activations(w)[:M].copy()
    Ws = [(0.02 * rng.standard_normal((N, K))).astype(np.float16) for _ in range(E)]
    rots_o = []
    for e in range(E):
        cal = wl.make_activations(wl.small("grpc", 64, n1, n2, N, seed=70 + (0 if shared else e))).astype(np.float32)
        rots_o.append(ora.build_rotation(cal, n1, n2, O=ora.haar_orthogonal(n1 - 2, np.random.default_rng(0 if shared else e))))
    if shared:
        one = sq.sq_rotation_from_factors(*rots_o[0])
        rots = [one] * E
    else:
        rots = [sq.sq_rotation_from_factors(R1, R2) for R1, R2 in rots_o]
    wqs, sws = [], []
    for e in range(E):
        q, s = Guarded(N * K // 2), Guarded(N * 2)
        sq.sq_pack_weight(rots[e], dev(Ws[e]), N, K, q, s)
        wqs.append(q); sws.append(s)
    nbytes = sq.sq_linear_workspace_bytes(M, K)
    ws = torch.empty(nbytes + 256, dtype=torch.uint8, device="cuda")
    wsp = ws.data_ptr() + (-ws.data_ptr()) % 256
    dX = dev(X)
    y = Guarded(M * N * 2)
    before = sq.sq_kernel_launch_count()
    sq.sq_linear_grouped(rots, offsets, dX, wqs, sws, N, K, wsp, nbytes, y)
    launched = sq.sq_kernel_launch_count() - before
    _sync_ok(sq)
    y.check()
    with_rows = sum(1 for c in counts if c > 0)                     # experts without tokens cost nothing
    if with_rows >= 2:
        # steps 1+2 once (one handle) or once per expert; step 3 for sixteen experts per launch (the decode
        # kernel's grouped form when every expert has at most 64 rows, else the CTA-pair kernel's)
        assert launched == (1 if shared else with_rows) + (with_rows + 15) // 16
    else:
        assert launched == 2 * with_rows
    Yg = y.numpy(np.float16, (M, N))
    Yo = ora.linear_grouped(X, offsets, Ws, rots_o).astype(np.float64)
    for e in range(E):
        a, b = int(offsets[e]), int(offsets[e + 1])
        if b > a:
            assert np.linalg.norm(Yg[a:b].astype(np.float64) - Yo[a:b]) <= 1e-2 * np.linalg.norm(Yo[a:b]), e
            # the same rows through sq_linear with that expert's matrices: identical bits
            y1 = Guarded((b - a) * N * 2)
            sq.sq_linear(rots[e], dX[a:b], b - a, wqs[e], sws[e], N, K, wsp, nbytes, y1)
            _sync_ok(sq)
            assert np.array_equal(y1.numpy(np.float16, (b - a, N)).view(np.uint16), Yg[a:b].view(np.uint16))
    for r in ([rots[0]] if shared else rots):
        r.close()


def test_linear_grouped_refuses_bad_arguments_before_any_launch(sq):
    torch = torch_mod()
    lib = sq.load()
    import ctypes
    n1, n2, N = 8, 8, 16
    K = 64
    w = wl.small("grpa", 8, n1, n2, N, seed=3)
    X, W = wl.make_layer(w)
    R1, R2 = ora.build_rotation(X.astype(np.float32), n1, n2)
    rot = sq.sq_rotation_from_factors(R1, R2)
    q, s = Guarded(N * K // 2), Guarded(N * 2)
    sq.sq_pack_weight(rot, dev(W), N, K, q, s)
    torch.cuda.synchronize()
    nbytes = sq.sq_linear_workspace_bytes(8, K)
    ws = torch.empty(nbytes + 256, dtype=torch.uint8, device="cuda")
    wsp = ws.data_ptr() + (-ws.data_ptr()) % 256
    dX, y = dev(X), Guarded(8 * N * 2)
    h = (ctypes.c_void_p * 2)(rot.handle, rot.handle)
    wq = (ctypes.c_void_p * 2)(q.data_ptr(), q.data_ptr())
    sw = (ctypes.c_void_p * 2)(s.data_ptr(), s.data_ptr())
    before = sq.sq_kernel_launch_count()

    def call(off, wq=wq, sw=sw, h=h, nb=nbytes):
        o = (ctypes.c_int64 * 3)(*off)
        return lib.sq_linear_grouped(h, 2, o, dX.data_ptr(), wq, sw, N, K, wsp, nb, y.data_ptr(), None)

    assert call([0, 5, 3]) == sq.SQ_ERR_INVALID_ARG             # offsets must not decrease
    assert call([1, 4, 8]) == sq.SQ_ERR_INVALID_ARG             # and start at 0
    assert call([0, 4, 8], nb=16) == sq.SQ_ERR_NOMEM
    bad = (ctypes.c_void_p * 2)(q.data_ptr(), None)
    assert call([0, 4, 8], wq=bad) == sq.SQ_ERR_INVALID_ARG     # the second expert's weights are missing
    assert sq.sq_kernel_launch_count() == before
    assert call([0, 8, 8], wq=bad) == sq.SQ_OK                  # an expert without tokens is never looked at
    assert sq.sq_kernel_launch_count() == before + 2
    _sync_ok(sq)
    y.check()
    rot.close()
