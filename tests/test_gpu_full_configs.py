"""Every benchmark workload at its full size, in the launch configuration the benchmark times:
  (i)  the GEMM fed oracle-packed random INT4 codes must give bit-exact int32 accumulators on a
       sample of token rows (all rows for the decode workloads) and every output channel;
  (ii) the whole layer through sq_linear must agree with the oracle's layer within 1e-2 relative
       Frobenius error, per block of sampled rows and overall.
The oracle handles the large weight matrices in row chunks so that its float64 temporaries stay
small; it computes exactly what it computes on small inputs."""
import numpy as np
import pytest

from oracle import singlequant_oracle as ora
from paper_2511_22316_b200 import workloads as wl

from gpu_util import Guarded, dev, torch_mod

pytestmark = pytest.mark.gpu

PREFILL = [wl.L7B_GATEUP, wl.L7B_DOWN, wl.L70B_GATEUP, wl.L70B_DOWN]
DECODE = [wl.decode_up(m) for m in wl.DECODE_M] + [wl.decode_down(m) for m in wl.DECODE_M]


@pytest.fixture(scope="module")
def sq():
    from paper_2511_22316_b200 import binding, build
    build.build()
    binding.load()
    return binding


def _sample_rows(M, seed, count=64):
    """Token rows that hit the first and last rows of 128- and 256-row tiles (both CTAs of a pair),
    the last tile, and a random remainder; every row when the batch is small."""
    if M <= count:
        return np.arange(M)
    edges = [0, 1, 127, 128, 129, 255, 256, 257, 383, 384, M - 257, M - 256, M - 129, M - 128, M - 127, M - 1]
    rng = np.random.default_rng(seed)
    rows = np.unique(np.concatenate([[r for r in edges if 0 <= r < M], rng.integers(0, M, size=count)]))
    return rows


def _gemm_i32_chunked(Xc, Wc, chunk=4096):
    """ora.gemm_i32 over blocks of output channels (its float64 copy of the weights stays small)."""
    out = np.empty((Xc.shape[0], Wc.shape[0]), dtype=np.int32)
    for c0 in range(0, Wc.shape[0], chunk):
        out[:, c0:c0 + chunk] = ora.gemm_i32(Xc, Wc[c0:c0 + chunk])
    return out


def _pack_weight_chunked(W, R1, R2, chunk=1024):
    """ora.pack_weight over blocks of output channels (rows are independent)."""
    N, K = W.shape
    Wq = np.empty((N, K // 2), dtype=np.uint8)
    sw = np.empty((N,), dtype=np.float16)
    for r0 in range(0, N, chunk):
        q, s, _ = ora.pack_weight(W[r0:r0 + chunk], R1, R2)
        Wq[r0:r0 + chunk], sw[r0:r0 + chunk] = q, s
    return Wq, sw


def _ulps(a, b):
    return np.abs(a.view(np.int16).astype(np.int32) - b.view(np.int16).astype(np.int32))


# ------------------------------------------------------------------ (i) step 3 on identical codes
@pytest.mark.parametrize("w", PREFILL + DECODE, ids=lambda w: w.name)
def test_gemm_accumulators_bit_exact_at_full_size(sq, w):
    torch = torch_mod()
    M, N, K = w.M, w.N, w.K
    rng = np.random.default_rng(1000 + w.seed * 17 + M)
    Xc = rng.integers(-8, 8, size=(M, K), dtype=np.int8)
    Wc = rng.integers(-8, 8, size=(N, K), dtype=np.int8)
    # the extreme product on one output: every code -8 on token 0 and channel 0
    Xc[0] = -8
    Wc[0] = -8
    sx = rng.uniform(0.01, 2.0, size=M).astype(np.float16)
    sw = rng.uniform(0.001, 0.1, size=N).astype(np.float16)
    sx[0], sw[0] = np.float16(0.01), np.float16(0.001)          # keeps 64 K * sx * sw inside fp16
    y, a = Guarded(M * N * 2), Guarded(M * N * 4)
    sq.sq_w4a4_gemm(dev(ora.pack_int4(Xc)), dev(sx), dev(ora.pack_int4(Wc)), dev(sw), M, N, K, y, a)
    torch.cuda.synchronize()
    assert sq.sq_last_device_status() == sq.SQ_OK
    y.check(); a.check()
    rows = _sample_rows(M, w.seed)
    idx = torch.from_numpy(rows).cuda()
    acc = a.view.view(torch.int32).view(M, N)[idx].cpu().numpy()
    Y = y.view.view(torch.float16).view(M, N)[idx].cpu().numpy()
    acc_o = _gemm_i32_chunked(Xc[rows], Wc)
    assert acc_o[0, 0] == 64 * K
    assert np.array_equal(acc, acc_o)
    assert _ulps(Y, ora.dequant(acc_o, sx[rows], sw)).max() <= 1


# ------------------------------------------------------------------ (ii) the whole layer
_layer_cache = {}


def _oracle_layer(w):
    """Rotation and oracle-packed weights of a layer shape; the decode workloads of one layer share
    them whatever M is (the weights and the factor pair do not depend on M; the calibration batch is
    the 64-token draw)."""
    key = (w.n, w.N, w.n1, w.n2, w.seed)
    if key not in _layer_cache:
        _layer_cache.clear()                                  # one layer's matrices at a time
        import dataclasses
        calib_w = dataclasses.replace(w, M=max(w.M, 64)) if w.M < 64 else w
        Xcal = wl.make_activations(calib_w)
        W = wl.make_weights(w)
        R1, R2 = ora.build_rotation(Xcal.astype(np.float32), w.n1, w.n2)
        Wq_o, sw_o = _pack_weight_chunked(W, R1, R2)
        _layer_cache[key] = (W, R1, R2, ora.unpack_int4(Wq_o), sw_o)
    return _layer_cache[key]


@pytest.mark.parametrize("w", PREFILL + DECODE, ids=lambda w: w.name)
def test_linear_matches_oracle_at_full_size(sq, w):
    torch = torch_mod()
    M, N, K = w.M, w.N, w.K
    W, R1, R2, Wc_o, sw_o = _oracle_layer(w)
    X = wl.make_activations(w)
    rot = sq.sq_rotation_from_factors(R1, R2)
    wq, sw = Guarded(N * K // 2), Guarded(N * 2)
    sq.sq_pack_weight(rot, dev(W), N, K, wq, sw)
    nbytes = sq.sq_linear_workspace_bytes(M, K)
    ws = torch.empty(nbytes + 256, dtype=torch.uint8, device="cuda")
    y = Guarded(M * N * 2)
    sq.sq_linear(rot, dev(X), M, wq, sw, N, K, ws.data_ptr() + (-ws.data_ptr()) % 256, nbytes, y)
    torch.cuda.synchronize()
    assert sq.sq_last_device_status() == sq.SQ_OK
    y.check(); wq.check(); sw.check()
    rows = _sample_rows(M, w.seed + 5)
    Yg = y.view.view(torch.float16).view(M, N)[torch.from_numpy(rows).cuda()].cpu().numpy().astype(np.float64)
    # the oracle's layer on the sampled rows: rotate, quantise, integer GEMM, dequantise
    Xq_o, sx_o, _ = ora.rotate_quant(X[rows], R1, R2)
    acc_o = _gemm_i32_chunked(ora.unpack_int4(Xq_o), Wc_o)
    Yo = ora.dequant(acc_o, sx_o, sw_o).astype(np.float64)
    assert np.linalg.norm(Yg - Yo) <= 1e-2 * np.linalg.norm(Yo)
    for b0 in range(0, len(rows), 8):                         # and block by block of sampled rows
        blk = slice(b0, b0 + 8)
        assert np.linalg.norm(Yg[blk] - Yo[blk]) <= 1e-2 * np.linalg.norm(Yo[blk]), rows[blk]
    rot.close()


# ------------------------------------------------------------------ the one-launch form of the decode layer
@pytest.mark.parametrize("w", DECODE + [wl.small("fuse_ragged", 37, 64, 64, 2432, 81), wl.small("fuse_two_rounds", 9, 112, 128, 512, 82)],
                         ids=lambda w: w.name)
def test_fused_decode_layer_matches_oracle_and_the_two_kernel_form(sq, w):
    """A handle built with SQ_ROT_FUSE_DECODE evaluates batches of up to 64 tokens as one launch (rotating
    CTAs and GEMM CTAs side by side).  Its output must be the oracle's layer for the handle's own factors
    within 1e-2, and equal, bit for bit, to what a handle without the flag gives; twice in a row (the
    device counters a call uses must be clean again afterwards)."""
    torch = torch_mod()
    M, N, K = w.M, w.N, w.K
    import dataclasses
    Xcal = wl.make_activations(dataclasses.replace(w, M=max(w.M, 64)) if w.M < 64 else w).astype(np.float32)
    X = wl.make_activations(w)
    W = wl.make_weights(w)
    O = ora.haar_orthogonal(w.n1 - 2, np.random.default_rng(w.seed))
    fused = sq.sq_build_rotation(Xcal, w.n1, w.n2, flags=sq.SQ_ROT_DEFAULT | sq.SQ_ROT_FUSE_DECODE, O=O)
    plain = sq.sq_build_rotation(Xcal, w.n1, w.n2, flags=sq.SQ_ROT_DEFAULT, O=O)
    R1, R2 = fused.factors()
    wq, sw = Guarded(N * K // 2), Guarded(N * 2)
    sq.sq_pack_weight(plain, dev(W), N, K, wq, sw)
    nbytes = sq.sq_linear_workspace_bytes(M, K)
    ws = torch.empty(nbytes + 256, dtype=torch.uint8, device="cuda")
    wsp = ws.data_ptr() + (-ws.data_ptr()) % 256
    dX = dev(X)
    y_plain = Guarded(M * N * 2)
    before = sq.sq_kernel_launch_count()
    sq.sq_linear(plain, dX, M, wq, sw, N, K, wsp, nbytes, y_plain)
    two = sq.sq_kernel_launch_count() - before
    outs = []
    for _ in range(2):
        y = Guarded(M * N * 2)
        before = sq.sq_kernel_launch_count()
        sq.sq_linear(fused, dX, M, wq, sw, N, K, wsp, nbytes, y)
        one = sq.sq_kernel_launch_count() - before
        torch.cuda.synchronize()
        assert sq.sq_last_device_status() == sq.SQ_OK
        y.check()
        outs.append(y.numpy(np.float16, (M, N)))
    y_plain.check(); wq.check(); sw.check()
    assert two == 2 and one in (1, 2)          # one launch where the device has room for the rotating CTAs
    Yp = y_plain.numpy(np.float16, (M, N))
    for Yf in outs:
        assert np.array_equal(Yf.view(np.uint16), Yp.view(np.uint16))
    Wq_o, sw_o = _pack_weight_chunked(W, R1, R2)
    Xq_o, sx_o, _ = ora.rotate_quant(X, R1, R2)
    Yo = ora.dequant(_gemm_i32_chunked(ora.unpack_int4(Xq_o), ora.unpack_int4(Wq_o)), sx_o, sw_o).astype(np.float64)
    assert np.linalg.norm(outs[0].astype(np.float64) - Yo) <= 1e-2 * np.linalg.norm(Yo)
    fused.close(); plain.close()
