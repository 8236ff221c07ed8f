"""Boundary behaviour that needs a device: arguments are refused before anything is queued, the
bounded-wait status path reports a wait that ran out and leaves the context usable, and the plain
integer GEMM takes more token rows than a grid's y extent."""
import ctypes

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


def _small_layer(sq, seed=71):
    w = wl.small("bnd", 24, 64, 64, 264, seed)
    X, W = wl.make_layer(w)
    R1, R2 = ora.build_rotation(X.astype(np.float32), w.n1, w.n2)
    rot = sq.sq_rotation_from_factors(R1, R2)
    wq, sw = Guarded(w.N * w.n // 2), Guarded(w.N * 2)
    sq.sq_pack_weight(rot, dev(W), w.N, w.n, wq, sw)
    torch_mod().cuda.synchronize()
    return w, X, W, R1, R2, rot, wq, sw


def test_layer_calls_refuse_bad_gemm_arguments_before_any_launch(sq):
    """A valid handle and valid activations, but a NULL or misaligned weight / output pointer: the
    error comes back with nothing launched (sq_linear, sq_linear_static and sq_linear_host)."""
    torch = torch_mod()
    lib = sq.load()
    w, X, W, R1, R2, rot, wq, sw = _small_layer(sq)
    M, N, K = w.M, w.N, w.n
    dX = dev(X)
    y = Guarded(M * N * 2)
    nbytes = sq.sq_linear_workspace_bytes(M, K)
    ws = torch.empty(nbytes + 256, dtype=torch.uint8, device="cuda")
    wsp = ws.data_ptr() + (-ws.data_ptr()) % 256
    hbytes = sq.sq_linear_host_workspace_bytes(M, N, K)
    hws = torch.empty(hbytes + 256, dtype=torch.uint8, device="cuda")
    hwsp = hws.data_ptr() + (-hws.data_ptr()) % 256
    Xh = torch.from_numpy(X).pin_memory()
    Yh = torch.empty((M, N), dtype=torch.float16).pin_memory()
    h, st = rot.handle, None
    good = dict(X=dX.data_ptr(), Wq=wq.data_ptr(), sw=sw.data_ptr(), Y=y.data_ptr())
    cases = [("Wq", None, sq.SQ_ERR_INVALID_ARG), ("sw", None, sq.SQ_ERR_INVALID_ARG),
             ("Y", None, sq.SQ_ERR_INVALID_ARG), ("Wq", good["Wq"] + 4, sq.SQ_ERR_ALIGN),
             ("Y", good["Y"] + 2, sq.SQ_ERR_ALIGN), ("X", good["X"] + 8, sq.SQ_ERR_ALIGN)]
    torch.cuda.synchronize()
    before = sq.sq_kernel_launch_count()
    for name, bad, code in cases:
        a = dict(good)
        a[name] = bad
        assert lib.sq_linear(h, a["X"], M, a["Wq"], a["sw"], N, K, wsp, nbytes, a["Y"], st) == code, name
        assert lib.sq_linear_static(h, a["X"], M, a["Wq"], a["sw"], N, K, a["Y"], st) == code, name
        if name in ("Wq", "sw"):
            assert lib.sq_linear_host(h, Xh.data_ptr(), M, a["Wq"], a["sw"], N, K, hwsp, hbytes, Yh.data_ptr(), st) == code
    assert lib.sq_linear(h, good["X"], M, good["Wq"], good["sw"], N, K + 2, wsp, nbytes, good["Y"], st) == sq.SQ_ERR_SHAPE
    assert lib.sq_linear(h, good["X"], M, good["Wq"], good["sw"], N, K, wsp, 16, good["Y"], st) == sq.SQ_ERR_NOMEM
    assert sq.sq_kernel_launch_count() == before
    # and the same buffers with good arguments still give the layer
    sq.sq_linear(rot, dX, M, wq, sw, N, K, wsp, nbytes, y)
    torch.cuda.synchronize()
    assert sq.sq_last_device_status() == sq.SQ_OK
    y.check()
    Yo = ora.linear(X, W, R1, R2).astype(np.float64)
    Yg = y.numpy(np.float16, (M, N)).astype(np.float64)
    assert np.linalg.norm(Yg - Yo) <= 1e-2 * np.linalg.norm(Yo)
    rot.close()


def test_handle_of_another_device_is_refused(sq):
    torch = torch_mod()
    if torch.cuda.device_count() < 2:
        pytest.skip("needs two devices")
    w, X, W, R1, R2, rot, wq, sw = _small_layer(sq)
    lib = sq.load()
    before = sq.sq_kernel_launch_count()
    with torch.cuda.device(1):
        x1 = torch.zeros((w.M, w.n), dtype=torch.float16, device="cuda:1")
        q1 = torch.zeros((w.M, w.n // 2), dtype=torch.uint8, device="cuda:1")
        s1 = torch.zeros((w.M,), dtype=torch.float16, device="cuda:1")
        code = lib.sq_rotate_quant_act(rot.handle, x1.data_ptr(), w.M, q1.data_ptr(), s1.data_ptr(), None, None)
    assert code == sq.SQ_ERR_INVALID_ARG
    assert sq.sq_kernel_launch_count() == before
    rot.close()


def test_bounded_wait_that_runs_out_is_reported_and_leaves_the_context_usable(sq):
    """The diagnostic kernel waits on a barrier nothing completes, with the library's own bounded
    wait and nothing in flight; after a few thousand polls it gives up.  The status call reports
    SQ_ERR_TIMEOUT once, then SQ_OK, and an ordinary layer call afterwards is correct."""
    torch = torch_mod()
    torch.cuda.synchronize()
    assert sq.sq_last_device_status() == sq.SQ_OK
    sq.sq_debug_bounded_wait(3000)
    assert sq.sq_last_device_status() == sq.SQ_ERR_TIMEOUT
    assert sq.sq_last_device_status() == sq.SQ_OK
    w, X, W, R1, R2, rot, wq, sw = _small_layer(sq, seed=72)
    M, N, K = w.M, w.N, w.n
    nbytes = sq.sq_linear_workspace_bytes(M, K)
    ws = torch.empty(nbytes + 256, dtype=torch.uint8, device="cuda")
    y = Guarded(M * N * 2)
    sq.sq_linear(rot, dev(X), M, wq, sw, N, K, ws.data_ptr() + (-ws.data_ptr()) % 256, nbytes, y)
    torch.cuda.synchronize()
    assert sq.sq_last_device_status() == sq.SQ_OK
    y.check()
    Yo = ora.linear(X, W, R1, R2).astype(np.float64)
    Yg = y.numpy(np.float16, (M, N)).astype(np.float64)
    assert np.linalg.norm(Yg - Yo) <= 1e-2 * np.linalg.norm(Yo)
    rot.close()


def test_plain_integer_gemm_takes_more_rows_than_a_grid_has_y_blocks(sq):
    """K = 6 is not a multiple of 128, so the plain integer kernel runs; 70001 token rows exceed the
    65535 blocks of a grid's y extent.  Accumulators are exact on every row."""
    M, N, K = 70001, 5, 6
    rng = np.random.default_rng(123)
    Xc = rng.integers(-8, 8, size=(M, K)).astype(np.int8)
    Wc = rng.integers(-8, 8, size=(N, K)).astype(np.int8)
    sx = rng.uniform(0.01, 2.0, size=M).astype(np.float16)
    sw = rng.uniform(0.001, 0.1, size=N).astype(np.float16)
    y, a = Guarded(M * N * 2), Guarded(M * N * 4)
    sq.sq_w4a4_gemm(dev(ora.pack_int4(Xc)), dev(sx), dev(ora.pack_int4(Wc)), dev(sw), M, N, K, y, a)
    torch_mod().cuda.synchronize()
    assert sq.sq_last_device_status() == sq.SQ_OK
    y.check(); a.check()
    acc_o = ora.gemm_i32(Xc, Wc)
    assert np.array_equal(a.numpy(np.int32, (M, N)), acc_o)
    Yo = ora.dequant(acc_o, sx, sw)
    Yg = y.numpy(np.float16, (M, N))
    ulps = np.abs(Yg.view(np.int16).astype(np.int32) - Yo.view(np.int16).astype(np.int32))
    assert ulps.max() <= 1
