"""sq_linear_static: the layer evaluated with the library's built-in scratch instead of a caller
workspace, for callers that cannot allocate device memory where they run the layer (a serving
loop that must stay out of cudaMalloc, a plugin that gets tensors but no allocator from its host
framework).  Its output must be the one sq_linear gives with an ordinary workspace.

The file name sorts last on purpose: a run that stops at the first failure has then already run
every other test.  The test passes alone in a fresh process and after the other tests."""
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


def _layer(sq, w):
    X, W = wl.make_layer(w)
    R1, R2 = ora.build_rotation(X.astype(np.float32), w.n1, w.n2)
    rot = sq.sq_rotation_from_factors(R1, R2)
    wq, sw = Guarded(w.N * w.n // 2), Guarded(w.N * 2)
    sq.sq_pack_weight(rot, dev(W), w.N, w.n, wq, sw)
    torch_mod().cuda.synchronize()
    return X, W, R1, R2, rot, wq, sw


def test_static_scratch_matches_workspace_path_twice_in_a_row(sq):
    torch = torch_mod()
    # two different layers back to back: the second call finds the first call's bytes in the scratch
    cases = [wl.small("na1", 300, 64, 64, 264, 61), wl.small("na2", 70, 112, 128, 136, 62)]
    for w in cases:
        X, W, R1, R2, rot, wq, sw = _layer(sq, w)
        M, N, K = w.M, w.N, w.n
        dX = dev(X)
        nbytes = sq.sq_linear_workspace_bytes(M, K)
        assert nbytes <= sq.SQ_LINEAR_STATIC_SCRATCH_BYTES
        ws = torch.empty(nbytes + 256, dtype=torch.uint8, device="cuda")
        off = (-ws.data_ptr()) % 256
        y_ref, y_new = Guarded(M * N * 2), Guarded(M * N * 2)
        sq.sq_linear(rot, dX, M, wq, sw, N, K, ws.data_ptr() + off, nbytes, y_ref)
        sq.sq_linear_static(rot, dX, M, wq, sw, N, K, y_new)
        torch.cuda.synchronize()
        assert sq.sq_last_device_status() == sq.SQ_OK
        y_ref.check(); y_new.check()
        a = y_ref.numpy(np.float16, (M, N)).astype(np.float64)
        b = y_new.numpy(np.float16, (M, N)).astype(np.float64)
        # same kernels on the same inputs: the tolerance of the layer tests, and in fact equal
        assert np.linalg.norm(a - b) <= 1e-2 * np.linalg.norm(a)
        assert np.array_equal(a, b)
        # and both are the layer the oracle defines
        Yo = ora.linear(X, W, R1, R2).astype(np.float64)
        assert np.linalg.norm(b - Yo) <= 1e-2 * np.linalg.norm(Yo)
        rot.close()


def test_static_scratch_rejects_problems_beyond_its_size(sq):
    w = wl.small("na3", 4, 64, 64, 8, 63)
    X, W, R1, R2, rot, wq, sw = _layer(sq, w)
    M_big = sq.SQ_LINEAR_STATIC_SCRATCH_BYTES // (w.n // 2) + 1     # packed rows alone exceed the array
    before = sq.sq_kernel_launch_count()
    with pytest.raises(sq.SingleQuantError) as e:
        sq.sq_linear_static(rot, dev(X), M_big, wq, sw, w.N, w.n, None)
    assert e.value.code == sq.SQ_ERR_UNSUPPORTED
    assert sq.sq_kernel_launch_count() == before
    sq.sq_linear_static(rot, None, 0, None, None, w.N, w.n, None)    # empty batch: a no-op
    assert sq.sq_kernel_launch_count() == before
    rot.close()
