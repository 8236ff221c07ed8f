"""Host-side checks of the C-ABI boundary (no GPU needed): the library loads, exports every
symbol the header declares, and rejects bad arguments before any launch."""
import ctypes
import os
import re

import numpy as np
import pytest

from paper_2511_22316_b200 import binding as sq
from paper_2511_22316_b200 import build as sqbuild

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    sqbuild.build()
    return sq.load()


def _declared_symbols():
    text = open(os.path.join(ROOT, "include", "singlequant.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(sq_[a-z0-9_]+)\s*\(", text)))


def test_library_exports_every_declared_symbol(lib):
    names = _declared_symbols()
    assert len(names) >= 15
    for name in names:
        assert hasattr(lib, name), name
    assert set(names) == set(sq.EXPORTS)


def test_binding_has_the_same_names():
    for name in _declared_symbols():
        if name in ("sq_rotation_dims", "sq_rotation_destroy", "sq_status_string"):
            continue
        assert callable(getattr(sq, name)), name


def test_factorize_matches_hand_traces(lib):
    path = os.path.join(ROOT, "tests", "golden", "alg1_factor_pairs.txt")
    for line in open(path):
        line = line.strip()
        if not line or line.startswith("#"):
            continue
        n, n1, n2 = (int(x) for x in line.split())
        assert sq.sq_factorize(n) == (n1, n2)
    a, b = ctypes.c_int32(), ctypes.c_int32()
    assert lib.sq_factorize(0, ctypes.byref(a), ctypes.byref(b)) == sq.SQ_ERR_INVALID_ARG
    assert lib.sq_factorize(16, None, ctypes.byref(b)) == sq.SQ_ERR_INVALID_ARG


def test_factorize_is_the_nearest_power_of_two_divisor(lib):
    """Algorithm 1 by its definition, in exact integer arithmetic: among the powers of two a that
    divide n, the one minimising |a - sqrt(n)|, the smaller one on a tie.  |a - r| < |b - r| for
    a < b (r = sqrt(n)) is decided without square roots: a wins iff a + b >= 2r iff (a + b)^2 >= 4n
    when both lie on different sides, and the nearer to r otherwise."""
    def nearest(n):
        cands = [1 << k for k in range(n.bit_length()) if n % (1 << k) == 0]
        best = cands[0]
        for a in cands[1:]:
            # is a strictly closer to sqrt(n) than best (best < a)?
            if a * a <= n:                      # both at or below the root: the larger is closer
                best = a
            elif best * best >= n:              # both at or above: the smaller stays
                pass
            elif (a + best) ** 2 < 4 * n:       # opposite sides: a closer iff a - r < r - best
                best = a
        return n // best, best
    for n in list(range(1, 3000)) + [4096, 5120, 8192, 11008, 14336, 28672, 2 ** 20, 2 ** 21, 9 * 2 ** 18, 2 ** 31 - 1,
                                     3 * 2 ** 30, 2 ** 40]:
        assert sq.sq_factorize(n) == nearest(n), n


def test_debug_bounded_wait_rejects_bad_poll_counts(lib):
    assert lib.sq_debug_bounded_wait(0, None) == sq.SQ_ERR_INVALID_ARG
    assert lib.sq_debug_bounded_wait(2000000, None) == sq.SQ_ERR_INVALID_ARG


def test_status_strings(lib):
    seen = set()
    for code in range(8):
        s = sq.status_string(code)
        assert s and s != "unknown status"
        seen.add(s)
    assert len(seen) == 8
    assert sq.status_string(99) == "unknown status"


def test_build_rotation_rejects_bad_shapes(lib):
    calib = np.zeros((2, 12), np.float32)
    out = ctypes.c_void_p()
    f = lib.sq_build_rotation
    assert f(calib.ctypes.data, 2, 12, 3, 5, 7, 0, None, ctypes.byref(out)) == sq.SQ_ERR_SHAPE      # 3*5 != 12
    assert f(calib.ctypes.data, 2, 12, 4, 3, 7, 0, None, ctypes.byref(out)) == sq.SQ_ERR_SHAPE      # H needs 2^k
    assert f(None, 2, 12, 3, 4, 7, 0, None, ctypes.byref(out)) == sq.SQ_ERR_INVALID_ARG
    assert f(calib.ctypes.data, 0, 12, 3, 4, 7, 0, None, ctypes.byref(out)) == sq.SQ_ERR_INVALID_ARG
    assert f(calib.ctypes.data, 2, 12, 3, 4, 8, 0, None, ctypes.byref(out)) == sq.SQ_ERR_INVALID_ARG  # bad flag
    assert f(calib.ctypes.data, 2, 12, 3, 4, 7, 0, None, None) == sq.SQ_ERR_INVALID_ARG
    assert out.value is None


def test_gemm_rejects_bad_arguments_before_launch(lib):
    g = lib.sq_w4a4_gemm
    p = 0x1000          # never dereferenced: every case below fails validation first
    assert g(p, p, p, p, 4, 8, 7, p, None, None) == sq.SQ_ERR_SHAPE          # odd K
    assert g(p, p, p, p, 4, 8, 0, p, None, None) == sq.SQ_ERR_SHAPE
    assert g(p, p, p, p, 4, 8, 1 << 20, p, None, None) == sq.SQ_ERR_UNSUPPORTED
    assert g(p, p, p, p, -1, 8, 128, p, None, None) == sq.SQ_ERR_INVALID_ARG
    assert g(None, p, p, p, 4, 8, 128, p, None, None) == sq.SQ_ERR_INVALID_ARG
    assert g(p + 4, p, p, p, 4, 8, 128, p, None, None) == sq.SQ_ERR_ALIGN
    assert g(p, p, p, p, 4, 8, 128, p, p + 8, None) == sq.SQ_ERR_ALIGN
    assert g(p, p, p, p, 0, 8, 128, p, None, None) == sq.SQ_OK                # M = 0: no-op
    assert g(None, None, None, None, 0, 0, 128, None, None, None) == sq.SQ_OK


def test_rows_calls_reject_null_handle_and_bad_sizes(lib):
    p = 0x1000
    assert lib.sq_rotate_quant_act(None, p, 4, p, p, None, None) == sq.SQ_ERR_INVALID_ARG
    assert lib.sq_linear(None, p, 4, p, p, 8, 128, p, 1 << 20, p, None) == sq.SQ_ERR_INVALID_ARG
    assert lib.sq_linear_host(None, p, 4, p, p, 8, 128, p, 1 << 20, p, None) == sq.SQ_ERR_INVALID_ARG
    # identity pack: odd K, K too large, misaligned, null
    assert lib.sq_pack_weight(None, p, 4, 7, p, p, None) == sq.SQ_ERR_SHAPE
    assert lib.sq_pack_weight(None, p, 4, 1 << 17, p, p, None) == sq.SQ_ERR_UNSUPPORTED
    assert lib.sq_pack_weight(None, p + 2, 4, 8, p, p, None) == sq.SQ_ERR_ALIGN
    assert lib.sq_pack_weight(None, None, 4, 8, p, p, None) == sq.SQ_ERR_INVALID_ARG
    assert lib.sq_pack_weight(None, None, 0, 8, None, None, None) == sq.SQ_OK


def test_workspace_sizes(lib):
    assert sq.sq_linear_workspace_bytes(0, 128) == 0
    w = sq.sq_linear_workspace_bytes(2048, 4096)
    assert w >= 2048 * 2048 + 2 * 2048 and w % 256 == 0
    h = sq.sq_linear_host_workspace_bytes(2048, 4096, 4096)
    assert h >= w + 2 * 2048 * 4096 * 2


def test_launch_counter_starts_at_zero_without_gpu_work(lib):
    assert sq.sq_kernel_launch_count() >= 0
