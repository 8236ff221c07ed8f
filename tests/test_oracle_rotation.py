"""Pins for the oracle's rotation construction and application (CPU only).

Each test checks the oracle against something the paper or the mathematics fixes, not
against itself: closed forms, explicit dense matrices built by loops, brute force."""
import math
import os

import numpy as np
import pytest

from oracle import singlequant_oracle as ora
from paper_2511_22316_b200 import workloads as wl

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def _rows(name):
    out = []
    with open(os.path.join(GOLDEN, name)) as f:
        for line in f:
            line = line.strip()
            if line and not line.startswith("#"):
                out.append([float(x) for x in line.split()])
    return out


def _dense_kron_loops(R1, R2):
    """K[(p, q), (p', q')] = R1[p, p'] * R2[q, q'] written out entry by entry."""
    n1, n2 = R1.shape[0], R2.shape[0]
    K = np.zeros((n1 * n2, n1 * n2))
    for p in range(n1):
        for q in range(n2):
            for pp in range(n1):
                for qq in range(n2):
                    K[p * n2 + q, pp * n2 + qq] = R1[p, pp] * R2[q, qq]
    return K


def _random_orthogonal(n, seed):
    rng = np.random.default_rng(seed)
    Q, _ = np.linalg.qr(rng.standard_normal((n, n)))
    return Q


# ---------------------------------------------------------------- Alg. 1 (P11)
def test_factorize_hand_traces():
    for n, n1, n2 in _rows("alg1_factor_pairs.txt"):
        assert ora.factorize(int(n)) == (int(n1), int(n2)), n


def test_factorize_properties():
    for n in list(range(1, 300)) + [4096, 5120, 11008, 14336, 28672, 8192]:
        n1, n2 = ora.factorize(n)
        assert n1 * n2 == n
        assert n2 & (n2 - 1) == 0
        # no other power-of-two divisor is strictly closer to sqrt(n)
        a = 1
        while a <= n:
            if n % a == 0:
                assert abs(n2 - math.sqrt(n)) <= abs(a - math.sqrt(n))
            a *= 2


# ---------------------------------------------------------------- Lemma 1 (P3)
def test_lemma1_closed_form():
    for a, b, expect in _rows("lemma1_equalisation.txt"):
        th = ora.equalizing_angle(a, b)
        G = ora.givens(2, 0, 1, th)
        out = np.array([a, b]) @ G
        assert np.allclose(out, [expect, expect], rtol=0, atol=1e-9 * max(1.0, expect))
        # the proof's expansion: V G(theta) = (a cos + b sin, b cos - a sin)
        assert math.isclose(out[0], a * math.cos(th) + b * math.sin(th), abs_tol=1e-9)
        assert math.isclose(out[1], b * math.cos(th) - a * math.sin(th), abs_tol=1e-9)


def test_lemma1_is_the_minimum_over_a_grid():
    rng = np.random.default_rng(5)
    for _ in range(20):
        a, b = rng.standard_normal(2) * 10
        r = math.hypot(a, b)
        best = min(np.max(np.abs(np.array([a, b]) @ ora.givens(2, 0, 1, t)))
                   for t in np.linspace(-math.pi, math.pi, 2001))
        assert best >= r / math.sqrt(2) - 1e-9
        assert best <= r / math.sqrt(2) * (1 + 2e-3)     # grid step pi/1000
        # reflections (the other component of O(2)) cannot do better either
        F = np.diag([1.0, -1.0])
        best_f = min(np.max(np.abs(np.array([a, b]) @ F @ ora.givens(2, 0, 1, t)))
                     for t in np.linspace(-math.pi, math.pi, 2001))
        assert best_f >= r / math.sqrt(2) - 1e-9


def test_givens_embedding():
    G = ora.givens(5, 1, 3, 0.3)
    assert np.allclose(G.T @ G, np.eye(5), atol=1e-15)
    assert G[1, 1] == pytest.approx(math.cos(0.3)) and G[3, 3] == pytest.approx(math.cos(0.3))
    assert G[1, 3] == pytest.approx(-math.sin(0.3)) and G[3, 1] == pytest.approx(math.sin(0.3))
    mask = np.ones((5, 5), bool)
    mask[np.ix_([1, 3], [1, 3])] = False
    assert np.array_equal(G[mask], np.eye(5)[mask])


# ---------------------------------------------------------------- ART (P4)
@pytest.mark.parametrize("steps", [2, 3, 8, 33])
def test_repeated_art_steps_equalise_one_pair_each(steps):
    """Paragraph "Effect of ART Steps": every further step is a rotation in the plane of the
    current (outlier, minimum) pair that leaves both at r/sqrt(2) (Lemma 1) and touches nothing
    else; the product stays orthogonal, keeps the norm and never raises the column's absmax."""
    rng = np.random.default_rng(steps)
    n = 24
    c = rng.standard_normal(n)
    c[5] = 800.0
    c[11] = -300.0
    O = ora.haar_orthogonal(n - 2, rng)
    prev = ora.art_matrix_steps(c, O, steps - 1)
    full = ora.art_matrix_steps(c, O, steps)
    assert np.allclose(full.T @ full, np.eye(n), atol=1e-12)
    before, after = prev @ c, full @ c
    i, j = ora.art_indices(before)
    r = math.hypot(before[i], before[j])
    assert abs(after[i] - r / math.sqrt(2)) < 1e-9 and abs(after[j] - r / math.sqrt(2)) < 1e-9
    others = [k for k in range(n) if k not in (i, j)]
    assert np.allclose(after[others], before[others], atol=1e-12)
    assert abs(np.linalg.norm(after) - np.linalg.norm(c)) < 1e-9
    assert np.max(np.abs(after)) <= np.max(np.abs(before)) + 1e-12
    # one step is the plain ART
    assert np.array_equal(ora.art_matrix_steps(c, O, 1), ora.art_matrix(c, O))


def test_repeated_art_steps_lower_the_massive_outlier_further():
    c = np.array([800.0, 0.3, -1.0, 2.0, 0.5, -0.7, 1.5, 0.1])
    peaks = [np.max(np.abs(ora.art_matrix_steps(c, None, k) @ c)) for k in (1, 2, 3, 4)]
    assert abs(peaks[0] - math.hypot(800.0, 0.1) / math.sqrt(2)) < 1e-9      # (800, 0.1): smallest magnitude is index 7
    assert all(b <= a + 1e-12 for a, b in zip(peaks, peaks[1:]))
    # two equal halves of 800/sqrt(2) are each halved again against a small entry: 800/2 after three steps
    assert abs(peaks[1] - peaks[0]) < 1e-9 and abs(peaks[2] - 400.0) < 1e-2
    R1, R2 = ora.build_rotation(np.tile(c, (2, 4)).reshape(2, 32), 8, 4, art_steps=3)
    assert np.allclose(R1.astype(np.float64).T @ R1.astype(np.float64), np.eye(8), atol=1e-6)


@pytest.mark.parametrize("n", [2, 3, 8, 16, 64])
def test_art_equalises_outlier_pair(n):
    rng = np.random.default_rng(n)
    c = rng.standard_normal(n)
    i = int(rng.integers(n))
    c[i] = 800.0 * (-1) ** n
    ii, jj = ora.art_indices(c)
    assert ii == i
    others = [k for k in range(n) if k != i]
    assert abs(c[jj]) == min(abs(c[k]) for k in others)
    O = _random_orthogonal(n - 2, 100 + n) if n > 2 else None
    RA = ora.art_matrix(c, O)
    assert np.allclose(RA.T @ RA, np.eye(n), atol=1e-12)
    out = RA @ c
    r = math.hypot(c[ii], c[jj])
    assert out[0] == pytest.approx(r / math.sqrt(2), rel=1e-12)
    assert out[1] == pytest.approx(r / math.sqrt(2), rel=1e-12)
    rest = np.array([c[k] for k in range(n) if k not in (ii, jj)])
    assert np.linalg.norm(out[2:]) == pytest.approx(np.linalg.norm(rest), rel=1e-12, abs=1e-12)
    # the outlier's magnitude drops by sqrt(2) and nothing else grows beyond the rest's norm
    assert np.max(np.abs(out[:2])) < abs(c[i]) * 0.7072 + abs(c[jj])


def test_art_without_O_only_touches_the_pair():
    c = np.array([0.5, -800.0, 0.25, 3.0, -0.01, 7.0])
    RA = ora.art_matrix(c, None)
    out = RA @ c
    # i = 1 (outlier), j = 4 (smallest magnitude); the others keep their order
    assert ora.art_indices(c) == (1, 4)
    assert np.allclose(out[2:], [0.5, 0.25, 3.0, 7.0])
    r = math.hypot(800.0, 0.01)
    assert np.allclose(out[:2], [r / math.sqrt(2)] * 2)


# ---------------------------------------------------------------- URT (P5, P6)
@pytest.mark.parametrize("n", [2, 3, 5, 16, 64, 172])
def test_map_to_e1(n):
    rng = np.random.default_rng(n + 7)
    V = rng.standard_normal(n) * 3
    R, count = ora.map_to_e1(V)
    assert count == n - 1
    assert np.allclose(R.T @ R, np.eye(n), atol=1e-12)
    e1 = np.zeros(n)
    e1[0] = np.linalg.norm(V)
    assert np.allclose(V @ R, e1, atol=1e-10)


@pytest.mark.parametrize("n", [2, 5, 16, 64, 112])
def test_urt_maps_V_to_uniform_target(n):
    rng = np.random.default_rng(n + 11)
    V = rng.standard_normal(n)
    V[rng.integers(n)] *= 20
    RU = ora.urt_matrix(V)
    assert np.allclose(RU.T @ RU, np.eye(n), atol=1e-12)
    U = V @ RU
    assert np.linalg.norm(U) == pytest.approx(np.linalg.norm(V), rel=1e-12)
    assert np.array_equal(np.argsort(U, kind="stable"), np.argsort(V, kind="stable"))
    s = np.sort(U)
    gaps = np.diff(s)
    assert np.allclose(gaps, gaps[0], rtol=1e-8, atol=1e-12)
    # closed form of the template: q_k = (2k-n-1)/n, ||q||^2 = (n^2-1)/(3n)
    k = np.arange(1, n + 1)
    q = (2 * k - n - 1) / n
    assert np.dot(q, q) == pytest.approx((n * n - 1) / (3 * n), rel=1e-12)
    assert np.allclose(s, np.linalg.norm(V) / math.sqrt((n * n - 1) / (3 * n)) * q, atol=1e-9)
    assert s[0] == pytest.approx(-s[-1], rel=1e-9)      # centred
    assert np.allclose(ora.uniform_target(V), U, atol=1e-9)


def test_urt_degenerate():
    assert np.array_equal(ora.urt_matrix(np.zeros(4)), np.eye(4))
    assert np.array_equal(ora.urt_matrix(np.array([3.0])), np.eye(1))
    V = np.array([1.0, 1.0, 1.0])                      # ties: broken by index, still a rotation
    RU = ora.urt_matrix(V)
    assert np.allclose(RU.T @ RU, np.eye(3), atol=1e-12)
    assert np.allclose(V @ RU, ora.uniform_target(V), atol=1e-12)


@pytest.mark.parametrize("scale", [1.0, 1e6, 1e-6])
def test_near_ties_in_outlier_minimum_and_rank(scale):
    """Magnitudes within a RELATIVE 1e-9 count as tied and the lowest index wins (ART's outlier and
    minimum; URT's rank order keeps the index order); magnitudes 1e-6 apart do not tie.  Expected
    indices and targets are written out by hand; scaling the vector by 1e6 or 1e-6 must change
    nothing (an absolute tolerance would flip the first case at 1e6 and the second at 1e-6)."""
    e12, e6 = 1e-12, 1e-6
    # |c_1| = 5 and |c_2| = 5(1 + 1e-12) tie for the outlier -> i = 1;
    # |c_0| = 0.5(1 + 1e-12) and |c_3| = 0.5 tie for the minimum -> j = 0
    c = scale * np.array([0.5 * (1 + e12), -5.0, 5.0 * (1 + e12), 0.5, 2.0])
    assert ora.art_indices(c) == (1, 0)
    # 1e-6 apart: the larger one is the outlier (i = 2), the smaller one the minimum (j = 3)
    c = scale * np.array([0.5 * (1 + e6), -5.0, 5.0 * (1 + e6), 0.5, 2.0])
    assert ora.art_indices(c) == (2, 3)
    # URT target for n = 4: q = (-3, -1, 1, 3)/4, ||q||^2 = 5/4.
    # V = (1 + 1e-12, 3, 1, -2): entries 0 and 2 tie, so the ascending order is 3, 0, 2, 1 (index order
    # inside the tie) and U = ||V||/||q|| * (-1/4, 3/4, 1/4, -3/4) with ||V||^2 = 15 (+ 2e-12).
    V = scale * np.array([1.0 * (1 + e12), 3.0, 1.0, -2.0])
    s = scale * math.sqrt(15.0 / 1.25)
    assert np.allclose(ora.uniform_target(V), s * np.array([-0.25, 0.75, 0.25, -0.75]), rtol=1e-11, atol=0)
    # 1e-6 apart: entry 2 (1.0) now ranks below entry 0 -> order 3, 2, 0, 1
    V = scale * np.array([1.0 * (1 + e6), 3.0, 1.0, -2.0])
    s = scale * math.sqrt((15.0 + 2e-6 + 1e-12) / 1.25)
    assert np.allclose(ora.uniform_target(V), s * np.array([0.25, 0.75, -0.25, -0.75]), rtol=1e-11, atol=0)


# ---------------------------------------------------------------- Hadamard (P7)
@pytest.mark.parametrize("n", [1, 2, 4, 32, 128])
def test_hadamard(n):
    H = ora.hadamard(n)
    assert np.allclose(np.abs(H), 1 / math.sqrt(n))
    assert np.allclose(H.T @ H, np.eye(n), atol=1e-12)
    if n >= 2:
        assert np.array_equal(np.sign(H[:2, :2]), [[1, 1], [1, -1]])
    with pytest.raises(ValueError):
        ora.hadamard(12)


# ---------------------------------------------------------------- overall R (P1)
@pytest.mark.parametrize("w", [wl.TINY, wl.small("s1", 5, 3, 4, 8, 3), wl.small("s2", 7, 12, 8, 8, 4),
                               wl.small("s3", 4, 2, 2, 8, 5), wl.small("s4", 3, 1, 8, 8, 6)])
@pytest.mark.parametrize("flags", [0, 1, 2, 4, 7])
def test_build_rotation_orthogonal(w, flags):
    X = wl.make_activations(w).astype(np.float32)
    R1, R2, R1d, R2d = ora.build_rotation(X, w.n1, w.n2, flags=flags, seed=3, return_f64=True)
    assert R1.dtype == np.float32 and R2.dtype == np.float32
    assert np.allclose(R1d.T @ R1d, np.eye(w.n1), atol=1e-12)
    assert np.allclose(R2d.T @ R2d, np.eye(w.n2), atol=1e-12)
    assert np.allclose(R1.astype(np.float64).T @ R1.astype(np.float64), np.eye(w.n1), atol=1e-6)
    assert np.allclose(R2.astype(np.float64).T @ R2.astype(np.float64), np.eye(w.n2), atol=1e-6)
    if w.n <= 96:
        R = _dense_kron_loops(R1d, R2d)
        assert np.allclose(R.T @ R, np.eye(w.n), atol=1e-12)
    if flags == 0:
        assert np.array_equal(R1d, np.eye(w.n1)) and np.array_equal(R2d, np.eye(w.n2))


def test_build_rotation_structure_on_tiny_config():
    """R1 = (R1^U R^A)^T and R2 = H R2^U, checked by undoing the factors: with URT off, R1^T is
    the ART matrix of the chosen column; with ART and URT off, R2 is exactly H."""
    w = wl.TINY
    X = wl.make_activations(w).astype(np.float64)
    # token 0 holds the +-800 outliers: channel 3 -> (p, q) = (0, 3); channel 77 -> (2, 13)
    A = X[0].reshape(w.n1, w.n2)
    assert abs(A[0, 3]) == 800 and abs(A[2, 13]) == 800
    O = _random_orthogonal(w.n1 - 2, 9)
    _, _, R1d, R2d = ora.build_rotation(X, w.n1, w.n2, flags=ora.ROT_ART, O=O, return_f64=True)
    c = A[:, 3]
    assert np.allclose(R1d.T, ora.art_matrix(c, O), atol=1e-14)
    assert np.array_equal(R2d, np.eye(w.n2))
    _, _, R1d, R2d = ora.build_rotation(X, w.n1, w.n2, flags=ora.ROT_HADAMARD, return_f64=True)
    assert np.array_equal(R1d, np.eye(w.n1))
    assert np.allclose(R2d, ora.hadamard(w.n2))
    # full build: the calibration column goes to the uniform target of its ART image, and the
    # selected row goes to the uniform target of its Hadamard image
    _, _, R1d, R2d = ora.build_rotation(X, w.n1, w.n2, flags=7, O=O, return_f64=True)
    cp = ora.art_matrix(c, O) @ c
    assert np.allclose(R1d.T @ c, ora.uniform_target(cp), atol=1e-8)
    Ap = R1d.T @ A
    row = int(np.argmax(np.max(np.abs(Ap), axis=1)))
    H = ora.hadamard(w.n2)
    assert np.allclose(Ap[row] @ R2d, ora.uniform_target(Ap[row] @ H), atol=1e-8)
    # massive outlier smoothed: the token's absmax falls by far more than sqrt(2)
    Z = ora.rotate(X[:1], R1d, R2d)
    assert np.max(np.abs(Z)) < 800 / 4


# ---------------------------------------------------------------- Kronecker identity (P2)
@pytest.mark.parametrize("n1,n2", [(3, 4), (2, 2), (5, 8), (16, 32), (1, 4), (4, 1)])
def test_kronecker_identity_against_dense(n1, n2):
    rng = np.random.default_rng(n1 * 100 + n2)
    R1 = _random_orthogonal(n1, 1) if n1 > 1 else np.ones((1, 1))
    R2 = _random_orthogonal(n2, 2) if n2 > 1 else np.ones((1, 1))
    # non-symmetric, non-orthogonal factors too: the identity is pure algebra
    if n1 > 1:
        R1 = R1 + 0.1 * rng.standard_normal((n1, n1))
    K = _dense_kron_loops(R1, R2)
    assert np.allclose(K, ora.kron_dense(R1, R2), atol=0)
    V = rng.standard_normal((3, n1 * n2))
    Z = ora.rotate(V, R1, R2)
    assert np.allclose(Z, V @ K, atol=1e-12)
    for t in range(3):
        Vm = V[t].reshape(n1, n2)
        # v (R1 (x) R2) = rvec(R1^T V_mat R2)
        assert np.allclose(Z[t], (R1.T @ Vm @ R2).reshape(-1), atol=1e-12)
        # (R1 (x) R2) v = rvec(R1 V_mat R2^T)
        assert np.allclose(K @ V[t], (R1 @ Vm @ R2.T).reshape(-1), atol=1e-12)
    # a transposed operand or swapped factor would be caught
    if n1 > 1 and n2 > 1:
        assert not np.allclose(Z[0], (R1 @ V[0].reshape(n1, n2) @ R2).reshape(-1), atol=1e-6)


# ---------------------------------------------------------------- invariances (P8, P9)
@pytest.mark.parametrize("w", [wl.TINY,
                               wl.small("qkvo_small", 24, 64, 64, 40, 1),
                               wl.small("down7b_small", 8, 172, 64, 24, 2),
                               wl.small("down8b_small", 6, 112, 128, 16, 3),
                               wl.small("up70b_small", 6, 64, 128, 16, 4),
                               wl.small("down70b_small", 3, 224, 128, 8, 4)])
def test_rotation_invariance_before_quantisation(w):
    X, W = wl.make_layer(w)
    R1, R2 = ora.build_rotation(X.astype(np.float32), w.n1, w.n2, seed=w.seed)
    ZX = ora.rotate(X, R1, R2)
    ZW = ora.rotate(W, R1, R2)
    Y = ora.linear_fp(X, W)
    Yr = ZX @ ZW.T
    assert np.linalg.norm(Yr - Y) / np.linalg.norm(Y) < 1e-4
    assert np.max(np.abs(Yr - Y)) / np.max(np.abs(Y)) < 1e-4
    Xd = X.astype(np.float64)
    assert np.allclose(np.linalg.norm(ZX, axis=1), np.linalg.norm(Xd, axis=1), rtol=1e-5)
    G, Gr = Xd[:8] @ Xd[:8].T, ZX[:8] @ ZX[:8].T
    assert np.allclose(G, Gr, rtol=1e-5, atol=1e-5 * np.max(np.abs(G)))
