"""CPU oracle for the SingleQuant W4A4 linear hot path.  TEST INFRASTRUCTURE ONLY.

Plain, slow, float64 numpy written from the paper's statement of the method.  It shares no
code with the CUDA path and must never be imported by the product package: only tests, the
smoke check and the benchmark's CPU-baseline leg may use it.

Every function cites the passage of the paper it follows.  Where the method has a plain
definition (the Kronecker rotation, the integer GEMM) the oracle IS that definition; where it
is a construction (ART, URT, the quantiser) the oracle takes the paper's steps in the paper's
order and notation.

Conventions (paper, Section "SingleQuant", paragraph "Kronecker Product"):
  * activations X in R^{T x n}, one token per row; weights are handled as rows of W^T in
    R^{C x n} (one output channel per row);
  * R = R1 (x) R2 with R1 in R^{n1 x n1}, R2 in R^{n2 x n2}, n = n1*n2;
  * rvec = row-major flattening: channel c of a token is entry (p, q) = (c // n2, c % n2)
    of the reshaped token V_mat in R^{n1 x n2};
  * V (R1 (x) R2) = rvec(R1^T V_mat R2)                                   (Eq. "eq18").

Parity status: every function below is pinned by tests/test_oracle_*.py against closed forms,
brute force or library routines (the weight-only variant and the grouped layer at the end of the
file by tests/test_oracle_weight_only.py).  Agreement with the authors' own R1, R2 (which depend on
choices the paper leaves open: the calibration vector, the random block O, the order of the
Givens chain) is "parity unpinned": no code, weights or data of theirs is available.
"""
from __future__ import annotations

import math
from typing import Optional, Tuple

import numpy as np

ROT_ART = 1
ROT_URT = 2
ROT_HADAMARD = 4
ROT_DEFAULT = ROT_ART | ROT_URT | ROT_HADAMARD


# --------------------------------------------------------------------------------------
# Algorithm 1: Kronecker dimension factorisation
# --------------------------------------------------------------------------------------
def factorize(n: int) -> Tuple[int, int]:
    """Algorithm 1 ("Kronecker Dimension Factorization"): n2 is the power of two dividing n
    that is closest to sqrt(n) (the first one found wins ties: the comparison is strict),
    n1 = n / n2.  Returns (n1, n2)."""
    if n < 1:
        raise ValueError("n must be >= 1")
    root = math.sqrt(n)
    n2 = 1
    k_max = int(math.floor(math.log2(n)))
    for k in range(0, k_max + 1):
        a = 2 ** k
        if n % a != 0:
            continue
        if abs(a - root) < abs(n2 - root):
            n2 = a
    return n // n2, n2


# --------------------------------------------------------------------------------------
# Givens rotations and Lemma 1
# --------------------------------------------------------------------------------------
def givens(n: int, i: int, j: int, theta: float) -> np.ndarray:
    """G(i, j; theta) of Section "Givens Rotation": identity except that cos/sin sit at the
    crossings of rows/columns i and j, in the orientation of Lemma 1's 2x2 matrix
    [[cos, -sin], [sin, cos]] (row i first).  A row vector x is rotated as x @ G."""
    G = np.eye(n, dtype=np.float64)
    c, s = math.cos(theta), math.sin(theta)
    G[i, i] = c
    G[i, j] = -s
    G[j, i] = s
    G[j, j] = c
    return G


def equalizing_angle(a: float, b: float) -> float:
    """Lemma 1: theta* = atan2(b, a) - pi/4, for which (a, b) G(theta*) = (r, r)/sqrt(2)."""
    return math.atan2(b, a) - math.pi / 4.0


# --------------------------------------------------------------------------------------
# ART: alignment rotation (massive outliers)
# --------------------------------------------------------------------------------------
def haar_orthogonal(m: int, rng: np.random.Generator) -> np.ndarray:
    """A "randomly orthogonalized matrix" (ART paragraph): QR of a standard-normal matrix with
    the sign convention diag(R) > 0, which makes Q Haar distributed.  The paper does not fix
    the distribution; any orthogonal O is admissible."""
    if m <= 0:
        return np.zeros((0, 0), dtype=np.float64)
    A = rng.standard_normal((m, m))
    Q, R = np.linalg.qr(A)
    d = np.sign(np.diag(R))
    d[d == 0] = 1.0
    return Q * d[None, :]


def art_indices(c: np.ndarray) -> Tuple[int, int]:
    """ART paragraph: i = dimension of the outlier (largest |c|), j = dimension of the minimum
    value, read as the smallest magnitude among the others; ties go to the lowest index.
    Magnitudes within a relative 1e-9 of each other count as tied: after an ART step two entries
    are equal in exact arithmetic, and rounding must not decide which of them is "the" outlier."""
    n = c.shape[0]
    mag = np.abs(np.asarray(c, dtype=np.float64))
    i = 0
    for k in range(1, n):
        if mag[k] > mag[i] * (1.0 + 1e-9):
            i = k
    if n < 2:
        return i, i
    j = -1
    for k in range(n):
        if k == i:
            continue
        if j < 0 or mag[k] < mag[j] * (1.0 - 1e-9):
            j = k
    return i, j


def art_matrix(c: np.ndarray, O: Optional[np.ndarray]) -> np.ndarray:
    """R^A = diag(G(theta*), O) P_ij, acting on the LEFT of the column c (it is a factor of
    R1^T = R1^U R^A, which multiplies V_mat from the left in Eq. "eq18").

    P_ij moves entries i and j of c to positions 0 and 1 and keeps the others in order.  The
    2x2 block is the one that sends the column (a, b)^T = (c_i, c_j)^T to (r, r)^T/sqrt(2):
    Lemma 1 states it for a row vector, V G(theta*), so on a column it is G(theta*)^T.
    O (orthogonal, (n-2) x (n-2)) acts on the remaining entries; None means identity."""
    c = np.asarray(c, dtype=np.float64)
    n = c.shape[0]
    if n < 2:
        return np.eye(n, dtype=np.float64)
    i, j = art_indices(c)
    order = [i, j] + [k for k in range(n) if k != i and k != j]
    P = np.zeros((n, n), dtype=np.float64)
    for new, old in enumerate(order):
        P[new, old] = 1.0                      # (P c)[new] = c[old]
    a, b = float(c[i]), float(c[j])
    D = np.eye(n, dtype=np.float64)
    if a != 0.0 or b != 0.0:
        th = equalizing_angle(a, b)
        G2 = np.array([[math.cos(th), -math.sin(th)], [math.sin(th), math.cos(th)]])
        D[:2, :2] = G2.T
    if O is not None and n > 2:
        O = np.asarray(O, dtype=np.float64)
        assert O.shape == (n - 2, n - 2)
        D[2:, 2:] = O
    return D @ P


def art_repeat_step(c: np.ndarray) -> np.ndarray:
    """One further ART step ("Effect of ART Steps": repeated ART rotations): the plane rotation in
    coordinates (i, j) = (outlier, minimum) of the CURRENT column c that sends (c_i, c_j) to
    (r, r)/sqrt(2) (Lemma 1) and leaves every other coordinate alone.  The paper does not say how
    a repeated step treats the permutation and the random block of the first one; this reading
    repeats only the closed-form Givens rotation, which is what its ablation varies."""
    c = np.asarray(c, dtype=np.float64)
    n = c.shape[0]
    M = np.eye(n, dtype=np.float64)
    if n < 2:
        return M
    i, j = art_indices(c)
    a, b = float(c[i]), float(c[j])
    if a == 0.0 and b == 0.0:
        return M
    th = equalizing_angle(a, b)
    cs, sn = math.cos(th), math.sin(th)
    M[i, i], M[i, j], M[j, i], M[j, j] = cs, sn, -sn, cs
    return M


def art_matrix_steps(c: np.ndarray, O: Optional[np.ndarray], steps: int) -> np.ndarray:
    """R^A for `steps` >= 1 ART steps: the first is art_matrix, each further one art_repeat_step
    on the column as rotated so far."""
    RA = art_matrix(c, O)
    for _ in range(steps - 1):
        RA = art_repeat_step(RA @ np.asarray(c, dtype=np.float64)) @ RA
    return RA


# --------------------------------------------------------------------------------------
# URT: uniformity rotation (normal outliers)
# --------------------------------------------------------------------------------------
def map_to_e1(V: np.ndarray) -> Tuple[np.ndarray, int]:
    """R_map with V R_map = ||V|| e_1^T, as a product of n-1 Givens rotations (URT paragraph).
    The paper does not give the order of the chain; this one works from the last coordinate
    down: for k = n-1 .. 1 rotate the plane (k-1, k) by atan2(v_k, v_{k-1}), which zeroes v_k
    and leaves v_{k-1} = hypot >= 0.  Returns (R_map, number of Givens factors)."""
    v = np.asarray(V, dtype=np.float64).copy()
    n = v.shape[0]
    R = np.eye(n, dtype=np.float64)
    count = 0
    for k in range(n - 1, 0, -1):
        th = math.atan2(v[k], v[k - 1])
        G = givens(n, k - 1, k, th)
        v = v @ G
        R = R @ G
        count += 1
    return R, count


def uniform_target(V: np.ndarray) -> np.ndarray:
    """U of the URT paragraph: q_k = (2k - n - 1)/n for k = 1..n, assigned by the rank order
    of V (stable ascending sort pi) and scaled so that ||U|| = ||V||.  Entries closer than
    1e-9 max|V| count as equal and keep their index order (after ART two entries of the column
    are equal in exact arithmetic; rounding must not decide their rank)."""
    V = np.asarray(V, dtype=np.float64)
    n = V.shape[0]
    k = np.arange(1, n + 1, dtype=np.float64)
    q = (2.0 * k - n - 1.0) / n
    qn = np.linalg.norm(q)
    U = np.zeros(n, dtype=np.float64)
    if qn == 0.0:
        return U
    vmax = float(np.max(np.abs(V)))
    keys = np.rint(V / (1e-9 * vmax)) if vmax > 0.0 else np.zeros(n)
    pi = np.argsort(keys, kind="stable")
    U[pi] = np.linalg.norm(V) / qn * q
    return U


def urt_matrix(V: np.ndarray) -> np.ndarray:
    """R^U = R_map (R'_map)^T with V R_map = U R'_map = ||V|| e_1^T, so that V R^U = U.
    Degenerate inputs (V = 0, or n = 1 where the template q is zero) give the identity."""
    V = np.asarray(V, dtype=np.float64)
    n = V.shape[0]
    if n < 2 or not np.any(V):
        return np.eye(n, dtype=np.float64)
    U = uniform_target(V)
    R_map, _ = map_to_e1(V)
    R_map_p, _ = map_to_e1(U)
    return R_map @ R_map_p.T


def hadamard(n: int) -> np.ndarray:
    """Sylvester Hadamard matrix of order n (a power of two) scaled to be orthogonal."""
    if n < 1 or (n & (n - 1)) != 0:
        raise ValueError("Hadamard order must be a power of two")
    H = np.ones((1, 1), dtype=np.float64)
    while H.shape[0] < n:
        H = np.block([[H, H], [H, -H]])
    return H / math.sqrt(n)


# --------------------------------------------------------------------------------------
# Overall rotation R = (R1^U R^A)^T (x) (H R2^U)
# --------------------------------------------------------------------------------------
def build_rotation(calib: np.ndarray, n1: int, n2: int, flags: int = ROT_DEFAULT,
                   O: Optional[np.ndarray] = None, seed: int = 0,
                   return_f64: bool = False, art_steps: int = 1):
    """Paragraph "The Overall SingleQuant Method": R1 = (R1^U R^A)^T, R2 = H R2^U.

    The paper builds ART/URT "according to" the activation X without saying which vectors.  Any
    choice yields an orthogonal R; the reading taken here:
      1. t* = the calibration token with the largest |entry|; A = its n1 x n2 reshape;
         (p*, q*) = position of that entry; c = column q* of A (length n1).
      2. R^A from c (ART).  c' = R^A c.
      3. R1^U: the URT for the row vector c'^T; acting on the left it is (R^U)^T.
         L = (R^U)^T R^A is R1^T; R1 = L^T.
      4. A' = L A; r = the row of A' with the largest |entry|; R2^U = URT for the row r H;
         R2 = H R2^U.
    `flags` switches components to the identity (the paper's ablation of ART / URT);
    `art_steps` > 1 repeats the ART rotation (the paper's ablation of ART steps).
    Factors are built in float64 and returned rounded to float32 (the stored precision);
    with return_f64 the unrounded pair is returned as well."""
    calib = np.asarray(calib, dtype=np.float64)
    T, n = calib.shape
    if n1 * n2 != n:
        raise ValueError("n1*n2 must equal n")
    amax_tok = np.max(np.abs(calib), axis=1)
    t_star = int(np.argmax(amax_tok))
    A = calib[t_star].reshape(n1, n2)
    flat = int(np.argmax(np.abs(A)))
    p_star, q_star = divmod(flat, n2)
    c = A[:, q_star].copy()

    if flags & ROT_ART:
        if O is None and n1 > 2:
            O = haar_orthogonal(n1 - 2, np.random.default_rng(seed))
        RA = art_matrix_steps(c, O, art_steps)
    else:
        RA = np.eye(n1)
    c_prime = RA @ c
    if flags & ROT_URT:
        RU1 = urt_matrix(c_prime)
    else:
        RU1 = np.eye(n1)
    L = RU1.T @ RA
    R1 = L.T

    if flags & ROT_HADAMARD:
        H = hadamard(n2)
    else:
        H = np.eye(n2)
    A_prime = L @ A
    row = int(np.argmax(np.max(np.abs(A_prime), axis=1)))
    r = A_prime[row]
    if flags & ROT_URT:
        RU2 = urt_matrix(r @ H)
    else:
        RU2 = np.eye(n2)
    R2 = H @ RU2
    R1f, R2f = R1.astype(np.float32), R2.astype(np.float32)
    if return_f64:
        return R1f, R2f, R1, R2
    return R1f, R2f


# --------------------------------------------------------------------------------------
# Step 1: Kronecker rotation of every token
# --------------------------------------------------------------------------------------
def rotate(X: np.ndarray, R1: np.ndarray, R2: np.ndarray) -> np.ndarray:
    """Z_t = rvec(R1^T X~_t R2) for every row t of X (Eq. "eq18" and the per-slice form of
    the mode products), in float64 from the factors as given."""
    X = np.asarray(X, dtype=np.float64)
    R1 = np.asarray(R1, dtype=np.float64)
    R2 = np.asarray(R2, dtype=np.float64)
    n1, n2 = R1.shape[0], R2.shape[0]
    T, n = X.shape
    assert n == n1 * n2
    Xt = X.reshape(T, n1, n2)
    Z = np.matmul(np.matmul(R1.T[None, :, :], Xt), R2[None, :, :])
    return Z.reshape(T, n)


# --------------------------------------------------------------------------------------
# Step 2: per-row symmetric INT4 quantisation and nibble packing
# --------------------------------------------------------------------------------------
def quantize_rows(Z: np.ndarray, decision: str = "f64") -> Tuple[np.ndarray, np.ndarray]:
    """Q_Delta(z) = Delta * floor(z/Delta + 1/2) (Section 3.2) with one step per row:
    Delta_t = fp16(max_c |Z_tc| / 7), codes clamped to [-8, 7]; an all-zero row has Delta = 0
    and codes 0.  Returns (codes int8 [T x n], Delta fp16 [T]).

    decision = "f64": the paper's expression evaluated in float64 (z / Delta).
    decision = "f32": the same decision taken in float32 arithmetic, the precision the CUDA
      kernel computes in: amax/7 and 1/Delta are float32 divisions, the code is
      floor(fl32(fl32(z * inv) + 0.5)).  Z is first rounded to float32."""
    if decision == "f64":
        Z = np.asarray(Z, dtype=np.float64)
        amax = np.max(np.abs(Z), axis=1) if Z.shape[1] else np.zeros(Z.shape[0])
        delta = (amax / 7.0).astype(np.float16)
        d = delta.astype(np.float64)
        codes = np.zeros(Z.shape, dtype=np.int8)
        nz = d > 0
        if np.any(nz):
            q = np.floor(Z[nz] / d[nz, None] + 0.5)
            codes[nz] = np.clip(q, -8, 7).astype(np.int8)
        return codes, delta
    if decision == "f32":
        Z = np.asarray(Z, dtype=np.float32)
        amax = np.max(np.abs(Z), axis=1) if Z.shape[1] else np.zeros(Z.shape[0], np.float32)
        delta = (amax.astype(np.float32) / np.float32(7.0)).astype(np.float16)
        d = delta.astype(np.float32)
        codes = np.zeros(Z.shape, dtype=np.int8)
        nz = d > 0
        if np.any(nz):
            inv = (np.float32(1.0) / d[nz]).astype(np.float32)
            t = (Z[nz] * inv[:, None]).astype(np.float32)
            q = np.floor((t + np.float32(0.5)).astype(np.float32))
            codes[nz] = np.clip(q, -8, 7).astype(np.int8)
        return codes, delta
    raise ValueError(decision)


def pack_int4(codes: np.ndarray) -> np.ndarray:
    """Two's-complement nibbles, two per byte: byte k/2 = (code[k] & 15) | (code[k+1] & 15) << 4
    for even k (the low nibble holds the even channel)."""
    codes = np.asarray(codes, dtype=np.int8)
    assert codes.shape[-1] % 2 == 0
    u = codes.astype(np.uint8) & np.uint8(0x0F)
    return (u[..., 0::2] | (u[..., 1::2] << np.uint8(4))).astype(np.uint8)


def unpack_int4(packed: np.ndarray) -> np.ndarray:
    """Inverse of pack_int4: sign-extended int8 codes."""
    packed = np.asarray(packed, dtype=np.uint8)
    lo = (packed & np.uint8(0x0F)).astype(np.int16)
    hi = (packed >> np.uint8(4)).astype(np.int16)
    lo = np.where(lo >= 8, lo - 16, lo)
    hi = np.where(hi >= 8, hi - 16, hi)
    out = np.empty(packed.shape[:-1] + (packed.shape[-1] * 2,), dtype=np.int8)
    out[..., 0::2] = lo
    out[..., 1::2] = hi
    return out


# --------------------------------------------------------------------------------------
# Step 3: INT4 x INT4 GEMM with int32 accumulation, and dequantisation
# --------------------------------------------------------------------------------------
def gemm_i32(Xc: np.ndarray, Wc: np.ndarray) -> np.ndarray:
    """acc[t, c] = sum_k Xc[t, k] * Wc[c, k] (the "NT" product Flat(X~_R) Flat(W~_R)^T on the
    integer codes).  Evaluated with a float64 matmul, which is exact here: every product is at
    most 64 in magnitude and every partial sum is an integer below 64*K < 2^53."""
    Xc = np.asarray(Xc)
    Wc = np.asarray(Wc)
    assert Xc.shape[1] == Wc.shape[1]
    acc = Xc.astype(np.float64) @ Wc.astype(np.float64).T
    return acc.astype(np.int32)


def gemm_i32_loops(Xc: np.ndarray, Wc: np.ndarray) -> np.ndarray:
    """The same product by plain Python integer loops (tiny shapes only; pins gemm_i32)."""
    T, K = Xc.shape
    C = Wc.shape[0]
    out = np.zeros((T, C), dtype=np.int32)
    for t in range(T):
        for c in range(C):
            s = 0
            for k in range(K):
                s += int(Xc[t, k]) * int(Wc[c, k])
            out[t, c] = s
    return out


def dequant(acc: np.ndarray, sx: np.ndarray, sw: np.ndarray) -> np.ndarray:
    """Y[t, c] = fp16(acc[t, c] * s_x[t] * s_w[c]) in float64 with one final rounding."""
    y = acc.astype(np.float64) * sx.astype(np.float64)[:, None] * sw.astype(np.float64)[None, :]
    return y.astype(np.float16)


# --------------------------------------------------------------------------------------
# Compositions
# --------------------------------------------------------------------------------------
def rotate_quant(X: np.ndarray, R1: Optional[np.ndarray], R2: Optional[np.ndarray],
                 decision: str = "f64"):
    """Steps 1+2 on the rows of X.  R1 = R2 = None means the identity rotation.
    Returns (packed uint8 [T x n/2], Delta fp16 [T], Z float64 [T x n])."""
    if R1 is None:
        Z = np.asarray(X, dtype=np.float64)
    else:
        Z = rotate(X, R1, R2)
    codes, delta = quantize_rows(Z, decision)
    return pack_int4(codes), delta, Z


def pack_weight(W: np.ndarray, R1, R2, decision: str = "f64"):
    """Offline weight path: Flat(W~_R) = W^T R, i.e. the same operator as the activations
    applied to the rows of W [C x n] ("structurally equivalent rotations to the original weight
    matrix"), then round-to-nearest INT4 with one step per output channel."""
    return rotate_quant(W, R1, R2, decision)


def linear(X: np.ndarray, W: np.ndarray, R1, R2, decision: str = "f64") -> np.ndarray:
    """The whole W4A4 linear layer: rotate+quantise X, rotate+quantise W, integer GEMM, dequant."""
    Xq, sx, _ = rotate_quant(X, R1, R2, decision)
    Wq, sw, _ = pack_weight(W, R1, R2, decision)
    acc = gemm_i32(unpack_int4(Xq), unpack_int4(Wq))
    return dequant(acc, sx, sw)


def linear_fp(X: np.ndarray, W: np.ndarray) -> np.ndarray:
    """The unquantised layer X W^T in float64 (rotation invariance XW = (XR)(R^T W))."""
    return np.asarray(X, dtype=np.float64) @ np.asarray(W, dtype=np.float64).T


def kron_dense(R1: np.ndarray, R2: np.ndarray) -> np.ndarray:
    """The explicit n x n matrix R1 (x) R2 (small sizes only; used by the pins)."""
    return np.kron(np.asarray(R1, dtype=np.float64), np.asarray(R2, dtype=np.float64))


# --------------------------------------------------------------------------------------
# Weight-only variant (Appendix "Weight-only Quantization", Table "wquant": W4A16 / W3A16) and the
# grouped form of the layer for mixture-of-experts blocks (Section "Results on Mixtral Models")
#
# The paper gives the setting only: the same rotation, weights quantised to 4 or 3 bits with one
# step per output channel, activations left in 16 bits.  Readings taken here: the activations are
# rotated online exactly as in the W4A4 path and rounded once to fp16; a b-bit code is the W4A4
# quantiser with 7 replaced by 2^(b-1) - 1 and the clamp by [-2^(b-1), 2^(b-1) - 1]; the product
# is the plain real-valued one with a single rounding of the result to fp16.
# --------------------------------------------------------------------------------------
def quantize_rows_bits(Z: np.ndarray, bits: int, decision: str = "f64") -> Tuple[np.ndarray, np.ndarray]:
    """Q_Delta of Section 3.2 with b bits: Delta_t = fp16(max_c |Z_tc| / (2^(b-1) - 1)), code =
    floor(z / Delta + 1/2) clamped to [-2^(b-1), 2^(b-1) - 1]; an all-zero row has Delta = 0 and
    codes 0.  `decision` as in quantize_rows.  Returns (codes int8, Delta fp16)."""
    if bits < 2 or bits > 8:
        raise ValueError("bits")
    qmax = 2 ** (bits - 1) - 1
    qmin = -(2 ** (bits - 1))
    ft = {"f64": np.float64, "f32": np.float32}[decision]
    Z = np.asarray(Z, dtype=ft)
    T = Z.shape[0]
    codes = np.zeros(Z.shape, dtype=np.int8)
    delta = np.zeros(T, dtype=np.float16)
    for t in range(T):
        amax = ft(np.max(np.abs(Z[t]))) if Z.shape[1] else ft(0)
        delta[t] = np.float16(ft(amax / ft(qmax)))
        d = ft(delta[t])
        if d > 0:
            if decision == "f64":
                q = np.floor(Z[t] / d + 0.5)
            else:
                inv = ft(ft(1.0) / d)
                q = np.floor(((Z[t] * inv).astype(ft) + ft(0.5)).astype(ft))
            codes[t] = np.clip(q, qmin, qmax).astype(np.int8)
    return codes, delta


# Storage order of the weight-only format: nibble position i (bits 4i .. 4i+3 of a little-endian
# 32-bit word) holds channel WO_ORDER[i] of the word's eight consecutive channels, so that
# (word >> 4s) & 0x000F000F is the pair (channel 2s, channel 2s + 1) in the two 16-bit halves.
WO_ORDER = (0, 2, 4, 6, 1, 3, 5, 7)


def pack_int4_interleaved(codes: np.ndarray) -> np.ndarray:
    """Two's-complement nibbles in the weight-only storage order (see WO_ORDER); K % 8 == 0."""
    codes = np.asarray(codes, dtype=np.int8)
    K = codes.shape[-1]
    assert K % 8 == 0
    u = (codes.astype(np.uint8) & np.uint8(0x0F)).reshape(codes.shape[:-1] + (K // 8, 8))
    out = np.zeros(codes.shape[:-1] + (K // 8, 4), dtype=np.uint8)
    for pos in range(8):
        nib = u[..., WO_ORDER[pos]]
        out[..., pos // 2] |= (nib << np.uint8(4 * (pos % 2))).astype(np.uint8)
    return out.reshape(codes.shape[:-1] + (K // 2,))


def unpack_int4_interleaved(packed: np.ndarray) -> np.ndarray:
    """Inverse of pack_int4_interleaved: sign-extended int8 codes in channel order."""
    packed = np.asarray(packed, dtype=np.uint8)
    Kb = packed.shape[-1]
    assert Kb % 4 == 0
    b = packed.reshape(packed.shape[:-1] + (Kb // 4, 4))
    out = np.zeros(packed.shape[:-1] + (Kb // 4, 8), dtype=np.int8)
    for pos in range(8):
        nib = ((b[..., pos // 2] >> np.uint8(4 * (pos % 2))) & np.uint8(0x0F)).astype(np.int16)
        out[..., WO_ORDER[pos]] = np.where(nib >= 8, nib - 16, nib).astype(np.int8)
    return out.reshape(packed.shape[:-1] + (Kb * 2,))


def rotate_f16(X: np.ndarray, R1: Optional[np.ndarray], R2: Optional[np.ndarray]) -> np.ndarray:
    """The rotated activations of the weight-only path: Eq. "eq18" in float64, one rounding to fp16."""
    Z = np.asarray(X, dtype=np.float64) if R1 is None else rotate(X, R1, R2)
    return Z.astype(np.float16)


def pack_weight_wo(W: np.ndarray, R1, R2, bits: int, decision: str = "f64"):
    """Offline weight path of the weight-only variant: rotate the rows of W, b-bit codes with one
    step per output channel, stored in the weight-only order.  Returns (packed uint8 [C x n/2],
    Delta fp16 [C], rotated rows float64)."""
    Z = np.asarray(W, dtype=np.float64) if R1 is None else rotate(W, R1, R2)
    codes, delta = quantize_rows_bits(Z, bits, decision)
    return pack_int4_interleaved(codes), delta, Z


def gemm_w4a16(Z16: np.ndarray, codes: np.ndarray, sw: np.ndarray) -> np.ndarray:
    """Y[t, c] = fp16((sum_k Z16[t, k] * code[c, k]) * s_w[c]): the real-valued product in float64
    with one final rounding."""
    acc = np.asarray(Z16, dtype=np.float64) @ np.asarray(codes, dtype=np.float64).T
    return (acc * np.asarray(sw, dtype=np.float64)[None, :]).astype(np.float16)


def linear_wo(X: np.ndarray, W: np.ndarray, R1, R2, bits: int, decision: str = "f64") -> np.ndarray:
    """The weight-only layer: fp16 rotated activations against b-bit pre-rotated weights."""
    Wq, sw, _ = pack_weight_wo(W, R1, R2, bits, decision)
    return gemm_w4a16(rotate_f16(X, R1, R2), unpack_int4_interleaved(Wq), sw)


def linear_grouped(X: np.ndarray, offsets, Ws, rotations, decision: str = "f64") -> np.ndarray:
    """The W4A4 layer of a mixture-of-experts block: the tokens are sorted by expert, expert e owns
    rows offsets[e] .. offsets[e+1]-1 of X and has its own weights Ws[e] [C x n] and its own factor
    pair rotations[e] = (R1, R2); every expert's rows go through `linear` with that expert's
    matrices.  Returns Y [T x C]."""
    X = np.asarray(X)
    E = len(Ws)
    assert len(offsets) == E + 1 and offsets[0] == 0 and offsets[-1] == X.shape[0]
    C = Ws[0].shape[0]
    Y = np.zeros((X.shape[0], C), dtype=np.float16)
    for e in range(E):
        a, b = int(offsets[e]), int(offsets[e + 1])
        assert a <= b
        if b > a:
            Y[a:b] = linear(X[a:b], Ws[e], rotations[e][0], rotations[e][1], decision)
    return Y
