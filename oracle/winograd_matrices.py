"""Winograd transformation matrices rebuilt from interpolation points (test infrastructure).

This module belongs to the CPU oracle.  It is imported only by the tests, by the
smoke check and by the benchmark's CPU-baseline leg; the CUDA product path never
imports it and carries its own hand-written tables.

Everything here is exact rational arithmetic (``fractions.Fraction``) and follows
the paper's supplementary section "Standard Winograd transforms":

* the polynomial points ``(f_i, g_i)`` of F(4,3) and F(6,3) (and, beyond the paper, of the
  textbook F(2,3): points 0, 1, -1, infinity, scales chosen so that the matrices are the
  familiar ones of the fast-convolution literature),
* the Vandermonde matrix ``V_{a x b}[i][j] = f_i**j * g_i**(b-1-j)``,
* ``A^T = V_{n x m}^T S_A``      (Eq. ``scale_a``),
* ``B^T = S_B V_{n x n}^{-T}``   (Eq. ``scale_b``),
* ``G   = S_G V_{n x r}``        (Eq. ``scale_g``),
* the condition ``S_A S_B S_G = I`` (Eq. ``scaling_condition``),

and the short-hands of Section 4.1: ``V_B = V_{n x n}^{-T}``, ``V_G = V_{n x r}``,
``V_A = V_{n x m}^T``.
"""
from fractions import Fraction as Fr

import numpy as np

R = 3  # filter size; the paper uses F(m, 3) throughout

# Polynomial points (f_i, g_i); the last one, (1, 0), is the point at infinity.
POINTS = {
    2: [(Fr(0), Fr(1)), (Fr(1), Fr(1)), (Fr(-1), Fr(1)), (Fr(1), Fr(0))],
    4: [(Fr(0), Fr(1)), (Fr(1), Fr(1)), (Fr(-1), Fr(1)),
        (Fr(2), Fr(1)), (Fr(-2), Fr(1)), (Fr(1), Fr(0))],
    6: [(Fr(0), Fr(1)), (Fr(1), Fr(1)), (Fr(-1), Fr(1)), (Fr(2), Fr(1)),
        (Fr(-2), Fr(1)), (Fr(1, 2), Fr(1)), (Fr(-1, 2), Fr(1)), (Fr(1), Fr(0))],
}

# Standard scaling factors printed next to the points.
STANDARD_SCALES = {
    2: dict(SA=[Fr(1), Fr(1), Fr(1), Fr(-1)],
            SB=[Fr(1), Fr(2), Fr(2), Fr(-1)],
            SG=[Fr(1), Fr(1, 2), Fr(1, 2), Fr(1)]),
    4: dict(SA=[Fr(1)] * 6,
            SB=[Fr(4), Fr(-6), Fr(-6), Fr(24), Fr(24), Fr(1)],
            SG=[Fr(1, 4), Fr(-1, 6), Fr(-1, 6), Fr(1, 24), Fr(1, 24), Fr(1)]),
    6: dict(SA=[Fr(1)] * 8,
            SB=[Fr(1), Fr(-9, 2), Fr(-9, 2), Fr(90), Fr(90), Fr(45, 32), Fr(45, 32), Fr(1)],
            SG=[Fr(1), Fr(-2, 9), Fr(-2, 9), Fr(1, 90), Fr(1, 90), Fr(32, 45), Fr(32, 45), Fr(1)]),
}


def _pow(base, e):
    # 0**0 == 1 by the Vandermonde convention (first/last column of the points
    # (0,1) and (1,0)).
    return Fr(1) if e == 0 else base ** e


def vandermonde(points, b):
    """V_{a x b}: row i is f_i^j g_i^(b-1-j) for j = 0..b-1 (a = len(points))."""
    return [[_pow(f, j) * _pow(g, b - 1 - j) for j in range(b)] for (f, g) in points]


def transpose(M):
    return [list(r) for r in zip(*M)]


def matmul(A, B):
    return [[sum((A[i][k] * B[k][j] for k in range(len(B))), Fr(0))
             for j in range(len(B[0]))] for i in range(len(A))]


def inverse(M):
    """Gauss-Jordan over the rationals; raises if M is singular."""
    n = len(M)
    aug = [list(M[i]) + [Fr(int(i == j)) for j in range(n)] for i in range(n)]
    for col in range(n):
        piv = next(r for r in range(col, n) if aug[r][col] != 0)
        aug[col], aug[piv] = aug[piv], aug[col]
        d = aug[col][col]
        aug[col] = [v / d for v in aug[col]]
        for r in range(n):
            if r != col and aug[r][col] != 0:
                fct = aug[r][col]
                aug[r] = [vr - fct * vc for vr, vc in zip(aug[r], aug[col])]
    return [row[n:] for row in aug]


def diag_mul_left(s, M):
    """diag(s) @ M."""
    return [[s[i] * v for v in M[i]] for i in range(len(M))]


def diag_mul_right(M, s):
    """M @ diag(s)."""
    return [[M[i][j] * s[j] for j in range(len(s))] for i in range(len(M))]


def vandermonde_parts(m):
    """(V_A, V_B, V_G) of Section 4.1 for F(m,3), exact.

    V_A = V_{n x m}^T (m x n), V_B = V_{n x n}^{-T} (n x n), V_G = V_{n x 3} (n x 3).
    """
    pts = POINTS[m]
    n = m + R - 1
    assert len(pts) == n
    VA = transpose(vandermonde(pts, m))
    VB = transpose(inverse(vandermonde(pts, n)))
    VG = vandermonde(pts, R)
    return VA, VB, VG


def scaled_matrices(m, SA=None, SB=None, SG=None):
    """(A^T, B^T, G) with the given diagonal scales (default: the standard ones)."""
    std = STANDARD_SCALES[m]
    SA = std["SA"] if SA is None else SA
    SB = std["SB"] if SB is None else SB
    SG = std["SG"] if SG is None else SG
    VA, VB, VG = vandermonde_parts(m)
    return diag_mul_right(VA, SA), diag_mul_left(SB, VB), diag_mul_left(SG, VG)


def to_f64(M):
    """Exact rationals -> float64 ndarray (each entry rounded once)."""
    return np.array([[float(v) for v in row] for row in M], dtype=np.float64)


def vandermonde_parts_f64(m):
    VA, VB, VG = vandermonde_parts(m)
    return to_f64(VA), to_f64(VB), to_f64(VG)


def standard_scales_f64(m):
    std = STANDARD_SCALES[m]
    f = lambda v: np.array([float(x) for x in v], dtype=np.float64)
    return f(std["SA"]), f(std["SB"]), f(std["SG"])
