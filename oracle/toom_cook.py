"""Exact Toom-Cook / Winograd matrix construction (oracle side).

TEST INFRASTRUCTURE ONLY - see oracle/__init__.py.

Follows Algorithm 3 ("Symbolic Cook-Toom Construction") and Section 2.1:
points alpha_0..alpha_{n-2} are exact rationals, the last point is infinity,
n = m + r - 1.  All arithmetic is fractions.Fraction; conversion to floating
point happens once, at the end.
"""
from fractions import Fraction
import numpy as np


def split_points(points):
    """Return the finite points as Fractions; the single (x, 0) entry is infinity.

    Raises ValueError for no / several infinities, an infinity that is not
    last, or repeated finite points (Theorem A.2 needs distinct points).
    """
    fin = []
    n_inf = 0
    for idx, (num, den) in enumerate(points):
        if den == 0:
            n_inf += 1
            if idx != len(points) - 1:
                raise ValueError("the point at infinity must be the last point")
        else:
            fin.append(Fraction(num, den))
    if n_inf != 1:
        raise ValueError("exactly one point at infinity is required")
    if len(set(fin)) != len(fin):
        raise ValueError("finite points must be distinct")
    return fin


def _poly_mul_linear(coeffs, root):
    """coeffs (ascending powers) times (t - root)."""
    out = [Fraction(0)] * (len(coeffs) + 1)
    for i, c in enumerate(coeffs):
        out[i + 1] += c
        out[i] -= c * root
    return out


def build_matrices(m, r, points):
    """Exact A^T (m x n), G (n x r), B^T (n x n) as nested lists of Fraction.

    Algorithm 3, in its own order:
      Lagrange factors  F_i = prod_{j != i} (alpha_i - alpha_j)
      A^T[i][p] = alpha_p^i  (Vandermonde basis truncated to m rows);
                  infinity column = e_{m-1}
      G[p][k]   = alpha_p^k / F_p ; infinity row = e_{r-1}
      B^T[p][:] = coefficients (ascending) of prod_{j != p} (t - alpha_j),
                  zero padded to n; infinity row = coefficients of
                  prod_j (t - alpha_j)
    """
    n = m + r - 1
    if len(points) != n:
        raise ValueError("need n = m + r - 1 points")
    al = split_points(points)
    nf = n - 1
    F = []
    for i in range(nf):
        f = Fraction(1)
        for j in range(nf):
            if j != i:
                f *= (al[i] - al[j])
        F.append(f)
    AT = [[Fraction(0)] * n for _ in range(m)]
    for i in range(m):
        for p in range(nf):
            AT[i][p] = al[p] ** i
    AT[m - 1][n - 1] = Fraction(1)
    G = [[Fraction(0)] * r for _ in range(n)]
    for p in range(nf):
        for k in range(r):
            G[p][k] = al[p] ** k / F[p]
    G[n - 1][r - 1] = Fraction(1)
    BT = [[Fraction(0)] * n for _ in range(n)]
    for p in range(nf):
        poly = [Fraction(1)]
        for j in range(nf):
            if j != p:
                poly = _poly_mul_linear(poly, al[j])
        for j, c in enumerate(poly):
            BT[p][j] = c
    poly = [Fraction(1)]
    for j in range(nf):
        poly = _poly_mul_linear(poly, al[j])
    for j, c in enumerate(poly):
        BT[n - 1][j] = c
    return AT, G, BT


def decomposition_residual(m, r, AT, G, BT):
    """Exact residual of the convolution tensor identity (Section 2.4):
    sum_p A^T[i][p] G[p][k] B^T[p][j] - 1[j == i + k]; list of non-zero entries."""
    n = m + r - 1
    bad = []
    for i in range(m):
        for k in range(r):
            for j in range(n):
                s = sum(AT[i][p] * G[p][k] * BT[p][j] for p in range(n))
                if s != (1 if j == i + k else 0):
                    bad.append((i, k, j, s))
    return bad


def to_float(M, dtype=np.float64):
    """Correctly rounded Fraction -> float64, then round-to-nearest-even to dtype."""
    a = np.array([[float(v) for v in row] for row in M], dtype=np.float64)
    return a.astype(dtype)


def vandermonde(points):
    """V_ij = alpha_i^j over the n-1 finite points only (Section 2.2)."""
    al = split_points(points)
    nf = len(al)
    return np.array([[float(a ** j) for j in range(nf)] for a in al], dtype=np.float64)


def kappa2(M):
    """Spectral condition number sigma_max / sigma_min (Section 2.2)."""
    s = np.linalg.svd(np.asarray(M, dtype=np.float64), compute_uv=False)
    return float(s[0] / s[-1])


def kappa2_V(points):
    return kappa2(vandermonde(points))
