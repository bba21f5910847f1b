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


def build_matrices(m, r, points, scale_G=None, scale_B=None):
    """Exact A^T (m x n), G (n x r), B^T (n x n) as nested lists of Fraction.

    Algorithm 3, in its own order:
      Lagrange factors  F_i = prod_{j != i} (alpha_i - alpha_j)
      A^T[i][p] = alpha_p^i  (Vandermonde basis truncated to m rows);
                  infinity column = e_{m-1}
      G[p][k]   = alpha_p^k / F_p ; infinity row = e_{r-1}
      B^T[p][:] = coefficients (ascending) of prod_{j != p} (t - alpha_j),
                  zero padded to n; infinity row = coefficients of
                  prod_j (t - alpha_j)

    scale_G / scale_B (optional, one non-zero rational per point) apply the
    diagonal rescaling of the comparison with learned-scale methods
    (Appendix "Relation to complementary techniques"): D_G multiplies the rows
    of G, D_B the rows of B^T, and D_A = (D_G D_B)^-1 the columns of A^T, so
    that D_A D_G D_B = I and the bilinear identity is unchanged.
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
    if scale_G is not None or scale_B is not None:
        sg = [Fraction(1)] * n if scale_G is None else [Fraction(*v) if isinstance(v, tuple) else Fraction(v) for v in scale_G]
        sb = [Fraction(1)] * n if scale_B is None else [Fraction(*v) if isinstance(v, tuple) else Fraction(v) for v in scale_B]
        if len(sg) != n or len(sb) != n or any(v == 0 for v in sg + sb):
            raise ValueError("need one non-zero scale per point")
        for p in range(n):
            G[p] = [sg[p] * v for v in G[p]]
            BT[p] = [sb[p] * v for v in BT[p]]
            for i in range(m):
                AT[i][p] = AT[i][p] / (sg[p] * sb[p])
    return AT, G, BT


def snap_to_rational(x, d_max=10):
    """Nearest simple rational (Definition "Snap-to-Rational", Section "Snap-to-Rational";
    Algorithm 2): argmin |x - a/b| over 1 <= b <= d_max, |a| <= 5 b.  Candidates are visited
    by increasing denominator, then increasing numerator, and only a strictly smaller
    distance replaces the incumbent, so ties keep the first (smallest-denominator) one."""
    x = Fraction(x)
    best, best_dist = None, None
    for b in range(1, d_max + 1):
        for a in range(-5 * b, 5 * b + 1):
            f = Fraction(a, b)
            dist = abs(x - f)
            if best is None or dist < best_dist:
                best, best_dist = f, dist
    return best


def norm2(M):
    """Spectral norm (largest singular value)."""
    return float(np.linalg.svd(np.asarray(M, dtype=np.float64), compute_uv=False)[0])


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


def symmetric_search(n_finite, d_max=6, p_max=2):
    """Symmetric search (Section "Symmetric Search"): configurations made of pairs (p, -p), plus 0
    when the number of finite points is odd.  Candidates p are the positive rationals of the
    snap-to-rational grid (denominator <= d_max) up to p_max; every combination is evaluated and
    the one with the lowest kappa_2 of the Vandermonde matrix wins.  Returns (finite points in the
    order 0, +p1, -p1, +p2, -p2, .. with p1 < p2 < .., kappa_2).  Plain enumeration."""
    import itertools
    cands = sorted({Fraction(a, b) for b in range(1, d_max + 1) for a in range(1, p_max * b + 1)})
    pairs = n_finite // 2
    best, best_k = None, None
    for combo in itertools.combinations(cands, pairs):
        pts = ([Fraction(0)] if n_finite % 2 else []) + [s * p for p in combo for s in (1, -1)]
        k = kappa2(np.array([[float(a) ** j for j in range(n_finite)] for a in pts]))
        if best is None or k < best_k:
            best, best_k = pts, k
    return best, best_k
