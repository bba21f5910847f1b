"""Interpolation point sets used by the workloads.

Each set is a list of (numerator, denominator) pairs for the finite points,
followed by the point at infinity written as (1, 0) (projective coordinates,
Section 2.4).  Standard sets are the integer points of Table 1 (Section 2.2);
"nova" sets are the discovered configurations of Table 3 (Section 5.2).  The
half-integer F(6,3) set is the customary Lavin-Gray choice that the workload
list names as "standard" for that tile.
"""

INF = (1, 0)


def _sym(*pos):
    out = [(0, 1)]
    for (a, b) in pos:
        out.append((a, b))
        out.append((-a, b))
    out.append(INF)
    return out


POINT_SETS = {
    # Table 1: standard integer points
    ("std", 2): _sym((1, 1)),
    ("std", 4): _sym((1, 1), (2, 1)),
    ("std", 6): _sym((1, 1), (2, 1), (3, 1)),
    ("std", 8): _sym((1, 1), (2, 1), (3, 1), (4, 1)),
    # customary F(6,3) set with +-1/2 (named "standard" by the F(6,3) workload)
    ("half", 6): _sym((1, 1), (2, 1), (1, 2)),
    # Table 3: discovered points
    ("nova", 2): _sym((1, 1)),
    ("nova", 4): _sym((5, 6), (7, 6)),
    ("nova", 6): _sym((3, 5), (1, 1), (7, 6)),
    ("nova", 8): _sym((2, 5), (5, 6), (1, 1), (7, 6)),
    # Table "Dtype-aware vs unconstrained discovery": dyadic points, exact in binary16
    ("dyadic", 4): _sym((3, 4), (5, 4)),
    # Not from the paper: rational sets that are NOT symmetric about 0, in no particular order.
    # Section 2.1 needs distinct points and nothing else; these exercise the general (dense) form
    # of the transforms, which no printed set reaches.
    ("asym", 2): [(1, 2), (-1, 1), (0, 1), INF],
    ("asym", 4): [(3, 7), (-2, 1), (0, 1), (5, 4), (-1, 3), INF],
    ("asym", 6): [(1, 1), (-1, 2), (2, 3), (0, 1), (-3, 2), (5, 4), (-3, 4), INF],
    ("asym", 8): [(2, 5), (-6, 5), (1, 1), (-1, 2), (0, 1), (7, 6), (-3, 4), (5, 6), (-1, 1), INF],
    # The discovered sets of Table 3 listed in another order (infinity stays last): the result is
    # the same convolution; only the order of the transformed-domain coordinates changes.
    ("shuf", 4): [(-7, 6), (5, 6), (0, 1), (7, 6), (-5, 6), INF],
    ("shuf", 6): [(1, 1), (-3, 5), (7, 6), (0, 1), (-1, 1), (3, 5), (-7, 6), INF],
    ("shuf", 8): [(-5, 6), (1, 1), (2, 5), (-7, 6), (0, 1), (7, 6), (-2, 5), (5, 6), (-1, 1), INF],
}


def point_set(kind, m):
    """Return a fresh list of (num, den) pairs; the last entry is infinity."""
    return list(POINT_SETS[(kind, m)])


def pow2_range_scales(G, BT):
    """Power-of-two row scales (scale_G, scale_B), as (num, den) pairs, that bring the largest
    magnitude of every row of G and of B^T into [1, 2).  G, BT: nested lists / arrays of numbers
    (the unscaled matrices).  Powers of two change no rounding of the transforms, only the range
    of the transformed filter and input - the hardware-friendly form of the per-tap scales in the
    appendix on complementary techniques.  The same scale serves both points of a +- pair because
    their rows differ by signs only."""
    import math

    def scale(row):
        mx = max(abs(float(v)) for v in row)
        e = math.floor(math.log2(mx))
        return (1, 2 ** e) if e >= 0 else (2 ** (-e), 1)
    return [scale(r) for r in G], [scale(r) for r in BT]
