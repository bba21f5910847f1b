"""Direct and Winograd r x r convolution (r = 3, or 5 for the appendix's 5 x 5 extension) on the CPU (oracle side).

TEST INFRASTRUCTURE ONLY - see oracle/__init__.py.

Conventions (Section 2.1): cross-correlation y_i = sum_k g_k x_{i+k} (no kernel
flip), stride 1, zero padding (r-1)/2, tensors NHWC: x [N,H,W,C], g [K,r,r,C],
y [N,H,W,K]; the filter size r is read from g.  The paper does not say how an image is cut into tiles; the
reading used everywhere here is: tile (th, tw) covers output rows
m*th .. m*th+m-1, reads the n x n input patch whose top-left corner is
(m*th - pad, m*tw - pad), pad = (r-1)/2, from the zero-extended image, and outputs that fall
outside H x W are dropped.
"""
from fractions import Fraction
import numpy as np

from . import toom_cook as tc


# --------------------------------------------------------------------------
# O1: the plain definition, fp64
# --------------------------------------------------------------------------
def direct_conv_fp64(x, g):
    """y[n,h,w,k] = sum_{a,b,c} xz[n,h+a-1,w+b-1,c] * g[k,a,b,c] in float64.

    Section 2.1's definition extended to 2-D and channels; xz is x extended by
    zeros.  A library matmul serves as the inner sum over c.
    """
    x = np.asarray(x, dtype=np.float64)
    g = np.asarray(g, dtype=np.float64)
    N, H, W, C = x.shape
    K, r = g.shape[0], g.shape[1]
    pad = (r - 1) // 2
    xp = np.zeros((N, H + 2 * pad, W + 2 * pad, C), dtype=np.float64)
    xp[:, pad:H + pad, pad:W + pad, :] = x
    y = np.zeros((N, H, W, K), dtype=np.float64)
    for a in range(r):
        for b in range(r):
            y += xp[:, a:a + H, b:b + W, :] @ g[:, a, b, :].T
    return y


def relu(x):
    return np.maximum(x, 0)


def maxpool2x2(x):
    """2x2 max pooling, stride 2, NHWC, even H and W."""
    N, H, W, C = x.shape
    return x.reshape(N, H // 2, 2, W // 2, 2, C).max(axis=(2, 4))


def rel_l2(y, y_ref):
    """||y - y_ref||_2 / ||y_ref||_2 over the whole tensor (Section 5.4 protocol)."""
    y = np.asarray(y, dtype=np.float64)
    y_ref = np.asarray(y_ref, dtype=np.float64)
    with np.errstate(all="ignore"):
        return float(np.linalg.norm((y - y_ref).ravel()) / np.linalg.norm(y_ref.ravel()))


# --------------------------------------------------------------------------
# tiling helpers shared by O3 / O4 (pure indexing, no arithmetic)
# --------------------------------------------------------------------------
def _gather_tiles(x, m, r=3):
    """d[N,Th,Tw,a,b,C] = xz[n, m*th-pad+a, m*tw-pad+b, c] with zero extension, pad = (r-1)/2."""
    N, H, W, C = x.shape
    n = m + r - 1
    pad = (r - 1) // 2
    Th, Tw = -(-H // m), -(-W // m)
    xp = np.zeros((N, m * Th + r - 1, m * Tw + r - 1, C), dtype=x.dtype)
    xp[:, pad:H + pad, pad:W + pad, :] = x
    d = np.empty((N, Th, Tw, n, n, C), dtype=x.dtype)
    for a in range(n):
        for b in range(n):
            d[:, :, :, a, b, :] = xp[:, a:a + m * Th:m, b:b + m * Tw:m, :]
    return d


def _scatter_tiles(Y, H, W):
    """Y[N,Th,Tw,i,j,K] -> y[N,H,W,K], dropping rows/cols beyond H, W."""
    N, Th, Tw, m, _, K = Y.shape
    y = Y.transpose(0, 1, 3, 2, 4, 5).reshape(N, Th * m, Tw * m, K)
    return np.ascontiguousarray(y[:, :H, :W, :])


def _two_sided(L, X, axes, dtype):
    """Apply L along two axes of X: out[..p..q..] = sum_ab L[p,a] L[q,b] X[..a..b..].

    Done as two successive one-sided products, each evaluated in `dtype`
    (the intermediate stays in `dtype`, it is not rounded any lower).
    """
    L = L.astype(dtype)
    X = X.astype(dtype)
    t = np.moveaxis(np.tensordot(L, X, axes=([1], [axes[0]])), 0, axes[0])
    t = t.astype(dtype)
    o = np.moveaxis(np.tensordot(L, t, axes=([1], [axes[1]])), 0, axes[1])
    return o.astype(dtype)


# --------------------------------------------------------------------------
# O3: Winograd in fp64 with the exact matrices
# --------------------------------------------------------------------------
def winograd_conv_fp64(x, g, m, points, scales=(None, None)):
    """Y = A^T [ (G g G^T) (.) (B^T d B) ] A per tile, summed over channels
    (Section B.5 for the 2-D nesting, Section 2.1 for the four steps).
    scales = (scale_G, scale_B): optional diagonal rescaling, see toom_cook.build_matrices."""
    r = np.asarray(g).shape[1]
    AT, G, BT = (tc.to_float(M_) for M_ in tc.build_matrices(m, r, points, *scales))
    x = np.asarray(x, dtype=np.float64)
    g = np.asarray(g, dtype=np.float64)
    N, H, W, C = x.shape
    U = _two_sided(G, g, (1, 2), np.float64)            # [K,n,n,C]
    d = _gather_tiles(x, m, r)                           # [N,Th,Tw,n,n,C]
    V = _two_sided(BT, d, (3, 4), np.float64)            # [N,Th,Tw,n,n,C]
    M = np.einsum("ntuxyc,kxyc->ntuxyk", V, U, optimize=True)
    Y = _two_sided(AT, M, (3, 4), np.float64)            # [N,Th,Tw,m,m,K]
    return _scatter_tiles(Y, H, W)


# --------------------------------------------------------------------------
# exact rational Winograd on tiny integer tensors (plain loops)
# --------------------------------------------------------------------------
def winograd_conv_exact(x, g, m, points):
    """Same four steps with fractions.Fraction; returns nested lists y[n][h][w][k].

    x, g are integer arrays.  Used to show the transforms reproduce direct
    convolution with zero error (Section 2.4, "exactly zero").
    """
    AT, G, BT = tc.build_matrices(m, 3, points)
    n = m + 2
    N, H, W, C = x.shape
    K = g.shape[0]
    Th, Tw = -(-H // m), -(-W // m)

    def xz(i, h, w, c):
        return int(x[i, h, w, c]) if 0 <= h < H and 0 <= w < W else 0

    U = [[[[sum(G[p][a] * int(g[k, a, b, c]) * G[q][b] for a in range(3) for b in range(3))
            for c in range(C)] for k in range(K)] for q in range(n)] for p in range(n)]
    y = [[[[Fraction(0)] * K for _ in range(W)] for _ in range(H)] for _ in range(N)]
    for i in range(N):
        for th in range(Th):
            for tw in range(Tw):
                d = [[[xz(i, m * th - 1 + a, m * tw - 1 + b, c) for c in range(C)]
                      for b in range(n)] for a in range(n)]
                V = [[[sum(BT[p][a] * d[a][b][c] * BT[q][b] for a in range(n) for b in range(n))
                       for c in range(C)] for q in range(n)] for p in range(n)]
                for k in range(K):
                    Mm = [[sum(U[p][q][k][c] * V[p][q][c] for c in range(C))
                           for q in range(n)] for p in range(n)]
                    for oi in range(m):
                        for oj in range(m):
                            h, w = m * th + oi, m * tw + oj
                            if h < H and w < W:
                                y[i][h][w][k] = sum(AT[oi][p] * Mm[p][q] * AT[oj][q]
                                                    for p in range(n) for q in range(n))
    return y


# --------------------------------------------------------------------------
# O4: rounding emulation of the low-precision pipeline
# --------------------------------------------------------------------------
def coefficient_tables(m, points, mode, coef="mode", scales=(None, None), r=3):
    """Transform matrices as the device evaluates them, returned as float32.

    mode "fp16", coef "mode": exact rational -> float64 -> float16 (round to
    nearest even) -> widened (Section 5.1 "cast to FP16"; Section C.3 "matrices
    stored in float16").  coef "fp32" or mode "fp32": rounded to float32 only.
    """
    mats = tc.build_matrices(m, r, points, *scales)
    out = []
    for M_ in mats:
        a = tc.to_float(M_)
        with np.errstate(over="ignore"):
            if mode == "fp16" and coef == "mode":
                a = a.astype(np.float16)
        out.append(a.astype(np.float32))
    return out  # AT, G, BT


def _stage_dtypes(mode):
    """(storage dtype of U, V and y; dtype the sums are evaluated in) for an arithmetic mode.

    "fp16": binary16 storage, sums in float32 (Section 5.1 "FP16 Setup": transforms computed
    in FP32 and cast to FP16; Section C.3: intermediates float32).  "fp32": float32 storage;
    every stored element is ONE rounding of a sum carried in float64, so that what the mode
    loses is the float32 storage of U, V, M and y and nothing else.  The paper only names the
    mode ("FP32 baseline", Section 5.1); this reading is the one under which the F(8,3) tile with
    well-conditioned points stays below a relative error of 1e-4 (sums carried in float32 sit at
    1.2e-4 .. 1.7e-4 for that tile)."""
    if mode == "fp16":
        return np.float16, np.float32
    return np.float32, np.float64


def filter_transform_emulated(g, m, points, mode, coef="mode", scales=(None, None)):
    """U[K,n,n,C]: G g G^T evaluated in the mode's sum precision, rounded once to the operand dtype."""
    _, G, _ = coefficient_tables(m, points, mode, coef, scales, r=np.asarray(g).shape[1])
    st, ev = _stage_dtypes(mode)
    with np.errstate(all="ignore"):
        U = _two_sided(G, np.asarray(g), (1, 2), ev).astype(st)
    return U


def winograd_conv_emulated(x, g, m, points, mode, coef="mode", apply_relu=False, scales=(None, None)):
    """The four steps with the pipeline's rounding points:

    tables rounded as in coefficient_tables; U and V evaluated in the mode's sum precision
    (float32 in mode "fp16") and rounded once to the operand dtype (float16); the product summed
    over channels in float32 (products of two float16 values are exact in float32) and stored as
    float32; the output transform evaluated in the sum precision and rounded once to the
    storage dtype.  Mode "fp32" stores U, V, M and y in float32 and carries every sum in float64
    (see _stage_dtypes).  Non-finite values propagate (Section C.4 "Saturation").
    """
    r = np.asarray(g).shape[1]
    AT, G, BT = coefficient_tables(m, points, mode, coef, scales, r=r)
    x = np.asarray(x)
    N, H, W, C = x.shape
    st, ev = _stage_dtypes(mode)
    with np.errstate(all="ignore"):
        U = _two_sided(G, np.asarray(g), (1, 2), ev).astype(st).astype(ev)
        d = _gather_tiles(x.astype(ev), m, r)
        V = _two_sided(BT, d, (3, 4), ev).astype(st).astype(ev)
        n = m + r - 1
        Th, Tw = d.shape[1], d.shape[2]
        K = U.shape[0]
        M = np.empty((N, Th, Tw, n, n, K), dtype=np.float32)
        for p in range(n):
            for q in range(n):
                M[:, :, :, p, q, :] = V[:, :, :, p, q, :] @ U[:, p, q, :].T     # summed in ev, stored float32
        Y = _two_sided(AT, M, (3, 4), ev)
        y = _scatter_tiles(Y, H, W)
        if apply_relu:
            y = np.where(y < 0, ev(0), y)   # negative -> 0; NaN and +inf pass through
        y = y.astype(st)
    return y


# --------------------------------------------------------------------------
# INT8 Winograd-domain pipeline (Section 5.1 "INT8 Setup"; Appendix "INT8 Convolution Error
# Validation"; Section "Rational Coefficients in Practice")
# --------------------------------------------------------------------------
def quantize_int8(v, scale):
    """Symmetric quantiser: round(v / scale) to nearest, ties to even, saturated to [-128, 127]
    (Section 5.1 "INT8 Setup": s = max|.|/127; the plain definition).  The quotient is one float32
    division and the rounding decision is taken on that float32 value.  scale may be an array
    broadcastable against v; a zero scale (an all-zero tensor) is treated as 1."""
    v = np.asarray(v, dtype=np.float32)
    s = np.asarray(scale, dtype=np.float32)
    s = np.where(s == 0, np.float32(1), s)
    q = np.rint((v / s).astype(np.float32))             # float32 quotient; rint = ties to even
    return np.clip(q, -128, 127).astype(np.int8)


def int8_scale(absmax):
    """s = max|.| / 127 in float32 (Section 5.1: "s = max(|w|)/127")."""
    return (np.asarray(absmax, dtype=np.float32) / np.float32(127)).astype(np.float32)


def winograd_conv_int8_emulated(x, g, m, points, per_channel=False, scale_U=None, scale_V=None,
                                coef="fp32", apply_relu=False, scales=(None, None), return_parts=False):
    """The four steps with the Winograd-domain tensors quantised to int8.

    The transform matrices stay in floating point (float32 tables by default, as the paper's
    note on rational coefficients states; coef="mode" rounds them through float16 like the
    half pipeline).  U = G g G^T and V = B^T d B are evaluated in float32 and quantised
    symmetrically: U with one scale per tensor, or one per output channel k when per_channel
    (s = max|.|/127 over the tensor / the channel's slice); V with one scale for the whole batch.
    scale_U (array of K) / scale_V (number) override the data-derived scales ("static" scales).
    The product over input channels is exact integer arithmetic (int32 on the device); it is
    converted to float32, multiplied by the float32 product s_U[k] * s_V, and the output
    transform is evaluated in float32 and rounded once to float16.
    """
    r = np.asarray(g).shape[1]
    AT, G, BT = coefficient_tables(m, points, "fp16", coef, scales, r=r)
    x = np.asarray(x)
    N, H, W, C = x.shape
    with np.errstate(all="ignore"):
        U = _two_sided(G, np.asarray(g), (1, 2), np.float32)                  # [K,n,n,C]
        K = U.shape[0]
        if scale_U is None:
            amax = np.abs(U).max(axis=(1, 2, 3)) if per_channel else np.full(K, np.abs(U).max(), np.float32)
            sU = int8_scale(amax)
        else:
            sU = np.broadcast_to(np.asarray(scale_U, dtype=np.float32), (K,)).copy()
        sU = np.where(sU == 0, np.float32(1), sU).astype(np.float32)
        Uq = quantize_int8(U, sU[:, None, None, None])
        d = _gather_tiles(x.astype(np.float32), m, r)
        V = _two_sided(BT, d, (3, 4), np.float32)                              # [N,Th,Tw,n,n,C]
        sV = int8_scale(np.abs(V).max()) if scale_V is None else np.float32(scale_V)
        if sV == 0:
            sV = np.float32(1)
        Vq = quantize_int8(V, sV)
        n = m + r - 1
        Th, Tw = d.shape[1], d.shape[2]
        Mi = np.empty((N, Th, Tw, n, n, K), dtype=np.int64)
        for p in range(n):
            for q in range(n):
                # exact: |sum| <= C * 128 * 128 < 2^53
                Mi[:, :, :, p, q, :] = np.rint(Vq[:, :, :, p, q, :].astype(np.float64) @ Uq[:, p, q, :].astype(np.float64).T)
        s = (sU * sV).astype(np.float32)                                        # one float32 product per filter
        Mf = Mi.astype(np.float32) * s                                          # int -> float32 (RNE), then one multiply
        Y = _two_sided(AT, Mf, (3, 4), np.float32)
        y = _scatter_tiles(Y, H, W)
        if apply_relu:
            y = np.where(y < 0, np.float32(0), y)
        y = y.astype(np.float16)
    if return_parts:
        return y, {"Uq": Uq, "scale_U": sU, "Vq": Vq, "scale_V": sV, "M": Mi}
    return y


# --------------------------------------------------------------------------
# VGG-16 convolution stack
# --------------------------------------------------------------------------
def vgg_stack_fp64(x, weights, layers):
    """conv3x3 -> ReLU (-> 2x2 max-pool) for each layer, all in float64."""
    a = np.asarray(x, dtype=np.float64)
    for gw, (_, _, pool) in zip(weights, layers):
        a = relu(direct_conv_fp64(a, gw))
        if pool:
            a = maxpool2x2(a)
    return a


def vgg_stack_emulated(x, weights, layers, m, points, mode="fp16", coef="mode"):
    """Same stack through the emulated Winograd pipeline; activations are stored
    in the storage dtype between layers."""
    a = np.asarray(x)
    for gw, (_, _, pool) in zip(weights, layers):
        a = winograd_conv_emulated(a, gw, m, points, mode, coef, apply_relu=True)
        if pool:
            with np.errstate(all="ignore"):
                a = maxpool2x2(a)
    return a
