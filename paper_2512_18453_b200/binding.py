"""ctypes binding of libnova.so: argument marshalling only."""
import ctypes
import os

_HERE = os.path.dirname(os.path.abspath(__file__))
_LIB_PATH = os.path.join(_HERE, "libnova.so")

FP32, FP16_F32ACC = 0, 1
COEF_ROUND_TO_MODE, COEF_FP32 = 0, 1
RELU = 1
GEMM_SIMT = 1 << 8
GEMM_TCGEN05 = 2 << 8
TRANSFORM_SIMT = 1 << 10
PROFILE_WAITS = 1 << 13
POOL2X2 = 1 << 14

EXPORTED_SYMBOLS = (
    "nova_plan_create", "nova_plan_destroy", "nova_plan_get_matrices", "nova_plan_get_device_tables",
    "nova_plan_kappa", "nova_filter_transform_bytes", "nova_filter_transform",
    "nova_conv2d_workspace_bytes", "nova_conv2d_min_workspace_bytes", "nova_conv2d_fwd",
    "nova_conv2d_fwd_host", "nova_conv2d_fwd_timed", "nova_conv2d_launch_count", "nova_maxpool2x2", "nova_last_device_status",
    "nova_status_string", "nova_conv2d_fwd_static", "nova_plan_frequency_order", "nova_last_cuda_error",
    "nova_plan_create_scaled", "nova_plan_create_f64", "nova_snap_to_rational", "nova_verify_decomposition",
    "nova_plan_get_matrices_rational", "nova_plan_kappa_matrices", "nova_symmetric_search",
    "nova_selftest_wait_timeout", "nova_probe_fabric", "nova_plan_wait_profile",
    "nova_filter_transform_int8_bytes", "nova_filter_transform_int8", "nova_conv2d_int8_workspace_bytes",
    "nova_conv2d_fwd_int8", "nova_conv2d_fwd_int8_timed",
)
QUANT_PER_TENSOR, QUANT_PER_CHANNEL, QUANT_GIVEN = 0, 1, 2
STATIC_SCRATCH_BYTES = 32 << 20


class NovaError(RuntimeError):
    def __init__(self, status, where):
        self.status = status
        extra = " [cudaError %d]" % lib().nova_last_cuda_error() if status == -8 else ""
        super().__init__("%s: %s (%d)%s" % (where, status_string(status), status, extra))


class _Rat(ctypes.Structure):
    _fields_ = [("num", ctypes.c_int64), ("den", ctypes.c_int64)]


_lib = None


def lib():
    """Load libnova.so; there is no fallback when it is missing."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(_LIB_PATH):
        raise ImportError("libnova.so is not built; run `python -m paper_2512_18453_b200.build`")
    L = ctypes.CDLL(_LIB_PATH)
    vp, i, sz = ctypes.c_void_p, ctypes.c_int, ctypes.c_size_t
    L.nova_plan_create.argtypes = [i, i, ctypes.POINTER(_Rat), i, i, i, ctypes.POINTER(vp)]
    L.nova_plan_create.restype = i
    rp = ctypes.POINTER(_Rat)
    dp = ctypes.POINTER(ctypes.c_double)
    L.nova_plan_create_scaled.argtypes = [i, i, rp, i, rp, rp, i, i, ctypes.POINTER(vp)]
    L.nova_plan_create_scaled.restype = i
    L.nova_plan_create_f64.argtypes = [i, i, dp, i, i, i, i, ctypes.POINTER(vp)]
    L.nova_plan_create_f64.restype = i
    L.nova_snap_to_rational.argtypes = [ctypes.c_double, i, rp]
    L.nova_snap_to_rational.restype = i
    L.nova_selftest_wait_timeout.argtypes = [vp, ctypes.c_uint, ctypes.POINTER(ctypes.c_ulonglong), vp]
    L.nova_selftest_wait_timeout.restype = i
    L.nova_symmetric_search.argtypes = [i, i, i, rp, dp]
    L.nova_symmetric_search.restype = i
    L.nova_verify_decomposition.argtypes = [i, i, i, rp, rp, rp]
    L.nova_verify_decomposition.restype = i
    L.nova_plan_get_matrices_rational.argtypes = [vp, rp, rp, rp]
    L.nova_plan_get_matrices_rational.restype = i
    L.nova_plan_kappa_matrices.argtypes = [vp, dp, dp]
    L.nova_plan_kappa_matrices.restype = i
    L.nova_plan_destroy.argtypes = [vp]
    L.nova_plan_destroy.restype = None
    dp, fp = ctypes.POINTER(ctypes.c_double), ctypes.POINTER(ctypes.c_float)
    L.nova_plan_get_matrices.argtypes = [vp, dp, dp, dp]
    L.nova_plan_get_matrices.restype = i
    L.nova_plan_get_device_tables.argtypes = [vp, fp, fp, fp]
    L.nova_plan_get_device_tables.restype = i
    L.nova_plan_frequency_order.argtypes = [vp, ctypes.POINTER(i), ctypes.POINTER(i)]
    L.nova_plan_frequency_order.restype = i
    L.nova_plan_wait_profile.argtypes = [vp, ctypes.POINTER(ctypes.c_double), vp]
    L.nova_plan_wait_profile.restype = i
    L.nova_probe_fabric.argtypes = [vp, i, vp, vp, sz, i, i, i, fp, vp]
    L.nova_probe_fabric.restype = i
    L.nova_last_cuda_error.argtypes = []
    L.nova_last_cuda_error.restype = i
    L.nova_plan_kappa.argtypes = [vp, dp]
    L.nova_plan_kappa.restype = i
    L.nova_filter_transform_bytes.argtypes = [vp, i, i]
    L.nova_filter_transform_bytes.restype = sz
    L.nova_filter_transform.argtypes = [vp, vp, i, i, vp, vp]
    L.nova_filter_transform.restype = i
    for name in ("nova_conv2d_workspace_bytes", "nova_conv2d_min_workspace_bytes"):
        getattr(L, name).argtypes = [vp, i, i, i, i, i]
        getattr(L, name).restype = sz
    L.nova_conv2d_fwd.argtypes = [vp, vp, vp, vp, i, i, i, i, i, vp, sz, i, vp]
    L.nova_conv2d_fwd.restype = i
    L.nova_conv2d_fwd_timed.argtypes = [vp, vp, vp, vp, i, i, i, i, i, vp, sz, i, vp, fp]
    L.nova_conv2d_fwd_timed.restype = i
    L.nova_conv2d_fwd_host.argtypes = [vp, vp, vp, vp, i, i, i, i, i, vp, vp, vp, sz, i, vp]
    L.nova_conv2d_fwd_host.restype = i
    L.nova_conv2d_fwd_static.argtypes = [vp, vp, vp, vp, i, i, i, i, i, i, vp]
    L.nova_conv2d_fwd_static.restype = i
    cf = ctypes.c_float
    L.nova_filter_transform_int8_bytes.argtypes = [vp, i, i]
    L.nova_filter_transform_int8_bytes.restype = sz
    L.nova_filter_transform_int8.argtypes = [vp, vp, i, i, i, vp, vp, vp]
    L.nova_filter_transform_int8.restype = i
    L.nova_conv2d_int8_workspace_bytes.argtypes = [vp, i, i, i, i, i]
    L.nova_conv2d_int8_workspace_bytes.restype = sz
    L.nova_conv2d_fwd_int8.argtypes = [vp, vp, vp, vp, cf, vp, i, i, i, i, i, vp, sz, i, vp]
    L.nova_conv2d_fwd_int8.restype = i
    L.nova_conv2d_fwd_int8_timed.argtypes = [vp, vp, vp, vp, cf, vp, i, i, i, i, i, vp, sz, i, vp, fp]
    L.nova_conv2d_fwd_int8_timed.restype = i
    L.nova_conv2d_launch_count.argtypes = [vp, i, i, i, i, i, sz, i]
    L.nova_conv2d_launch_count.restype = i
    L.nova_maxpool2x2.argtypes = [vp, vp, i, i, i, i, i, vp]
    L.nova_maxpool2x2.restype = i
    L.nova_last_device_status.argtypes = [vp, vp]
    L.nova_last_device_status.restype = i
    L.nova_status_string.argtypes = [i]
    L.nova_status_string.restype = ctypes.c_char_p
    _lib = L
    return L


def status_string(status):
    return lib().nova_status_string(int(status)).decode()


def _check(status, where):
    if status != 0:
        raise NovaError(status, where)


def _stream():
    import torch
    return ctypes.c_void_p(torch.cuda.current_stream().cuda_stream)


def _torch_dtype(mode):
    import torch
    return torch.float32 if mode == FP32 else torch.float16


def _rat_array(vals):
    out = []
    for v in vals:
        if isinstance(v, tuple):
            out.append(_Rat(int(v[0]), int(v[1])))
        else:                                   # int or fractions.Fraction
            out.append(_Rat(int(v.numerator), int(v.denominator)))
    return (_Rat * len(out))(*out)


def snap_to_rational(x, max_den=10):
    """Algorithm 2 through the C ABI; returns (num, den)."""
    r = _Rat()
    _check(lib().nova_snap_to_rational(float(x), int(max_den), ctypes.byref(r)), "nova_snap_to_rational")
    return int(r.num), int(r.den)


def symmetric_search(n_finite, max_den=6, max_abs=2):
    """Best-conditioned symmetric point set on the snap grid: ([(num, den), .., (1, 0)], kappa_2)."""
    pts = (_Rat * (n_finite + 1))()
    k = ctypes.c_double()
    _check(lib().nova_symmetric_search(n_finite, max_den, max_abs, pts, ctypes.byref(k)), "nova_symmetric_search")
    return [(int(p.num), int(p.den)) for p in pts], k.value


def verify_decomposition(m, r, AT, G, BT):
    """Exact check of the bilinear identity on matrices of Fractions / (num, den) pairs; True iff it holds."""
    n = m + r - 1
    flat = lambda M: _rat_array([v for row in M for v in row])
    st = lib().nova_verify_decomposition(m, r, n, flat(AT), flat(G), flat(BT))
    if st == 0:
        return True
    if st == -6:
        return False
    _check(st, "nova_verify_decomposition")


class Plan:
    """nova_plan: transform matrices for F(m x m, 3 x 3) from a point set.

    points: list of (num, den); exactly one entry, the last, has den == 0
    (the point at infinity).
    """

    def __init__(self, m, points, mode=FP16_F32ACC, coef=COEF_ROUND_TO_MODE, r=3, scale_G=None, scale_B=None):
        arr = _rat_array(points)
        h = ctypes.c_void_p()
        if scale_G is None and scale_B is None:
            _check(lib().nova_plan_create(m, r, arr, len(points), mode, coef, ctypes.byref(h)), "nova_plan_create")
        else:
            sg = _rat_array(scale_G) if scale_G is not None else None
            sb = _rat_array(scale_B) if scale_B is not None else None
            if any(a is not None and len(a) != len(points) for a in (sg, sb)):
                raise ValueError("one scale per point")
            _check(lib().nova_plan_create_scaled(m, r, arr, len(points), sg, sb, mode, coef, ctypes.byref(h)),
                   "nova_plan_create_scaled")
        self._h = h
        self.m, self.r, self.n, self.mode, self.coef = m, r, m + r - 1, mode, coef

    @classmethod
    def from_floats(cls, m, finite_points, max_den=10, mode=FP16_F32ACC, coef=COEF_ROUND_TO_MODE, r=3):
        """Snap continuous points to simple rationals (Algorithm 2), append infinity, build the plan."""
        arr = (ctypes.c_double * len(finite_points))(*[float(v) for v in finite_points])
        h = ctypes.c_void_p()
        _check(lib().nova_plan_create_f64(m, r, arr, len(finite_points), max_den, mode, coef, ctypes.byref(h)),
               "nova_plan_create_f64")
        self = cls.__new__(cls)
        self._h = h
        self.m, self.r, self.n, self.mode, self.coef = m, r, m + r - 1, mode, coef
        return self

    def close(self):
        if getattr(self, "_h", None):
            lib().nova_plan_destroy(self._h)
            self._h = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    # ---- host side
    def matrices(self):
        import numpy as np
        AT = np.empty((self.m, self.n)); G = np.empty((self.n, self.r)); BT = np.empty((self.n, self.n))
        dp = ctypes.POINTER(ctypes.c_double)
        _check(lib().nova_plan_get_matrices(self._h, AT.ctypes.data_as(dp), G.ctypes.data_as(dp),
                                            BT.ctypes.data_as(dp)), "nova_plan_get_matrices")
        return AT, G, BT

    def matrices_rational(self):
        """Exact A^T, G, B^T as nested lists of fractions.Fraction."""
        from fractions import Fraction
        AT = (_Rat * (self.m * self.n))(); G = (_Rat * (self.n * self.r))(); BT = (_Rat * (self.n * self.n))()
        _check(lib().nova_plan_get_matrices_rational(self._h, AT, G, BT), "nova_plan_get_matrices_rational")
        shape = lambda a, rows, cols: [[Fraction(a[i * cols + j].num, a[i * cols + j].den) for j in range(cols)]
                                       for i in range(rows)]
        return shape(AT, self.m, self.n), shape(G, self.n, self.r), shape(BT, self.n, self.n)

    def kappa_matrices(self):
        """(kappa_2, spectral norm) of A, G, B: two 3-tuples."""
        k = (ctypes.c_double * 3)(); nrm = (ctypes.c_double * 3)()
        _check(lib().nova_plan_kappa_matrices(self._h, k, nrm), "nova_plan_kappa_matrices")
        return tuple(k), tuple(nrm)

    def device_tables(self):
        import numpy as np
        AT = np.empty((self.m, self.n), np.float32); G = np.empty((self.n, self.r), np.float32)
        BT = np.empty((self.n, self.n), np.float32)
        fp = ctypes.POINTER(ctypes.c_float)
        _check(lib().nova_plan_get_device_tables(self._h, AT.ctypes.data_as(fp), G.ctypes.data_as(fp),
                                                 BT.ctypes.data_as(fp)), "nova_plan_get_device_tables")
        return AT, G, BT

    def frequency_order(self):
        """(perm, symmetric): internal point i is the caller's point perm[i]."""
        perm = (ctypes.c_int * self.n)()
        sym = ctypes.c_int()
        _check(lib().nova_plan_frequency_order(self._h, perm, ctypes.byref(sym)), "nova_plan_frequency_order")
        return list(perm), bool(sym.value)

    def wait_profile(self):
        """nova_plan_wait_profile: dict of mean SM cycles per CTA of the last product kernel run with PROFILE_WAITS."""
        out = (ctypes.c_double * 9)()
        _check(lib().nova_plan_wait_profile(self._h, out, _stream()), "nova_plan_wait_profile")
        names = ("producer_wait_stage", "producer_total", "mma_wait_accumulator", "mma_wait_operands", "mma_total",
                 "epilogue_wait_accumulator", "epilogue_total", "items_per_cta", "ctas")
        return dict(zip(names, list(out)))

    def probe_fabric(self, kind, src, dst, iters=10, ctas=148, depth=8):
        """nova_probe_fabric on two uint8 CUDA tensors of equal size; returns milliseconds for `iters` passes."""
        ms = ctypes.c_float()
        _check(lib().nova_probe_fabric(self._h, kind, src.data_ptr(), dst.data_ptr(), src.numel(), iters, ctas, depth,
                                       ctypes.byref(ms), _stream()), "nova_probe_fabric")
        return ms.value

    def kappa(self):
        k = ctypes.c_double()
        _check(lib().nova_plan_kappa(self._h, ctypes.byref(k)), "nova_plan_kappa")
        return k.value

    # ---- device side (torch tensors carry the memory)
    def filter_transform_bytes(self, K, C):
        return lib().nova_filter_transform_bytes(self._h, K, C)

    def filter_transform(self, g):
        """g [K,3,3,C] on the GPU in the plan's storage dtype -> opaque U tensor."""
        import torch
        assert g.is_cuda and g.is_contiguous() and g.dtype == _torch_dtype(self.mode)
        K, _, _, C = g.shape
        U = torch.empty(self.n * self.n, K, C, dtype=g.dtype, device=g.device)
        _check(lib().nova_filter_transform(self._h, g.data_ptr(), K, C, U.data_ptr(), _stream()),
               "nova_filter_transform")
        return U

    def workspace_bytes(self, N, H, W, C, K):
        return lib().nova_conv2d_workspace_bytes(self._h, N, H, W, C, K)

    def min_workspace_bytes(self, N, H, W, C, K):
        return lib().nova_conv2d_min_workspace_bytes(self._h, N, H, W, C, K)

    def launch_count(self, N, H, W, C, K, workspace_bytes, flags=0):
        return lib().nova_conv2d_launch_count(self._h, N, H, W, C, K, workspace_bytes, flags)

    def conv2d(self, x, U, y=None, workspace=None, flags=0):
        """x [N,H,W,C], U from filter_transform -> y [N,H,W,K]."""
        import torch
        assert x.is_cuda and x.is_contiguous() and x.dtype == _torch_dtype(self.mode)
        N, H, W, C = x.shape
        K = U.shape[1]
        if y is None:
            y = torch.empty((N, H // 2, W // 2, K) if flags & POOL2X2 else (N, H, W, K), dtype=x.dtype, device=x.device)
        if workspace is None:
            workspace = torch.empty(self.workspace_bytes(N, H, W, C, K), dtype=torch.uint8, device=x.device)
        _check(lib().nova_conv2d_fwd(self._h, x.data_ptr(), U.data_ptr(), y.data_ptr(), N, H, W, C, K,
                                     workspace.data_ptr(), workspace.numel(), flags, _stream()),
               "nova_conv2d_fwd")
        return y

    def conv2d_static(self, x, U, y, flags=0):
        """nova_conv2d_fwd_static: the convolution on the library's built-in scratch.

        For callers that may not allocate device memory; `y` is therefore
        required.  Problems beyond STATIC_SCRATCH_BYTES raise NovaError(-11).
        """
        N, H, W, C = x.shape
        K = U.shape[1]
        _check(lib().nova_conv2d_fwd_static(self._h, x.data_ptr(), U.data_ptr(), y.data_ptr(), N, H, W, C, K,
                                            flags, _stream()), "nova_conv2d_fwd_static")
        return y

    def conv2d_timed(self, x, U, y, workspace, flags=0):
        """Synchronous; returns (input, product, output) kernel milliseconds."""
        N, H, W, C = x.shape
        K = U.shape[1]
        ms = (ctypes.c_float * 3)()
        _check(lib().nova_conv2d_fwd_timed(self._h, x.data_ptr(), U.data_ptr(), y.data_ptr(), N, H, W, C, K,
                                           workspace.data_ptr(), workspace.numel(), flags, _stream(), ms),
               "nova_conv2d_fwd_timed")
        return tuple(ms)

    def conv2d_host(self, x_host, U, y_host, x_stage, y_stage, workspace, flags=0):
        """Host tensors in and out (pinned for asynchronous copies)."""
        N, H, W, C = x_host.shape
        K = U.shape[1]
        _check(lib().nova_conv2d_fwd_host(self._h, x_host.data_ptr(), U.data_ptr(), y_host.data_ptr(),
                                          N, H, W, C, K, x_stage.data_ptr(), y_stage.data_ptr(),
                                          workspace.data_ptr(), workspace.numel(), flags, _stream()),
               "nova_conv2d_fwd_host")
        return y_host

    # ---- INT8 Winograd-domain pipeline
    def filter_transform_int8(self, g, quant=QUANT_PER_TENSOR, scale_U=None):
        """g [K,3,3,C] half -> (Uq int8 [n*n, K, C], scale_U float32 [K])."""
        import torch
        K, _, _, C = g.shape
        assert g.is_cuda and g.is_contiguous() and g.dtype == torch.float16
        Uq = torch.empty(lib().nova_filter_transform_int8_bytes(self._h, K, C), dtype=torch.int8, device=g.device)
        if quant == QUANT_GIVEN:
            sc = scale_U.to(device=g.device, dtype=torch.float32).contiguous()
            assert sc.numel() == K
        else:
            sc = torch.empty(K, dtype=torch.float32, device=g.device)
        _check(lib().nova_filter_transform_int8(self._h, g.data_ptr(), K, C, quant, Uq.data_ptr(), sc.data_ptr(),
                                                _stream()), "nova_filter_transform_int8")
        return Uq.view(self.n * self.n, K, C), sc

    def int8_workspace_bytes(self, N, H, W, C, K):
        return lib().nova_conv2d_int8_workspace_bytes(self._h, N, H, W, C, K)

    def conv2d_int8(self, x, Uq, scale_U, scale_V=0.0, y=None, workspace=None, flags=0, timed=False):
        """x [N,H,W,C] half -> y [N,H,W,K] half.  scale_V = 0 derives the input scale from the data.
        timed=True returns (y, [input ms, product ms, output ms, total ms])."""
        import torch
        N, H, W, C = x.shape
        K = Uq.shape[1]
        assert x.is_cuda and x.is_contiguous() and x.dtype == torch.float16 and Uq.dtype == torch.int8
        if y is None:
            y = torch.empty((N, H // 2, W // 2, K) if flags & POOL2X2 else (N, H, W, K), dtype=torch.float16, device=x.device)
        if workspace is None:
            workspace = torch.empty(self.int8_workspace_bytes(N, H, W, C, K), dtype=torch.uint8, device=x.device)
        args = (self._h, x.data_ptr(), Uq.data_ptr(), scale_U.data_ptr(), float(scale_V), y.data_ptr(),
                N, H, W, C, K, workspace.data_ptr(), workspace.numel(), flags, _stream())
        if timed:
            ms = (ctypes.c_float * 4)()
            _check(lib().nova_conv2d_fwd_int8_timed(*args, ms), "nova_conv2d_fwd_int8_timed")
            return y, list(ms)
        _check(lib().nova_conv2d_fwd_int8(*args), "nova_conv2d_fwd_int8")
        return y

    def selftest_wait_timeout(self, limit_ms=50):
        """Let one warp's bounded wait expire after limit_ms; returns the nanoseconds it waited.
        device_status() then reports (and clears) the time-out."""
        w = ctypes.c_ulonglong()
        _check(lib().nova_selftest_wait_timeout(self._h, int(limit_ms), ctypes.byref(w), _stream()),
               "nova_selftest_wait_timeout")
        return int(w.value)

    def device_status(self):
        return lib().nova_last_device_status(self._h, _stream())


def maxpool2x2(x, mode):
    import torch
    N, H, W, C = x.shape
    y = torch.empty(N, H // 2, W // 2, C, dtype=x.dtype, device=x.device)
    _check(lib().nova_maxpool2x2(x.data_ptr(), y.data_ptr(), N, H, W, C, mode, _stream()), "nova_maxpool2x2")
    return y
