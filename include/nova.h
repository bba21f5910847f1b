/*
 * nova.h - C ABI of the B200 (sm_100a) Winograd convolution library.
 *
 * 2-D Winograd convolution F(m x m, 3 x 3), m in {2, 4, 6, 8}, driven by an
 * arbitrary set of interpolation points (possibly fractional) with the point
 * at infinity, as in Section 2.1 ("Winograd Convolution via Cook-Toom") of
 * "NOVA: Discovering Well-Conditioned Winograd Transforms through Numerical
 * Optimization of Vandermonde Arithmetic".
 *
 * Fixed semantics: cross-correlation y_i = sum_k g_k x_{i+k} (Section 2.1),
 * stride 1, zero padding 1, dilation 1, groups 1, tensors NHWC:
 *   x [N,H,W,C]   g [K,3,3,C]   y [N,H,W,K],  C % 8 == 0 and K % 8 == 0.
 * The image is cut into ceil(H/m) x ceil(W/m) tiles; tile (th, tw) reads the
 * n x n patch (n = m + 2) whose top-left corner is (m*th - 1, m*tw - 1) of the
 * zero-extended image; outputs beyond H x W are dropped.
 *
 * Every function returns an int status (0 = NOVA_OK, negative = error) unless
 * stated otherwise; nothing throws or aborts across this boundary.  Pointers
 * named *_dev are device pointers, *_host host pointers; the caller owns every
 * buffer.  Device work is enqueued on `stream` (a cudaStream_t passed as
 * void*) and is asynchronous.  There is no CPU fallback: without a CUDA device
 * the device entry points return NOVA_ERR_CUDA.  A plan belongs to the device
 * that was current when it was created (its status word and tables live
 * there); a device entry point called with another device current returns
 * NOVA_ERR_INVALID_ARG.
 */
#ifndef NOVA_H_
#define NOVA_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

/* A point alpha = num/den (den > 0).  den == 0 denotes the point at infinity,
 * projective (1:0) (Section 2.4, "Symbolic Verification"). */
typedef struct { int64_t num, den; } nova_rat;

/* Arithmetic mode.  NOVA_FP32: x, g, y and the stored intermediates (U, V, M) are float; every
 * stored element is one rounding of a sum carried in double (with float sums the F(8,3) tile
 * would not reach a relative error of 1e-4 even on well-conditioned points); accuracy path.
 * NOVA_FP16_F32ACC: x, g, y are IEEE half; transforms are evaluated in float
 * and rounded once to half; the transformed-domain product accumulates in
 * float (Section 5.1 "FP16 Setup"; Appendix "Float16 Precision Analysis"). */
enum { NOVA_FP32 = 0, NOVA_FP16_F32ACC = 1 };

/* Precision of the transform coefficient tables in NOVA_FP16_F32ACC mode:
 * rounded to half then widened (the paper's "cast to FP16"), or float. */
enum { NOVA_COEF_ROUND_TO_MODE = 0, NOVA_COEF_FP32 = 1 };

/* nova_conv2d_fwd flags (bitwise or). */
enum {
  NOVA_RELU = 1,            /* y = (v < 0) ? 0 : v after the output transform */
  NOVA_GEMM_SIMT = 1 << 8,  /* force the CUDA-core product kernel (fp16 mode; testing) */
  NOVA_GEMM_TCGEN05 = 2 << 8, /* force the tcgen05 tensor-core product kernel */
  NOVA_PROFILE_WAITS = 1 << 13, /* measurement aid: the tensor-core product kernel (half mode, K > 128) runs in a
                                   variant that sums the cycles its warps spend waiting; read them with
                                   nova_plan_wait_profile.  A few per cent slower; results unchanged */
  NOVA_POOL2X2 = 1 << 14,   /* 2 x 2 max-pool, stride 2, fused into the output transform (after the ReLU if
                               both are given): y_dev is [N, H/2, W/2, K]; the result equals nova_maxpool2x2
                               of the unpooled output.  H and W even; NOVA_FP16_F32ACC with the default
                               (TMA-staged) output transform only, NOVA_ERR_UNSUPPORTED otherwise; also
                               accepted by nova_conv2d_fwd_static, _host (y_host and y_stage pooled) and
                               the INT8 entry points */
  NOVA_TRANSFORM_SIMT = 1 << 10 /* plain transform kernels: the input transform on CUDA cores even
                                   where the tensor-core formulation applies, the output transform
                                   without TMA staging (testing) */
};

/* How nova_filter_transform_int8 obtains the scales of the transformed filter. */
enum {
  NOVA_QUANT_PER_TENSOR = 0,   /* one scale, max|U| / 127 over the whole tensor (written to all K entries) */
  NOVA_QUANT_PER_CHANNEL = 1,  /* one scale per output channel k, max over that channel's slice / 127 */
  NOVA_QUANT_GIVEN = 2         /* scale_U_dev already holds K scales chosen by the caller */
};

enum {
  NOVA_OK = 0,
  NOVA_ERR_INVALID_ARG = -1,        /* null / misaligned pointer, bad shape, m not in {2,4,6,8}, n != m+r-1 */
  NOVA_ERR_NO_INFINITY = -2,        /* the point set has no point at infinity */
  NOVA_ERR_MULTIPLE_INFINITY = -3,  /* more than one, or infinity not last */
  NOVA_ERR_DUPLICATE_POINT = -4,    /* finite points must be distinct (Theorem A.2) */
  NOVA_ERR_RATIONAL_OVERFLOW = -5,  /* an exact matrix entry does not fit 127-bit rationals */
  NOVA_ERR_VERIFY_FAILED = -6,      /* the exact decomposition identity is not zero */
  NOVA_ERR_UNSUPPORTED = -7,        /* r != 3, or an unsupported mode on this path */
  NOVA_ERR_CUDA = -8,               /* a CUDA runtime/driver call failed (or no device) */
  NOVA_ERR_DEVICE_TIMEOUT = -9,     /* a bounded device-side wait expired */
  NOVA_ERR_WORKSPACE = -10,         /* workspace too small or misaligned */
  NOVA_ERR_STATIC_LIMIT = -11       /* problem needs more than NOVA_STATIC_SCRATCH_BYTES of built-in scratch */
};

typedef struct nova_plan nova_plan;   /* opaque; immutable after creation */
typedef void* nova_stream;            /* a cudaStream_t */

/*
 * Build the transform matrices for F(m, r) from `n` points (n == m + r - 1),
 * exactly one of which - the last - is infinity.  Algorithm 3 ("Symbolic
 * Cook-Toom Construction"): Lagrange factors F_i = prod_{j!=i}(a_i - a_j);
 * A^T[i][p] = a_p^i (infinity column e_{m-1}); G[p][k] = a_p^k / F_p (infinity
 * row e_{r-1}); B^T[p][:] = ascending coefficients of prod_{j!=p}(t - a_j)
 * (infinity row: prod_j (t - a_j)).  All entries are computed as exact
 * rationals, the decomposition identity of Section 2.4 is checked to be
 * exactly zero, and the tables are then rounded (rational -> double -> float
 * or half, round to nearest even).  Host only: works without a CUDA device.
 * r = 3 plans have every kernel.  r = 5 (F(2,5), F(4,5), F(6,5); the appendix's 5 x 5
 * extension; g is then [K,5,5,C] and the padding 2) runs the filter transforms and the
 * convolutions, INT8 pipeline included, with the same kernels instantiated for n = m + 4.
 * On success *out must be released with nova_plan_destroy.
 */
int nova_plan_create(int m, int r, const nova_rat* points_host, int n,
                     int mode, int coef, nova_plan** out);
void nova_plan_destroy(nova_plan* plan);

/*
 * The same construction with a diagonal rescaling (the form Y = D_A A^T [(D_G G g) (.) (D_B B^T d)]
 * of the appendix comparing learned-scale methods): row p of G is multiplied by scale_G[p], row p of
 * B^T by scale_B[p] and column p of A^T by 1 / (scale_G[p] scale_B[p]), so that D_A D_G D_B = I and
 * the exact identity still holds (it is checked again).  Either scale array may be null (all ones);
 * each holds n non-zero finite rationals, the last one for the point at infinity.  Scales that differ
 * within a +-pair, or whose product scale_G scale_B is not 1 at the point 0 or at infinity, make the
 * plan non-symmetric (dense transforms, same results).  Powers of two change no rounding,
 * only the range of U and V - e.g. to keep a large tile inside binary16.
 */
int nova_plan_create_scaled(int m, int r, const nova_rat* points_host, int n,
                            const nova_rat* scale_G_host, const nova_rat* scale_B_host,
                            int mode, int coef, nova_plan** out);

/*
 * Snap-to-rational (Algorithm 2; definition in Section "Snap-to-Rational"): the a/b with
 * 1 <= b <= max_den and |a| <= 5 b closest to x, compared exactly; of equally close candidates the
 * one met first when b, then a, increase.  Returned in lowest terms.  1 <= max_den <= 4096.
 */
int nova_snap_to_rational(double x, int max_den, nova_rat* out);

/*
 * Symmetric search (Section "Symmetric Search"): among the point sets made of pairs (p, -p), plus 0
 * when n_finite is odd, with p a positive fraction of denominator <= max_den and p <= max_abs, the
 * one whose Vandermonde matrix has the lowest kappa_2; every combination is evaluated.
 * points_out receives n_finite + 1 points in the order 0, +p1, -p1, .. (p1 < p2 < ..), infinity;
 * *kappa2_out (may be null) the winning condition number.  With max_den = 6 and max_abs = 2 the
 * search returns the paper's discovered sets for F(4,3), F(6,3) and F(8,3) (n_finite = 5, 7, 9).
 * NOVA_ERR_UNSUPPORTED if more than four million combinations would have to be tried.
 */
int nova_symmetric_search(int n_finite, int max_den, int max_abs, nova_rat* points_out, double* kappa2_out);

/* Snap n_finite continuous points (the paper uses max_den = 10), append infinity and build the
 * plan; NOVA_ERR_DUPLICATE_POINT if two points snap to the same rational. */
int nova_plan_create_f64(int m, int r, const double* finite_points_host, int n_finite, int max_den,
                         int mode, int coef, nova_plan** out);

/* The exact verifier of Section 2.4 on caller-supplied matrices (row-major AT [m*n], G [n*r],
 * BT [n*n], n == m + r - 1 <= 64, denominators > 0): NOVA_OK iff
 * sum_p AT[i][p] G[p][k] BT[p][j] == [j == i + k] for all i, k, j in exact arithmetic,
 * NOVA_ERR_VERIFY_FAILED otherwise. */
int nova_verify_decomposition(int m, int r, int n, const nova_rat* AT_host, const nova_rat* G_host,
                              const nova_rat* BT_host);

/* The exact matrices as reduced fractions (same shapes and order as nova_plan_get_matrices);
 * NOVA_ERR_RATIONAL_OVERFLOW if an entry does not fit 64-bit numerator and denominator. */
int nova_plan_get_matrices_rational(const nova_plan* plan, nova_rat* AT_host, nova_rat* G_host, nova_rat* BT_host);

/* kappa_2 and spectral norm of A, G, B in that order (three doubles each; either may be null) -
 * the per-matrix table of "Transform Matrix Analysis (A, B, G)" and the norm
 * product of the forward error bound ("Norm Products" paragraph). */
int nova_plan_kappa_matrices(const nova_plan* plan, double* kappa2_host, double* norm2_host);

/* Copy the fp64 tables, row-major, in the caller's point order:
 * AT [m*n], G [n*r], BT [n*n].  Any pointer may be null. */
int nova_plan_get_matrices(const nova_plan* plan, double* AT_host, double* G_host, double* BT_host);

/* The tables as the kernels use them (after rounding to the coefficient
 * precision), as float, same shapes. */
int nova_plan_get_device_tables(const nova_plan* plan, float* AT_host, float* G_host, float* BT_host);

/* The library indexes the n*n transformed-domain coordinates ("frequencies") of U in an
 * internal point order: frequency (xi, nu) of U is the pair of caller points
 * (perm_host[xi], perm_host[nu]).  For a set that is symmetric about 0 ({0, +-a_1, ..,
 * +-a_q, infinity}, as every set in the paper is, given in any order) the internal order is 0,
 * +a_1, -a_1, .., infinity - the pairs in the order in which their first member appears in the
 * caller's list - and *symmetric_host is 1: the transforms then share the even/odd partial sums
 * of each +-pair and skip the structural zeros (Appendix A, "symmetric point sets").
 * Any other set keeps the caller's order and dense transforms.  Either pointer may be null. */
int nova_plan_frequency_order(const nova_plan* plan, int* perm_host, int* symmetric_host);

/* kappa_2 = sigma_max/sigma_min of the Vandermonde matrix V_ij = a_i^j over the
 * n-1 finite points only (Section 2.2, "Vandermonde Conditioning"). */
int nova_plan_kappa(const nova_plan* plan, double* kappa2_V_host);

/* Bytes of the transformed filter U for K filters of C channels. */
size_t nova_filter_transform_bytes(const nova_plan* plan, int K, int C);

/*
 * Kernel transform (Section 2.1 step 2, nested in 2-D as in Appendix B.5):
 * U = G g G^T for every (k, c), evaluated in float and rounded once to the
 * operand type.  g_dev [K,3,3,C] (half or float per the plan's mode);
 * U_dev receives a library-defined layout ([n*n][K][C], operand type) of
 * nova_filter_transform_bytes() bytes, 16-byte aligned.
 */
int nova_filter_transform(const nova_plan* plan, const void* g_dev, int K, int C,
                          void* U_dev, nova_stream stream);

/* Scratch (device global memory) nova_conv2d_fwd wants for this problem; any
 * size >= nova_conv2d_min_workspace_bytes() works (the batch of tiles is then
 * processed in more, smaller chunks). */
size_t nova_conv2d_workspace_bytes(const nova_plan* plan, int N, int H, int W, int C, int K);
size_t nova_conv2d_min_workspace_bytes(const nova_plan* plan, int N, int H, int W, int C, int K);

/*
 * Forward convolution (Section 2.1 steps 1, 3, 4; 2-D form
 * Y = A^T [ (G g G^T) (.) (B^T d B) ] A summed over input channels):
 * input-tile transform V = B^T d B (float, rounded once to the operand type),
 * transformed-domain product M[f] = V[f] U[f]^T for each of the n*n
 * frequencies f (float accumulation; tcgen05 tensor cores in fp16 mode), and
 * output transform Y = A^T M A (float, rounded once to the storage type).
 * x_dev [N,H,W,C], y_dev [N,H,W,K] in the storage type, 16-byte aligned;
 * U_dev from nova_filter_transform with the same plan, K and C.
 * workspace_dev: 256-byte aligned scratch of workspace_bytes; contents are
 * undefined afterwards (the kernels tell the L2 to drop its lines unwritten once
 * they have been read); calls sharing a workspace must be stream-ordered.
 * With C = 8 (NOVA_FP16_F32ACC, 3-tap filters, none of NOVA_GEMM_SIMT, NOVA_GEMM_TCGEN05,
 * NOVA_TRANSFORM_SIMT, NOVA_PROFILE_WAITS) the three steps run in ONE kernel that keeps V and M
 * on the SM: same arithmetic and rounding points, one launch, workspace checked but not touched
 * (problems of 2^31 tiles or more stay on the three-kernel path).
 */
int nova_conv2d_fwd(const nova_plan* plan, const void* x_dev, const void* U_dev, void* y_dev,
                    int N, int H, int W, int C, int K,
                    void* workspace_dev, size_t workspace_bytes, int flags, nova_stream stream);

/*
 * Measurement aid: the same work as nova_conv2d_fwd with CUDA events recorded
 * on `stream` around each kernel; synchronises the stream and writes the summed
 * device time in milliseconds of the three kernel classes to kernel_ms_host[0..2]
 * (input transform, transformed-domain product, output transform); the one-kernel
 * path of C = 8 reports its time as the product's and 0 for the transforms.
 */
int nova_conv2d_fwd_timed(const nova_plan* plan, const void* x_dev, const void* U_dev, void* y_dev,
                          int N, int H, int W, int C, int K,
                          void* workspace_dev, size_t workspace_bytes, int flags, nova_stream stream,
                          float* kernel_ms_host);

/*
 * The same call for host tensors: x_host is copied to x_stage_dev, convolved into
 * y_stage_dev and copied to y_host.  The batch is cut into up to eight groups of
 * images so that the copy in, the kernels and the copy out of different groups
 * overlap: the copies run on two streams the library creates once per device, the
 * kernels on `stream`; all of it is ordered after the work already in `stream`, and
 * `stream` waits for the last copy.  The staging buffers are device memory of the
 * sizes of x and y, the workspace as for nova_conv2d_fwd.  Host buffers must be
 * page-locked for the copies to overlap.  The first call on a device creates the
 * streams and events; calls from several host threads are serialised.
 */
int nova_conv2d_fwd_host(const nova_plan* plan, const void* x_host, const void* U_dev, void* y_host,
                         int N, int H, int W, int C, int K,
                         void* x_stage_dev, void* y_stage_dev,
                         void* workspace_dev, size_t workspace_bytes, int flags, nova_stream stream);

/*
 * Forward convolution for callers that cannot allocate device memory.
 * (The paper has no counterpart: this is a packaging variant of
 * nova_conv2d_fwd, same arithmetic, same kernels.)
 *
 * Some hosts of this library hand it tensors but own no allocator it may
 * call: a plug-in running inside another framework's memory pool, a
 * real-time loop that forbids cudaMalloc after start-up because it
 * synchronises the device, or a sandbox where only pre-mapped buffers exist.
 * They have nowhere to get the scratch that nova_conv2d_fwd asks for.  This
 * entry point brings its own: a fixed array of NOVA_STATIC_SCRATCH_BYTES of
 * device global memory that is part of the library image.  Every GPU that
 * loads the library keeps that array until the process exits, used or not.
 *
 * The caller still passes x_dev, U_dev and y_dev exactly as for
 * nova_conv2d_fwd.  The call makes no cudaMalloc / cudaFree and calls no
 * allocating routine.  A problem whose smallest chunk (128 tiles, or all of
 * them if fewer) does not fit the array - nova_conv2d_min_workspace_bytes() >
 * NOVA_STATIC_SCRATCH_BYTES - is refused with NOVA_ERR_STATIC_LIMIT and nothing
 * is launched; larger problems that fit are processed in more, smaller chunks.
 *
 * The first call on each device looks up the array's device address (a
 * symbol query, with that device current) and keeps it; make that first call
 * outside any stream capture.  All calls on one device share the one array
 * and it keeps whatever the previous call left there; every kernel writes
 * the part it later reads, so nothing needs clearing, but two calls whose
 * kernels overlap on the GPU (different streams without ordering) race on
 * it: order them.
 */
#define NOVA_STATIC_SCRATCH_BYTES ((size_t)32 << 20)
int nova_conv2d_fwd_static(const nova_plan* plan, const void* x_dev, const void* U_dev, void* y_dev,
                           int N, int H, int W, int C, int K, int flags, nova_stream stream);

/* Number of kernel launches one nova_conv2d_fwd call issues for this problem
 * and workspace size (negative = error). */
int nova_conv2d_launch_count(const nova_plan* plan, int N, int H, int W, int C, int K,
                             size_t workspace_bytes, int flags);

/*
 * INT8 Winograd-domain pipeline (Section 5.1 "INT8 Setup"; appendix "INT8 Convolution Error
 * Validation"; Section "Snap-to-Rational", paragraph "Rational Coefficients in Practice").  The
 * transform matrices stay in floating point (create the plan with NOVA_FP16_F32ACC and, as the
 * paper does, NOVA_COEF_FP32); the transformed filter U and the transformed input V are
 * quantised symmetrically to signed 8 bit - code = round-to-nearest-even(value * (1 / s))
 * saturated to [-128, 127], s = max|value| / 127, the reciprocal taken once per scale in float -
 * the product over the input
 * channels is exact int32 arithmetic on the tensor cores (tcgen05 kind::i8), and the output
 * transform runs in float on float(M) * (s_U[k] * s_V), rounded once to half.  x, g and y are
 * half tensors as in nova_conv2d_fwd (g is [K,5,5,C] for a plan with r = 5).  C and K must be
 * multiples of 16.
 *
 * nova_filter_transform_int8: g [K,3,3,C] half -> Uq (nova_filter_transform_int8_bytes() bytes,
 * opaque layout) and scale_U_dev[K] floats (device).  quant: one of NOVA_QUANT_*.
 */
size_t nova_filter_transform_int8_bytes(const nova_plan* plan, int K, int C);
int nova_filter_transform_int8(const nova_plan* plan, const void* g_dev, int K, int C, int quant,
                               void* Uq_dev, float* scale_U_dev, nova_stream stream);

/*
 * nova_conv2d_fwd_int8: scale_V > 0 is a static (calibrated) scale for the transformed input;
 * scale_V == 0 derives it from the data, max|V| / 127 over the whole batch, which costs a second
 * pass of the input transform.  The workspace (nova_conv2d_int8_workspace_bytes(), 256-byte
 * aligned) holds Vq, the int32 product and the scale; the whole batch is processed in one piece
 * (NOVA_ERR_WORKSPACE if it does not fit).  flags: NOVA_RELU; NOVA_GEMM_SIMT selects an exact
 * CUDA-core product (cross-check).  The scale used is left in the first float of the workspace.
 * Asynchronous on `stream`; allocates nothing.
 */
size_t nova_conv2d_int8_workspace_bytes(const nova_plan* plan, int N, int H, int W, int C, int K);
int nova_conv2d_fwd_int8(const nova_plan* plan, const void* x_dev, const void* Uq_dev,
                         const float* scale_U_dev, float scale_V, void* y_dev,
                         int N, int H, int W, int C, int K,
                         void* workspace_dev, size_t workspace_bytes, int flags, nova_stream stream);
/* The same with one CUDA event pair per kernel; ms_host[4] receives the input transform (all its
 * passes), the product, the output transform and the total, in milliseconds.  Synchronises. */
int nova_conv2d_fwd_int8_timed(const nova_plan* plan, const void* x_dev, const void* Uq_dev,
                               const float* scale_U_dev, float scale_V, void* y_dev,
                               int N, int H, int W, int C, int K,
                               void* workspace_dev, size_t workspace_bytes, int flags, nova_stream stream,
                               float* ms_host);

/*
 * Self-test of the failure reporting (no counterpart in the paper).  Every wait inside the
 * kernels is bounded by the clock; when one expires the kernel records NOVA_ERR_DEVICE_TIMEOUT in
 * the plan's status word and returns normally.  This call launches one warp that waits, with a
 * limit of limit_ms (1..1000) milliseconds, on a barrier that nothing completes, so that the path
 * from an expired wait to nova_last_device_status can be exercised on a healthy GPU.
 * *waited_ns_host receives the time the warp waited.  Synchronises `stream`; allocates one word.
 */
int nova_selftest_wait_timeout(const nova_plan* plan, unsigned limit_ms, unsigned long long* waited_ns_host,
                               nova_stream stream);

/*
 * Measurement aid (no counterpart in the paper): the rate at which the multiprocessors move bytes
 * to and from the L2 / device memory with one kind of access, timed with CUDA events.  The
 * transformed input and the transformed-domain product of the pipeline above cross that path
 * twice each, so these rates bound it.  One persistent CTA on each of `ctas` multiprocessors walks
 * `bytes` (a multiple of 16 KiB, at least 128 KiB) `iters` times:
 *   kind 0 vector loads; 1 vector stores; 2 half the warps load and half store;
 *   3 bulk asynchronous copies global -> shared, `depth` (1..12) 16 KiB pieces in flight per CTA;
 *   4 kind 3 plus vector stores from the other warps; 5 bulk copies shared -> global; 6 kinds 3 + 5.
 * Kinds 0-2 move `bytes` per iteration in total; 4 and 6 move `bytes` in each direction.
 * src_dev (read) and dst_dev (written, contents undefined afterwards) are 128-byte aligned device
 * buffers of `bytes`.  *ms_host receives the time of the `iters` passes.  Must run on the plan's
 * device; synchronises `stream`; allocates 64 bytes for the duration of the call.
 */
int nova_probe_fabric(const nova_plan* plan, int kind, const void* src_dev, void* dst_dev, size_t bytes,
                      int iters, int ctas, int depth, float* ms_host, nova_stream stream);

/*
 * Measurement aid (no counterpart in the paper): where the transformed-domain product kernel of the
 * last nova_conv2d_fwd call with NOVA_PROFILE_WAITS spent its time.  cycles_host receives 9 doubles,
 * SM clock cycles averaged over the CTAs that ran:
 *   [0] TMA producer warp waiting for a free ring stage      [1] its total
 *   [2] MMA warp waiting for a free TMEM accumulator         [3] MMA warp waiting for operands in the ring
 *   [4] MMA warp total                                       [5] an epilogue warp waiting for a finished accumulator
 *   [6] that epilogue warp's total (the rest of it is spent storing M)
 *   [7] work items per CTA                                   [8] number of CTAs
 * Synchronises `stream`.  The counters are the plan's: not thread-safe against a concurrent profiled call.
 */
int nova_plan_wait_profile(const nova_plan* plan, double* cycles_host, nova_stream stream);

/* 2x2 max pooling, stride 2, NHWC, H and W even, C % 8 == 0 (used between the
 * blocks of a VGG-style stack; not part of the paper's method).  `mode`
 * selects half or float elements. */
int nova_maxpool2x2(const void* x_dev, void* y_dev, int N, int H, int W, int C,
                    int mode, nova_stream stream);

/*
 * Device-side health: every wait inside the kernels is bounded; a wait that
 * expires records NOVA_ERR_DEVICE_TIMEOUT in a plan-owned device word.  This
 * call synchronises `stream`, reads and clears that word, and returns it (or
 * NOVA_ERR_CUDA if the stream reports an error).
 */
int nova_last_device_status(const nova_plan* plan, nova_stream stream);

/* The raw cudaError_t value of the last CUDA call that made a convolution entry point return
 * NOVA_ERR_CUDA (0 if none so far); not thread-safe, for diagnostics. */
int nova_last_cuda_error(void);

const char* nova_status_string(int status);

#ifdef __cplusplus
}
#endif
#endif  /* NOVA_H_ */
