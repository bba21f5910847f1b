// Transform kernels of the Winograd pipeline (Section 2.1 steps 1, 2 and 4 in
// their 2-D nested form, Appendix B.5): U = G g G^T, V = B^T d B, Y = A^T M A.
// Half storage: each is evaluated in float from coefficient tables held in the constant bank
// (a __grid_constant__ parameter) and rounded once to half (or quantised, for the int8
// pipeline).  The fp32 mode's transforms are in fp32_path.cu.
#include <cuda_fp16.h>
#include <cuda_runtime.h>

#include "nova_internal.h"
#include "transform_math.cuh"

namespace nova {
namespace {

using namespace xf;

// Where the float results of a transform go.  StoreSink rounds them to the operand type;
// AbsmaxSink only reduces them to their largest magnitude (first pass of a data-derived int8
// scale s = max|.| / 127); QuantSink multiplies by the reciprocal of a scale read from device
// memory, rounds to nearest even and saturates to [-128, 127] (the symmetric quantiser of the INT8 set-up,
// Section 5.1).  Offsets are in elements of the destination.
template <typename T>
struct StoreSink {
  T* out;
  __device__ __forceinline__ void begin(int) {}
  __device__ __forceinline__ void put(size_t off, float2 v) { st2(out + off, v); }
  __device__ __forceinline__ void finish() {}
};
struct AbsmaxSink {
  unsigned* slots;     // non-negative floats order like their bit patterns
  int per_channel;
  float mx;
  unsigned* slot;
  __device__ __forceinline__ void begin(int channel) { mx = 0.f; slot = slots + (per_channel ? channel : 0); }
  __device__ __forceinline__ void put(size_t, float2 v) { mx = fmaxf(mx, fmaxf(fabsf(v.x), fabsf(v.y))); }
  __device__ __forceinline__ void finish() {
    if (per_channel) {
      atomicMax(slot, __float_as_uint(mx));
    } else {
      const unsigned act = __activemask();
      const unsigned m = __reduce_max_sync(act, __float_as_uint(mx));
      if ((threadIdx.x & 31) == (unsigned)(__ffs(act) - 1)) atomicMax(slot, m);
    }
  }
};
// v times the reciprocal scale, rounded to nearest even and saturated to [-128, 127]
__device__ __forceinline__ int quant_code(float v, float r) {
  int q;
  asm("cvt.rni.sat.s8.f32 %0, %1;" : "=r"(q) : "f"(__fmul_rn(v, r)));
  return q;
}
struct QuantSink {
  int8_t* out;
  const float* scales;
  int per_channel;
  float s;
  __device__ __forceinline__ void begin(int channel) {
    s = scales[per_channel ? channel : 0];
    if (s == 0.f) s = 1.f;
    s = __fdiv_rn(1.f, s);                              // the quantiser multiplies by the reciprocal
  }
  __device__ __forceinline__ void put(size_t off, float2 v) {
    char2 q;
    q.x = (signed char)quant_code(v.x, s);
    q.y = (signed char)quant_code(v.y, s);
    *reinterpret_cast<char2*>(out + off) = q;
  }
  __device__ __forceinline__ void finish() {}
};

// absmax slots -> scales, in place: s = max / 127 (float division); per tensor, slot 0 is
// copied to all `count` entries.  One block.
__global__ void scales_from_absmax_kernel(float* slots, int count, int per_channel) {
  const float m0 = slots[0];
  __syncthreads();
  for (int i = threadIdx.x; i < count; i += blockDim.x) {
    const float m = per_channel ? slots[i] : m0;
    slots[i] = __fdiv_rn(m, 127.f);
  }
}
__global__ void set_scale_kernel(float* slot, float value) { *slot = value; }

// ---------------------------------------------------------------- U = G g G^T
// One thread per (filter k, channel pair).  g [K,3,3,C] -> U [n*n][K][C].
template <int M, typename T, typename Sink, int R = 3>
__global__ void __launch_bounds__(256)
filter_transform_kernel(const __grid_constant__ Coefs cf, const T* __restrict__ g, Sink sink,
                        int K, int C) {
  constexpr int N = M + R - 1;
  const int c2 = C >> 1;
  const long long idx = (long long)blockIdx.x * blockDim.x + threadIdx.x;
  if (idx >= (long long)K * c2) return;
  const int k = (int)(idx / c2);
  const int c = (int)(idx % c2) * 2;
  sink.begin(k);
  float2 gg[R][R];
#pragma unroll
  for (int a = 0; a < R; ++a)
#pragma unroll
    for (int b = 0; b < R; ++b) gg[a][b] = ld2(g + ((size_t)(k * R + a) * R + b) * C + c);
  float2 t[N][R];
#pragma unroll
  for (int p = 0; p < N; ++p)
#pragma unroll
    for (int b = 0; b < R; ++b) {
      float2 s = mul2(cf.G[p][0], gg[0][b]);
#pragma unroll
      for (int a = 1; a < R; ++a) s = fma2(cf.G[p][a], gg[a][b], s);
      t[p][b] = s;
    }
#pragma unroll
  for (int p = 0; p < N; ++p)
#pragma unroll
    for (int q = 0; q < N; ++q) {
      float2 s = mul2(cf.G[q][0], t[p][0]);
#pragma unroll
      for (int b = 1; b < R; ++b) s = fma2(cf.G[q][b], t[p][b], s);
      sink.put(((size_t)(p * N + q) * K + k) * C + c, s);
    }
  sink.finish();
}

// ---------------------------------------------------------------- V = B^T d B
// x [N,H,W,C] -> V [n*n][pc_pad][C] for the tiles p0 .. p0+pc-1.  A thread owns one
// (tile, channel pair) and one group of two B^T rows: it applies those two rows along the
// patch's columns (nu), keeps the n x 2 intermediate in registers, applies all n rows along
// the patch's rows (xi) and stores the 2n frequencies (xi, nu in its group).  The n/2 groups
// of a patch are rows of the grid: the patch comes from DRAM once and from L2 for the other groups.
template <int M, typename T, bool SYM, int G, typename Sink, int R = 3>
__device__ __forceinline__ void input_transform_group(const Coefs& cf, const T* __restrict__ x,
                                                      Sink& V, int H, int W, int C, int h0,
                                                      int w0, long long img, size_t out_off,
                                                      size_t f_stride) {
  constexpr int N = M + R - 1;
  constexpr int RA = (G == 0) ? 0 : 2 * G - 1;
  constexpr int RB = (G == 0) ? N - 1 : 2 * G;
  float2 ta[N], tb[N];
  const bool interior = h0 >= 0 && w0 >= 0 && h0 + N <= H && w0 + N <= W;
  if (interior) {
    const T* base = x + (((size_t)img * H + h0) * W + w0) * C;
#pragma unroll
    for (int a = 0; a < N; ++a) {
      float2 d[N];
#pragma unroll
      for (int b = 0; b < N; ++b) d[b] = ld2(base + ((size_t)a * W + b) * C);
      bt_two_rows<N, SYM, G>(cf, d, ta[a], tb[a]);
    }
  } else {
#pragma unroll
    for (int a = 0; a < N; ++a) {
      const int h = h0 + a;
      const bool hv = (h >= 0) && (h < H);
      float2 d[N];
#pragma unroll
      for (int b = 0; b < N; ++b) {
        const int w = w0 + b;
        d[b] = make_float2(0.f, 0.f);
        if (hv && w >= 0 && w < W) d[b] = ld2(x + (((size_t)img * H + h) * W + w) * C);
      }
      bt_two_rows<N, SYM, G>(cf, d, ta[a], tb[a]);
    }
  }
  float2 oa[N], ob[N];
  bt_all_rows<N, SYM>(cf, ta, oa);
  bt_all_rows<N, SYM>(cf, tb, ob);
#pragma unroll
  for (int xi = 0; xi < N; ++xi) {
    V.put(out_off + (size_t)(xi * N + RA) * f_stride, oa[xi]);
    V.put(out_off + (size_t)(xi * N + RB) * f_stride, ob[xi]);
  }
}

template <int M, typename T, bool SYM, typename Sink, int R = 3>
__global__ void __launch_bounds__(128)
input_transform_kernel(const __grid_constant__ Coefs cf, const T* __restrict__ x, Sink V,
                       int H, int W, int C, int Th, int Tw, long long p0, int pc, int pc_pad) {
  constexpr int N = M + R - 1;
  constexpr int PAD = (R - 1) / 2;
  constexpr int WORK = 128;                       // (tile, channel pair) items per block
  // threads [g*128, g*128+128) form group g (warp-uniform)
  // blockIdx.y is the group of B^T rows: every warp of a block - and, since blocks are handed out
  // with x fastest, nearly every block resident at a time - runs the same unrolled code, which
  // keeps it in the instruction cache (with all groups in one block the kernel spent most of its
  // issue slots waiting for instructions).
  const int g = blockIdx.y;
  const int c2 = C >> 1;
  const long long idx = (long long)blockIdx.x * WORK + threadIdx.x;
  if (idx >= (long long)pc * c2) return;
  const int pl = (int)(idx / c2);
  const int c = (int)(idx % c2) * 2;
  const long long p = p0 + pl;
  const int tw = (int)(p % Tw);
  const int th = (int)((p / Tw) % Th);
  const long long img = p / ((long long)Tw * Th);
  const int h0 = M * th - PAD, w0 = M * tw - PAD;
  const size_t out_off = (size_t)pl * C + c;
  const size_t f_stride = (size_t)pc_pad * C;
  const T* xc = x + c;
  V.begin(0);
  switch (g) {
    case 0: input_transform_group<M, T, SYM, 0, Sink, R>(cf, xc, V, H, W, C, h0, w0, img, out_off, f_stride); break;
    case 1: input_transform_group<M, T, SYM, 1, Sink, R>(cf, xc, V, H, W, C, h0, w0, img, out_off, f_stride); break;
    case 2: if constexpr (N >= 6) input_transform_group<M, T, SYM, 2, Sink, R>(cf, xc, V, H, W, C, h0, w0, img, out_off, f_stride); break;
    case 3: if constexpr (N >= 8) input_transform_group<M, T, SYM, 3, Sink, R>(cf, xc, V, H, W, C, h0, w0, img, out_off, f_stride); break;
    case 4: if constexpr (N >= 10) input_transform_group<M, T, SYM, 4, Sink, R>(cf, xc, V, H, W, C, h0, w0, img, out_off, f_stride); break;
  }
  V.finish();
}

// ---------------------------------------------------------------- Y = A^T M A
// M is stored [n*n][K/4][pc_pad][4] (filter quads outermost, then tiles): the product kernel
// writes it and this kernel reads it in 32-byte pieces.  A thread owns one tile and VEC
// consecutive filters; a warp covers 2 tiles x 16 such units, so that its M reads are whole
// 32-byte sectors and its y stores are 32*VEC contiguous bytes per pixel.
template <int M, typename T, bool SYM, int VEC, int R = 3>
__global__ void __launch_bounds__(256, (M == 8 || VEC == 1) ? 2 : 2)
output_transform_kernel(const __grid_constant__ Coefs cf, const float* __restrict__ Mb,
                        T* __restrict__ y, int H, int W, int K, int Th, int Tw, long long p0, int pc,
                        int pc_pad, int relu) {
  constexpr int N = M + R - 1;
  using Vv = typename VecOf<VEC>::type;
  const int t = threadIdx.x;
  const int unit = blockIdx.x * 128 + (t & 15) + 16 * (t >> 5);
  const int pl = blockIdx.y * 2 + ((t >> 4) & 1);
  const int k = unit * VEC;
  if (k >= K || pl >= pc) return;
  const long long p = p0 + pl;
  const int tw = (int)(p % Tw);
  const int th = (int)((p / Tw) % Th);
  const long long img = p / ((long long)Tw * Th);
  const size_t f_stride = (size_t)(K >> 2) * pc_pad * 4;
  const float* src = Mb + ((size_t)(k >> 2) * pc_pad + pl) * 4 + (k & 3);

  Vv Y[M][M];
  auto load_row = [&](int xi, Vv (&z)[M]) {
    Vv in[N];
#pragma unroll
    for (int nu = 0; nu < N; ++nu) in[nu] = *reinterpret_cast<const Vv*>(src + (size_t)(xi * N + nu) * f_stride);
    at_apply<M, SYM, Vv, N>(cf, in, z);
  };
  if constexpr (!SYM) {
#pragma unroll
    for (int i = 0; i < M; ++i)
#pragma unroll
      for (int j = 0; j < M; ++j) Y[i][j] = vzero<Vv>();
#pragma unroll
    for (int xi = 0; xi < N; ++xi) {
      Vv z[M];
      load_row(xi, z);
#pragma unroll
      for (int i = 0; i < M; ++i)
#pragma unroll
        for (int j = 0; j < M; ++j) Y[i][j] = vfma(cf.AT[i][xi], z[j], Y[i][j]);
    }
  } else {
    // A^T column 0 is e_0 and column n-1 is e_{m-1}; columns +a / -a share |coefficients|.
    {
      Vv zp[M], zm[M];
      load_row(1, zp);
      load_row(2, zm);
#pragma unroll
      for (int j = 0; j < M; ++j) {
        const Vv s = vadd(zp[j], zm[j]), d = vsub(zp[j], zm[j]);
#pragma unroll
        for (int i = 0; i < M; ++i) Y[i][j] = vmul(cf.AT[i][1], (i & 1) ? d : s);
      }
    }
#pragma unroll
    for (int q = 3; q < N - 1; q += 2) {
      Vv zp[M], zm[M];
      load_row(q, zp);
      load_row(q + 1, zm);
#pragma unroll
      for (int j = 0; j < M; ++j) {
        const Vv s = vadd(zp[j], zm[j]), d = vsub(zp[j], zm[j]);
#pragma unroll
        for (int i = 0; i < M; ++i) Y[i][j] = vfma(cf.AT[i][q], (i & 1) ? d : s, Y[i][j]);
      }
    }
    {
      Vv z0[M], zi[M];
      load_row(0, z0);
      load_row(N - 1, zi);
#pragma unroll
      for (int j = 0; j < M; ++j) {
        Y[0][j] = vadd(Y[0][j], z0[j]);
        Y[M - 1][j] = vadd(Y[M - 1][j], zi[j]);
      }
    }
  }
#pragma unroll
  for (int i = 0; i < M; ++i) {
    const int h = M * th + i;
    if (h >= H) continue;
#pragma unroll
    for (int j = 0; j < M; ++j) {
      const int w = M * tw + j;
      if (w >= W) continue;
      Vv v = Y[i][j];
      if (relu) v = vrelu(v);                     // NaN and +inf pass through
      vstore(y + (((size_t)img * H + h) * W + w) * K + k, v);
    }
  }
}

// ---------------------------------------------------------------- max pooling
template <typename T>
__device__ __forceinline__ T max_nan(T a, T b);
template <>
__device__ __forceinline__ float max_nan<float>(float a, float b) {
  return (a != a) ? a : ((b != b) ? b : fmaxf(a, b));
}
template <>
__device__ __forceinline__ __half max_nan<__half>(__half a, __half b) { return __hmax_nan(a, b); }

template <typename T>
__global__ void __launch_bounds__(256)
maxpool2x2_kernel(const T* __restrict__ x, T* __restrict__ y, int N, int H, int W, int C) {
  constexpr int VEC = 16 / sizeof(T);
  const int Ho = H >> 1, Wo = W >> 1, cv = C / VEC;
  const long long total = (long long)N * Ho * Wo * cv;
  const long long idx = (long long)blockIdx.x * blockDim.x + threadIdx.x;
  if (idx >= total) return;
  const int c = (int)(idx % cv) * VEC;
  const int wo = (int)((idx / cv) % Wo);
  const int ho = (int)((idx / ((long long)cv * Wo)) % Ho);
  const long long img = idx / ((long long)cv * Wo * Ho);
  union Pack { uint4 u; T e[VEC]; };
  Pack r[4];
#pragma unroll
  for (int q = 0; q < 4; ++q) {
    const int h = 2 * ho + (q >> 1), w = 2 * wo + (q & 1);
    r[q].u = *reinterpret_cast<const uint4*>(x + (((size_t)img * H + h) * W + w) * C + c);
  }
  Pack o;
#pragma unroll
  for (int e = 0; e < VEC; ++e)
    o.e[e] = max_nan<T>(max_nan<T>(r[0].e[e], r[1].e[e]), max_nan<T>(r[2].e[e], r[3].e[e]));
  *reinterpret_cast<uint4*>(y + (((size_t)img * Ho + ho) * Wo + wo) * C + c) = o.u;
}

inline unsigned blocks_for(long long work, int threads) {
  return (unsigned)((work + threads - 1) / threads);
}

template <int M, typename T>
int filter_launch(const nova_plan* plan, const void* g, int K, int C, void* U, cudaStream_t s) {
  const long long work = (long long)K * (C / 2);
  if (plan->r == 5) {
    if constexpr (M <= 6)
      filter_transform_kernel<M, T, StoreSink<T>, 5><<<blocks_for(work, 256), 256, 0, s>>>(
          plan->kcoefs, (const T*)g, StoreSink<T>{(T*)U}, K, C);
    else
      return (int)cudaErrorInvalidValue;
    return (int)cudaGetLastError();
  }
  filter_transform_kernel<M, T, StoreSink<T>><<<blocks_for(work, 256), 256, 0, s>>>(
      plan->kcoefs, (const T*)g, StoreSink<T>{(T*)U}, K, C);
  return (int)cudaGetLastError();
}
// int8 filter transform: absmax pass (unless the scales are given), scales, quantising pass.
template <int M, typename T>
int filter_launch_int8(const nova_plan* plan, const void* g, int K, int C, void* Uq, float* scales, int quant,
                       cudaStream_t s) {
  const long long work = (long long)K * (C / 2);
  const int per_channel = (quant & NOVA_QUANT_PER_CHANNEL) ? 1 : 0;
  const bool r5 = plan->r == 5;
  if (r5 && M > 6) return (int)cudaErrorInvalidValue;
  if (!(quant & NOVA_QUANT_GIVEN)) {
    cudaError_t e = cudaMemsetAsync(scales, 0, sizeof(float) * K, s);
    if (e != cudaSuccess) return (int)e;
    const AbsmaxSink sink{(unsigned*)scales, per_channel, 0.f, nullptr};
    if (r5) {
      if constexpr (M <= 6)
        filter_transform_kernel<M, T, AbsmaxSink, 5><<<blocks_for(work, 256), 256, 0, s>>>(plan->kcoefs, (const T*)g, sink, K, C);
    } else {
      filter_transform_kernel<M, T, AbsmaxSink><<<blocks_for(work, 256), 256, 0, s>>>(plan->kcoefs, (const T*)g, sink, K, C);
    }
    scales_from_absmax_kernel<<<1, 256, 0, s>>>(scales, K, per_channel);
  }
  const QuantSink qsink{(int8_t*)Uq, scales, 1, 0.f};
  if (r5) {
    if constexpr (M <= 6)
      filter_transform_kernel<M, T, QuantSink, 5><<<blocks_for(work, 256), 256, 0, s>>>(plan->kcoefs, (const T*)g, qsink, K, C);
  } else {
    filter_transform_kernel<M, T, QuantSink><<<blocks_for(work, 256), 256, 0, s>>>(plan->kcoefs, (const T*)g, qsink, K, C);
  }
  return (int)cudaGetLastError();
}
// int8 input transform over tiles p0 .. p0+pc-1.  pass 0: absmax into *slot (zeroed by the caller);
// pass 1: quantise with the scale at *slot.
template <int M, typename T>
int input_launch_int8(const nova_plan* plan, const Geom& g, const void* x, void* Vq, float* slot, int pass,
                      long long p0, int pc, int pc_pad, cudaStream_t s) {
  constexpr int THREADS = 128;
  const long long work = (long long)pc * (g.C / 2);
  const dim3 grid(blocks_for(work, 128), (M + 2) / 2);      // y: one block row per group of two B^T rows
#define NOVA_IT8(SYMV, SINK, ...)                                                                         \
  input_transform_kernel<M, T, SYMV, SINK><<<grid, THREADS, 0, s>>>(plan->kcoefs, (const T*)x, __VA_ARGS__, g.H, \
                                                                   g.W, g.C, g.Th, g.Tw, p0, pc, pc_pad)
#define NOVA_IT8R5(SYMV, SINK, ...)                                                                       \
  input_transform_kernel<M, T, SYMV, SINK, 5><<<grid5, THREADS, 0, s>>>(plan->kcoefs, (const T*)x, __VA_ARGS__, g.H, \
                                                                       g.W, g.C, g.Th, g.Tw, p0, pc, pc_pad)
  if (plan->r == 5) {
    if constexpr (M <= 6) {
      const dim3 grid5(blocks_for(work, 128), (M + 4) / 2);
      if (pass == 0) {
        if (plan->symmetric) NOVA_IT8R5(true, AbsmaxSink, AbsmaxSink{(unsigned*)slot, 0, 0.f, nullptr});
        else NOVA_IT8R5(false, AbsmaxSink, AbsmaxSink{(unsigned*)slot, 0, 0.f, nullptr});
      } else {
        if (plan->symmetric) NOVA_IT8R5(true, QuantSink, QuantSink{(int8_t*)Vq, slot, 0, 0.f});
        else NOVA_IT8R5(false, QuantSink, QuantSink{(int8_t*)Vq, slot, 0, 0.f});
      }
      return (int)cudaGetLastError();
    } else {
      return (int)cudaErrorInvalidValue;
    }
  }
  if (pass == 0) {
    if (plan->symmetric) NOVA_IT8(true, AbsmaxSink, AbsmaxSink{(unsigned*)slot, 0, 0.f, nullptr});
    else NOVA_IT8(false, AbsmaxSink, AbsmaxSink{(unsigned*)slot, 0, 0.f, nullptr});
  } else {
    if (plan->symmetric) NOVA_IT8(true, QuantSink, QuantSink{(int8_t*)Vq, slot, 0, 0.f});
    else NOVA_IT8(false, QuantSink, QuantSink{(int8_t*)Vq, slot, 0, 0.f});
  }
#undef NOVA_IT8
#undef NOVA_IT8R5
  return (int)cudaGetLastError();
}
template <int M, typename T>
int input_launch(const nova_plan* plan, const Geom& g, const void* x, void* V, long long p0, int pc,
                 int pc_pad, cudaStream_t s) {
  constexpr int THREADS = 128;
  const long long work = (long long)pc * (g.C / 2);
  const dim3 grid(blocks_for(work, 128), (M + 2) / 2);      // y: one block row per group of two B^T rows
  const dim3 grid5(blocks_for(work, 128), (M + 4) / 2);
  if (plan->r == 5) {                               // 5-tap filters: n = m + 4 points
    if constexpr (M <= 6) {
      if (plan->symmetric)
        input_transform_kernel<M, T, true, StoreSink<T>, 5><<<grid5, THREADS, 0, s>>>(
            plan->kcoefs, (const T*)x, StoreSink<T>{(T*)V}, g.H, g.W, g.C, g.Th, g.Tw, p0, pc, pc_pad);
      else
        input_transform_kernel<M, T, false, StoreSink<T>, 5><<<grid5, THREADS, 0, s>>>(
            plan->kcoefs, (const T*)x, StoreSink<T>{(T*)V}, g.H, g.W, g.C, g.Th, g.Tw, p0, pc, pc_pad);
    } else {
      return (int)cudaErrorInvalidValue;
    }
    return (int)cudaGetLastError();
  }
  if (plan->symmetric)
    input_transform_kernel<M, T, true, StoreSink<T>><<<grid, THREADS, 0, s>>>(
        plan->kcoefs, (const T*)x, StoreSink<T>{(T*)V}, g.H, g.W, g.C, g.Th, g.Tw, p0, pc, pc_pad);
  else
    input_transform_kernel<M, T, false, StoreSink<T>><<<grid, THREADS, 0, s>>>(
        plan->kcoefs, (const T*)x, StoreSink<T>{(T*)V}, g.H, g.W, g.C, g.Th, g.Tw, p0, pc, pc_pad);
  return (int)cudaGetLastError();
}
template <int M, typename T>
int output_launch(const nova_plan* plan, const Geom& g, const void* Mb, void* y, long long p0, int pc,
                  int pc_pad, int relu, cudaStream_t s) {
  constexpr int VEC = (M == 8) ? 1 : 2;
  dim3 grid(blocks_for(g.K / VEC, 128), (unsigned)((pc + 1) / 2));
  if (plan->r == 5) {
    if constexpr (M <= 6) {
      constexpr int V5 = (M == 6) ? 1 : 2;            // n = 10 at m = 6: registers as for F(8,3)
      dim3 grid5(blocks_for(g.K / V5, 128), (unsigned)((pc + 1) / 2));
      if (plan->symmetric)
        output_transform_kernel<M, T, true, V5, 5><<<grid5, 256, 0, s>>>(
            plan->kcoefs, (const float*)Mb, (T*)y, g.H, g.W, g.K, g.Th, g.Tw, p0, pc, pc_pad, relu);
      else
        output_transform_kernel<M, T, false, V5, 5><<<grid5, 256, 0, s>>>(
            plan->kcoefs, (const float*)Mb, (T*)y, g.H, g.W, g.K, g.Th, g.Tw, p0, pc, pc_pad, relu);
    } else {
      return (int)cudaErrorInvalidValue;
    }
    return (int)cudaGetLastError();
  }
  if (plan->symmetric)
    output_transform_kernel<M, T, true, VEC><<<grid, 256, 0, s>>>(
        plan->kcoefs, (const float*)Mb, (T*)y, g.H, g.W, g.K, g.Th, g.Tw, p0, pc, pc_pad, relu);
  else
    output_transform_kernel<M, T, false, VEC><<<grid, 256, 0, s>>>(
        plan->kcoefs, (const float*)Mb, (T*)y, g.H, g.W, g.K, g.Th, g.Tw, p0, pc, pc_pad, relu);
  return (int)cudaGetLastError();
}

}  // namespace

// Half storage only: the fp32 mode has its own transform kernels.
#define NOVA_DISPATCH_M_T(FN, ...)                                                   \
  do {                                                                               \
    if (plan->mode == NOVA_FP32) return (int)cudaErrorInvalidValue;                  \
    switch (plan->m) {                                                               \
      case 2: return FN<2, __half>(__VA_ARGS__);                                     \
      case 4: return FN<4, __half>(__VA_ARGS__);                                     \
      case 6: return FN<6, __half>(__VA_ARGS__);                                     \
      case 8: return FN<8, __half>(__VA_ARGS__);                                     \
    }                                                                                \
    return (int)cudaErrorInvalidValue;                                               \
  } while (0)

int launch_filter_transform(const nova_plan* plan, const void* g, int K, int C, void* U, void* stream) {
  NOVA_DISPATCH_M_T(filter_launch, plan, g, K, C, U, (cudaStream_t)stream);
}
int launch_input_transform(const nova_plan* plan, const Geom& g, const void* x, void* V, long long p0,
                           int pc, int pc_pad, void* stream) {
  NOVA_DISPATCH_M_T(input_launch, plan, g, x, V, p0, pc, pc_pad, (cudaStream_t)stream);
}
int launch_output_transform(const nova_plan* plan, const Geom& g, const void* M, void* y, long long p0,
                            int pc, int pc_pad, int relu, void* stream) {
  NOVA_DISPATCH_M_T(output_launch, plan, g, M, y, p0, pc, pc_pad, relu, (cudaStream_t)stream);
}
int launch_filter_transform_int8(const nova_plan* plan, const void* g, int K, int C, void* Uq, float* scales,
                                 int quant, void* stream) {
  NOVA_DISPATCH_M_T(filter_launch_int8, plan, g, K, C, Uq, scales, quant, (cudaStream_t)stream);
}
int launch_input_transform_int8(const nova_plan* plan, const Geom& g, const void* x, void* Vq, float* slot,
                                int pass, long long p0, int pc, int pc_pad, void* stream) {
  NOVA_DISPATCH_M_T(input_launch_int8, plan, g, x, Vq, slot, pass, p0, pc, pc_pad, (cudaStream_t)stream);
}
int launch_scale_slot(float* slot, float value, int from_absmax, void* stream) {
  if (from_absmax) scales_from_absmax_kernel<<<1, 32, 0, (cudaStream_t)stream>>>(slot, 1, 0);
  else set_scale_kernel<<<1, 1, 0, (cudaStream_t)stream>>>(slot, value);
  return (int)cudaGetLastError();
}
int launch_maxpool2x2(const void* x, void* y, int N, int H, int W, int C, int mode, void* stream) {
  const bool f32 = mode == NOVA_FP32;
  const int vec = f32 ? 4 : 8;
  const long long work = (long long)N * (H / 2) * (W / 2) * (C / vec);
  if (f32)
    maxpool2x2_kernel<float><<<blocks_for(work, 256), 256, 0, (cudaStream_t)stream>>>(
        (const float*)x, (float*)y, N, H, W, C);
  else
    maxpool2x2_kernel<__half><<<blocks_for(work, 256), 256, 0, (cudaStream_t)stream>>>(
        (const __half*)x, (__half*)y, N, H, W, C);
  return (int)cudaGetLastError();
}

}  // namespace nova
