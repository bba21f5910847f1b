// Transform kernels of the Winograd pipeline (Section 2.1 steps 1, 2 and 4 in
// their 2-D nested form, Appendix B.5): U = G g G^T, V = B^T d B, Y = A^T M A.
// Each is evaluated in float from coefficient tables held in the constant bank
// (a __grid_constant__ parameter) and rounded once to the destination type.
#include <cuda_fp16.h>
#include <cuda_runtime.h>

#include "nova_internal.h"

namespace nova {
namespace {

__device__ __forceinline__ float2 ld2(const __half* p) {
  return __half22float2(*reinterpret_cast<const __half2*>(p));
}
__device__ __forceinline__ float2 ld2(const float* p) { return *reinterpret_cast<const float2*>(p); }
__device__ __forceinline__ void st2(__half* p, float2 v) {
  *reinterpret_cast<__half2*>(p) = __floats2half2_rn(v.x, v.y);
}
__device__ __forceinline__ void st2(float* p, float2 v) { *reinterpret_cast<float2*>(p) = v; }
__device__ __forceinline__ float2 fma2(float a, float2 b, float2 c) {
  return make_float2(fmaf(a, b.x, c.x), fmaf(a, b.y, c.y));
}
__device__ __forceinline__ float2 mul2(float a, float2 b) { return make_float2(a * b.x, a * b.y); }

// ---------------------------------------------------------------- U = G g G^T
// One thread per (filter k, channel pair).  g [K,3,3,C] -> U [n*n][K][C].
template <int M, typename T>
__global__ void __launch_bounds__(256)
filter_transform_kernel(const __grid_constant__ Coefs cf, const T* __restrict__ g, T* __restrict__ U,
                        int K, int C) {
  constexpr int N = M + 2;
  const int c2 = C >> 1;
  const long long idx = (long long)blockIdx.x * blockDim.x + threadIdx.x;
  if (idx >= (long long)K * c2) return;
  const int k = (int)(idx / c2);
  const int c = (int)(idx % c2) * 2;
  float2 gg[3][3];
#pragma unroll
  for (int a = 0; a < 3; ++a)
#pragma unroll
    for (int b = 0; b < 3; ++b) gg[a][b] = ld2(g + ((size_t)(k * 3 + a) * 3 + b) * C + c);
  float2 t[N][3];
#pragma unroll
  for (int p = 0; p < N; ++p)
#pragma unroll
    for (int b = 0; b < 3; ++b) {
      float2 s = mul2(cf.G[p][0], gg[0][b]);
      s = fma2(cf.G[p][1], gg[1][b], s);
      s = fma2(cf.G[p][2], gg[2][b], s);
      t[p][b] = s;
    }
#pragma unroll
  for (int p = 0; p < N; ++p)
#pragma unroll
    for (int q = 0; q < N; ++q) {
      float2 s = mul2(cf.G[q][0], t[p][0]);
      s = fma2(cf.G[q][1], t[p][1], s);
      s = fma2(cf.G[q][2], t[p][2], s);
      st2(U + ((size_t)(p * N + q) * K + k) * C + c, s);
    }
}

// ---------------------------------------------------------------- V = B^T d B
// One thread per (tile, channel pair, column group).  x [N,H,W,C] ->
// V [n*n][pc_pad][C] for the tiles p0 .. p0+pc-1.  SPLITS threads share one
// patch; each produces the frequencies (xi, nu) with nu in its column group.
template <int M, typename T, int SPLITS, int SPLIT>
__device__ __forceinline__ void input_transform_body(const Coefs& cf, const T* __restrict__ x,
                                                     T* __restrict__ V, int H, int W, int C, int Th,
                                                     int Tw, long long p0, int pc, int pc_pad) {
  constexpr int N = M + 2;
  constexpr int NU = N / SPLITS;
  constexpr int NU0 = SPLIT * NU;
  const int c2 = C >> 1;
  const long long idx = (long long)blockIdx.x * blockDim.x + threadIdx.x;
  if (idx >= (long long)pc * c2) return;
  const int pl = (int)(idx / c2);
  const int c = (int)(idx % c2) * 2;
  const long long p = p0 + pl;
  const int tw = (int)(p % Tw);
  const int th = (int)((p / Tw) % Th);
  const long long img = p / ((long long)Tw * Th);
  const int h0 = M * th - 1, w0 = M * tw - 1;

  float2 t[N][NU];
#pragma unroll
  for (int a = 0; a < N; ++a) {
    const int h = h0 + a;
    const bool hv = (h >= 0) && (h < H);
    float2 d[N];
#pragma unroll
    for (int b = 0; b < N; ++b) {
      const int w = w0 + b;
      d[b] = make_float2(0.f, 0.f);
      if (hv && w >= 0 && w < W) d[b] = ld2(x + (((size_t)img * H + h) * W + w) * C + c);
    }
#pragma unroll
    for (int j = 0; j < NU; ++j) {
      float2 s = mul2(cf.BT[NU0 + j][0], d[0]);
#pragma unroll
      for (int b = 1; b < N; ++b) s = fma2(cf.BT[NU0 + j][b], d[b], s);
      t[a][j] = s;
    }
  }
#pragma unroll
  for (int j = 0; j < NU; ++j)
#pragma unroll
    for (int xi = 0; xi < N; ++xi) {
      float2 s = mul2(cf.BT[xi][0], t[0][j]);
#pragma unroll
      for (int a = 1; a < N; ++a) s = fma2(cf.BT[xi][a], t[a][j], s);
      st2(V + ((size_t)(xi * N + NU0 + j) * pc_pad + pl) * C + c, s);
    }
}

template <int M, typename T, int SPLITS>
__global__ void __launch_bounds__(128)
input_transform_kernel(const __grid_constant__ Coefs cf, const T* __restrict__ x, T* __restrict__ V,
                       int H, int W, int C, int Th, int Tw, long long p0, int pc, int pc_pad) {
  if constexpr (SPLITS == 1) {
    input_transform_body<M, T, 1, 0>(cf, x, V, H, W, C, Th, Tw, p0, pc, pc_pad);
  } else {
    if (blockIdx.y == 0) input_transform_body<M, T, 2, 0>(cf, x, V, H, W, C, Th, Tw, p0, pc, pc_pad);
    else input_transform_body<M, T, 2, 1>(cf, x, V, H, W, C, Th, Tw, p0, pc, pc_pad);
  }
}

// ---------------------------------------------------------------- Y = A^T M A
// One thread per (tile, filter pair).  M [n*n][pc_pad][K] float -> y [N,H,W,K].
template <int M, typename T>
__global__ void __launch_bounds__(128)
output_transform_kernel(const __grid_constant__ Coefs cf, const float* __restrict__ Mb,
                        T* __restrict__ y, int H, int W, int K, int Th, int Tw, long long p0, int pc,
                        int pc_pad, int relu) {
  constexpr int N = M + 2;
  const int k2 = K >> 1;
  const long long idx = (long long)blockIdx.x * blockDim.x + threadIdx.x;
  if (idx >= (long long)pc * k2) return;
  const int pl = (int)(idx / k2);
  const int k = (int)(idx % k2) * 2;
  const long long p = p0 + pl;
  const int tw = (int)(p % Tw);
  const int th = (int)((p / Tw) % Th);
  const long long img = p / ((long long)Tw * Th);

  float2 Y[M][M];
#pragma unroll
  for (int i = 0; i < M; ++i)
#pragma unroll
    for (int j = 0; j < M; ++j) Y[i][j] = make_float2(0.f, 0.f);

#pragma unroll
  for (int nu = 0; nu < N; ++nu) {
    float2 mm[N];
#pragma unroll
    for (int xi = 0; xi < N; ++xi)
      mm[xi] = *reinterpret_cast<const float2*>(Mb + ((size_t)(xi * N + nu) * pc_pad + pl) * K + k);
#pragma unroll
    for (int i = 0; i < M; ++i) {
      float2 z = mul2(cf.AT[i][0], mm[0]);
#pragma unroll
      for (int xi = 1; xi < N; ++xi) z = fma2(cf.AT[i][xi], mm[xi], z);
#pragma unroll
      for (int j = 0; j < M; ++j) Y[i][j] = fma2(cf.AT[j][nu], z, Y[i][j]);
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
      float2 v = Y[i][j];
      if (relu) {
        v.x = v.x < 0.f ? 0.f : v.x;   // NaN and +inf pass through
        v.y = v.y < 0.f ? 0.f : v.y;
      }
      st2(y + (((size_t)img * H + h) * W + w) * K + k, v);
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
  filter_transform_kernel<M, T><<<blocks_for(work, 256), 256, 0, s>>>(plan->coefs, (const T*)g, (T*)U, K, C);
  return (int)cudaGetLastError();
}
template <int M, typename T>
int input_launch(const nova_plan* plan, const Geom& g, const void* x, void* V, long long p0, int pc,
                 int pc_pad, cudaStream_t s) {
  const long long work = (long long)pc * (g.C / 2);
  constexpr int SPLITS = (M == 8) ? 2 : 1;
  dim3 grid(blocks_for(work, 128), SPLITS);
  input_transform_kernel<M, T, SPLITS><<<grid, 128, 0, s>>>(plan->coefs, (const T*)x, (T*)V, g.H, g.W, g.C,
                                                           g.Th, g.Tw, p0, pc, pc_pad);
  return (int)cudaGetLastError();
}
template <int M, typename T>
int output_launch(const nova_plan* plan, const Geom& g, const void* Mb, void* y, long long p0, int pc,
                  int pc_pad, int relu, cudaStream_t s) {
  const long long work = (long long)pc * (g.K / 2);
  output_transform_kernel<M, T><<<blocks_for(work, 128), 128, 0, s>>>(
      plan->coefs, (const float*)Mb, (T*)y, g.H, g.W, g.K, g.Th, g.Tw, p0, pc, pc_pad, relu);
  return (int)cudaGetLastError();
}

}  // namespace

#define NOVA_DISPATCH_M_T(FN, ...)                                                   \
  do {                                                                               \
    const bool f32 = plan->mode == NOVA_FP32;                                        \
    switch (plan->m) {                                                               \
      case 2: return f32 ? FN<2, float>(__VA_ARGS__) : FN<2, __half>(__VA_ARGS__);   \
      case 4: return f32 ? FN<4, float>(__VA_ARGS__) : FN<4, __half>(__VA_ARGS__);   \
      case 6: return f32 ? FN<6, float>(__VA_ARGS__) : FN<6, __half>(__VA_ARGS__);   \
      case 8: return f32 ? FN<8, float>(__VA_ARGS__) : FN<8, __half>(__VA_ARGS__);   \
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
