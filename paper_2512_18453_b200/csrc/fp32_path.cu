// The three transforms of the fp32 mode (Section 2.1 steps 1, 2 and 4 in their 2-D nested form,
// Appendix B.5): U = G g G^T, V = B^T d B, Y = A^T M A on float tensors.
//
// In this mode every STORED tensor (U, V, M, y) is float, and each stored element is one
// rounding of a sum carried in double: what the mode loses against exact arithmetic is the float
// storage of the transformed tensors and nothing else.  With sums carried in float the F(8,3)
// tile on well-conditioned points sits at a relative error of 1.2e-4 .. 1.7e-4; this way it stays
// below 1e-4.  The kernels are plain dense products with the plan's tables (internal point
// order); they are the accuracy path, not the throughput path.
#include <cuda_runtime.h>

#include "nova_internal.h"

namespace nova {
namespace {

inline unsigned blocks_for(long long work, int threads) { return (unsigned)((work + threads - 1) / threads); }

// One thread per (filter k, channel c).  g [K,R,R,C] -> U [N*N][K][C].
template <int N, int R>
__global__ void __launch_bounds__(128)
filter_transform_f32_kernel(const __grid_constant__ Coefs cf, const float* __restrict__ g, float* __restrict__ U,
                            int K, int C) {
  const long long idx = (long long)blockIdx.x * blockDim.x + threadIdx.x;
  if (idx >= (long long)K * C) return;
  const int k = (int)(idx / C), c = (int)(idx % C);
  double t[N][R];
#pragma unroll
  for (int b = 0; b < R; ++b) {
    double col[R];
#pragma unroll
    for (int a = 0; a < R; ++a) col[a] = (double)g[((size_t)(k * R + a) * R + b) * C + c];
#pragma unroll
    for (int p = 0; p < N; ++p) {
      double s = 0.0;
#pragma unroll
      for (int a = 0; a < R; ++a) s = fma((double)cf.G[p][a], col[a], s);
      t[p][b] = s;
    }
  }
#pragma unroll
  for (int p = 0; p < N; ++p)
#pragma unroll
    for (int q = 0; q < N; ++q) {
      double s = 0.0;
#pragma unroll
      for (int b = 0; b < R; ++b) s = fma(t[p][b], (double)cf.G[q][b], s);
      U[((size_t)(p * N + q) * K + k) * C + c] = (float)s;
    }
}

// One thread per (tile, channel, nu): column nu of V for that tile and channel.
// x [N,H,W,C] -> V [N*N][pc_pad][C] for the tiles p0 .. p0+pc-1.
template <int N, int R>
__global__ void __launch_bounds__(128)
input_transform_f32_kernel(const __grid_constant__ Coefs cf, const float* __restrict__ x, float* __restrict__ V,
                           int H, int W, int C, int Th, int Tw, long long p0, int pc, int pc_pad) {
  constexpr int M = N - R + 1;
  constexpr int PAD = (R - 1) / 2;
  const int nu = blockIdx.y;
  const long long idx = (long long)blockIdx.x * blockDim.x + threadIdx.x;
  if (idx >= (long long)pc * C) return;
  const int pl = (int)(idx / C), c = (int)(idx % C);
  const long long p = p0 + pl;
  const int tw = (int)(p % Tw), th = (int)((p / Tw) % Th);
  const long long img = p / ((long long)Tw * Th);
  const int h0 = M * th - PAD, w0 = M * tw - PAD;
  double t[N];                                  // t[a] = sum_b d[a][b] B^T[nu][b]
#pragma unroll
  for (int a = 0; a < N; ++a) {
    const int h = h0 + a;
    double s = 0.0;
    if (h >= 0 && h < H) {
#pragma unroll
      for (int b = 0; b < N; ++b) {
        const int w = w0 + b;
        if (w >= 0 && w < W)
          s = fma((double)x[(((size_t)img * H + h) * W + w) * C + c], (double)cf.BT[nu][b], s);
      }
    }
    t[a] = s;
  }
#pragma unroll
  for (int xi = 0; xi < N; ++xi) {
    double s = 0.0;
#pragma unroll
    for (int a = 0; a < N; ++a) s = fma((double)cf.BT[xi][a], t[a], s);
    V[((size_t)(xi * N + nu) * pc_pad + pl) * C + c] = (float)s;
  }
}

// One thread per (tile, filter k, output column j).  M [N*N][K/4][pc_pad][4] -> y [N,H,W,K].
template <int N, int R>
__global__ void __launch_bounds__(128)
output_transform_f32_kernel(const __grid_constant__ Coefs cf, const float* __restrict__ Mb, float* __restrict__ y,
                            int H, int W, int K, int Th, int Tw, long long p0, int pc, int pc_pad, int relu) {
  constexpr int M = N - R + 1;
  const int j = blockIdx.y;
  const long long idx = (long long)blockIdx.x * blockDim.x + threadIdx.x;
  if (idx >= (long long)pc * K) return;
  // filter within its quad fastest, then the tile, then the quad: the order M is stored in
  const int k4 = (int)(idx & 3);
  const int pl = (int)((idx >> 2) % pc);
  const int kq = (int)((idx >> 2) / pc);
  const int k = kq * 4 + k4;
  const long long p = p0 + pl;
  const int tw = (int)(p % Tw), th = (int)((p / Tw) % Th);
  const long long img = p / ((long long)Tw * Th);
  const int w = M * tw + j;
  if (w >= W) return;
  const size_t f_stride = (size_t)(K >> 2) * pc_pad * 4;
  const float* src = Mb + ((size_t)kq * pc_pad + pl) * 4 + k4;
  double z[N];                                  // z[xi] = sum_nu M[xi][nu] A^T[j][nu]
#pragma unroll
  for (int xi = 0; xi < N; ++xi) {
    double s = 0.0;
#pragma unroll
    for (int nu = 0; nu < N; ++nu) s = fma((double)src[(size_t)(xi * N + nu) * f_stride], (double)cf.AT[j][nu], s);
    z[xi] = s;
  }
#pragma unroll
  for (int i = 0; i < M; ++i) {
    const int h = M * th + i;
    if (h >= H) continue;
    double s = 0.0;
#pragma unroll
    for (int xi = 0; xi < N; ++xi) s = fma((double)cf.AT[i][xi], z[xi], s);
    float v = (float)s;
    if (relu && v < 0.f) v = 0.f;               // NaN and +inf pass through
    y[(((size_t)img * H + h) * W + w) * K + k] = v;
  }
}

template <int N, int R>
int filter_go(const nova_plan* plan, const void* g, int K, int C, void* U, cudaStream_t s) {
  filter_transform_f32_kernel<N, R><<<blocks_for((long long)K * C, 128), 128, 0, s>>>(
      plan->kcoefs, (const float*)g, (float*)U, K, C);
  return (int)cudaGetLastError();
}
template <int N, int R>
int input_go(const nova_plan* plan, const Geom& g, const void* x, void* V, long long p0, int pc, int pc_pad,
             cudaStream_t s) {
  const dim3 grid(blocks_for((long long)pc * g.C, 128), N);
  input_transform_f32_kernel<N, R><<<grid, 128, 0, s>>>(plan->kcoefs, (const float*)x, (float*)V, g.H, g.W, g.C, g.Th,
                                                         g.Tw, p0, pc, pc_pad);
  return (int)cudaGetLastError();
}
template <int N, int R>
int output_go(const nova_plan* plan, const Geom& g, const void* Mb, void* y, long long p0, int pc, int pc_pad,
              int relu, cudaStream_t s) {
  const dim3 grid(blocks_for((long long)pc * g.K, 128), N - R + 1);
  output_transform_f32_kernel<N, R><<<grid, 128, 0, s>>>(plan->kcoefs, (const float*)Mb, (float*)y, g.H, g.W, g.K,
                                                          g.Th, g.Tw, p0, pc, pc_pad, relu);
  return (int)cudaGetLastError();
}

}  // namespace

// n points, r taps: (4,3) (6,3) (8,3) (10,3) and (6,5) (8,5) (10,5)
#define NOVA_F32_DISPATCH(FN, ...)                                              \
  do {                                                                          \
    if (plan->r == 3) switch (plan->n) {                                        \
        case 4: return FN<4, 3>(__VA_ARGS__);                                   \
        case 6: return FN<6, 3>(__VA_ARGS__);                                   \
        case 8: return FN<8, 3>(__VA_ARGS__);                                   \
        case 10: return FN<10, 3>(__VA_ARGS__);                                 \
      }                                                                         \
    if (plan->r == 5) switch (plan->n) {                                        \
        case 6: return FN<6, 5>(__VA_ARGS__);                                   \
        case 8: return FN<8, 5>(__VA_ARGS__);                                   \
        case 10: return FN<10, 5>(__VA_ARGS__);                                 \
      }                                                                         \
    return (int)cudaErrorInvalidValue;                                          \
  } while (0)

int launch_filter_transform_f32(const nova_plan* plan, const void* g, int K, int C, void* U, void* stream) {
  NOVA_F32_DISPATCH(filter_go, plan, g, K, C, U, (cudaStream_t)stream);
}
int launch_input_transform_f32(const nova_plan* plan, const Geom& g, const void* x, void* V, long long p0, int pc,
                               int pc_pad, void* stream) {
  NOVA_F32_DISPATCH(input_go, plan, g, x, V, p0, pc, pc_pad, (cudaStream_t)stream);
}
int launch_output_transform_f32(const nova_plan* plan, const Geom& g, const void* M, void* y, long long p0, int pc,
                                int pc_pad, int relu, void* stream) {
  NOVA_F32_DISPATCH(output_go, plan, g, M, y, p0, pc, pc_pad, relu, (cudaStream_t)stream);
}

}  // namespace nova
