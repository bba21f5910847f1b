// Transformed-domain product on CUDA cores (Section 2.1 step 3, summed over
// input channels): for every frequency f,
//   M[f][p][k] = sum_c V[f][p][c] * U[f][k][c],
// stored as float [f][K/4][pc_pad][4] like the tensor-core kernel's output.
// This is the product kernel of the fp32 mode (a single-pass TF32 tensor-core
// product cannot meet a 1e-5 tolerance) and a cross-check for the tcgen05
// kernel in fp16 mode.  Half operands accumulate in float (their products are
// exact in float); float operands accumulate in double and the sum is rounded
// once to float, like every stored tensor of the fp32 mode.
#include <cuda_fp16.h>
#include <cuda_runtime.h>

#include "nova_internal.h"

namespace nova {
namespace {

constexpr int BM = 64, BN = 64, BK = 16;

__device__ __forceinline__ float to_f(float v) { return v; }
__device__ __forceinline__ float to_f(__half v) { return __half2float(v); }
template <typename T> struct AccOf { using type = float; };
template <> struct AccOf<float> { using type = double; };
__device__ __forceinline__ float mac(float a, float b, float c) { return fmaf(a, b, c); }
__device__ __forceinline__ double mac(float a, float b, double c) { return fma((double)a, (double)b, c); }

// 256 threads, each a 4 x 4 block of the 64 x 64 output tile.
template <typename T>
__global__ void __launch_bounds__(256)
gemm_simt_kernel(const T* __restrict__ V, const T* __restrict__ U, float* __restrict__ Mo,
                 int pc, int pc_pad, int C, int K) {
  __shared__ float sV[BK][BM + 4];
  __shared__ float sU[BK][BN + 4];
  const int f = blockIdx.z;
  const int pb = blockIdx.x * BM, kb = blockIdx.y * BN;
  const T* Vf = V + (size_t)f * pc_pad * C;
  const T* Uf = U + (size_t)f * K * C;
  float* Mf = Mo + (size_t)f * pc_pad * K;             // [K/4][pc_pad][4]
  const int tid = threadIdx.x;
  const int tx = tid & 15, ty = tid >> 4;           // tx -> k, ty -> p
  const int lr = tid >> 2, lc = (tid & 3) * 4;      // loader: row 0..63, 4 channels at lc
  using Acc = typename AccOf<T>::type;
  Acc acc[4][4] = {};
  for (int c0 = 0; c0 < C; c0 += BK) {
#pragma unroll
    for (int e = 0; e < 4; ++e) {
      const int c = c0 + lc + e;
      const int p = pb + lr, k = kb + lr;
      sV[lc + e][lr] = (p < pc && c < C) ? to_f(Vf[(size_t)p * C + c]) : 0.f;
      sU[lc + e][lr] = (k < K && c < C) ? to_f(Uf[(size_t)k * C + c]) : 0.f;
    }
    __syncthreads();
#pragma unroll
    for (int kk = 0; kk < BK; ++kk) {
      float a[4], b[4];
#pragma unroll
      for (int i = 0; i < 4; ++i) a[i] = sV[kk][ty * 4 + i];
#pragma unroll
      for (int j = 0; j < 4; ++j) b[j] = sU[kk][tx * 4 + j];
#pragma unroll
      for (int i = 0; i < 4; ++i)
#pragma unroll
        for (int j = 0; j < 4; ++j) acc[i][j] = mac(a[i], b[j], acc[i][j]);
    }
    __syncthreads();
  }
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    const int p = pb + ty * 4 + i;
    if (p >= pc) continue;
    const int k = kb + tx * 4;                        // K % 8 == 0: a filter quad is all in or all out
    if (k < K)
      *reinterpret_cast<float4*>(Mf + ((size_t)(k >> 2) * pc_pad + p) * 4) =
          make_float4((float)acc[i][0], (float)acc[i][1], (float)acc[i][2], (float)acc[i][3]);
  }
}

// The int8 product on CUDA cores (cross-check of the kind::i8 tensor-core kernel): one thread per
// (tile, filter quad), four dp4a-free integer dot products over the channels.  Exact.
__global__ void __launch_bounds__(256)
gemm_simt_i8_kernel(const int8_t* __restrict__ V, const int8_t* __restrict__ U, int32_t* __restrict__ Mo,
                    int pc, int pc_pad, int C, int K) {
  const int f = blockIdx.z;
  const int p = blockIdx.x * blockDim.x + threadIdx.x;
  const int k = blockIdx.y * 4;
  if (p >= pc || k >= K) return;
  const int8_t* v = V + ((size_t)f * pc_pad + p) * C;
  const int8_t* u = U + ((size_t)f * K + k) * C;
  int acc[4] = {0, 0, 0, 0};
  for (int c = 0; c < C; ++c) {
    const int a = v[c];
#pragma unroll
    for (int j = 0; j < 4; ++j) acc[j] += a * (int)u[(size_t)j * C + c];
  }
  *reinterpret_cast<int4*>(Mo + (((size_t)f * (K >> 2) + (k >> 2)) * pc_pad + p) * 4) =
      make_int4(acc[0], acc[1], acc[2], acc[3]);
}

}  // namespace

int launch_gemm_simt_i8(const void* V, const void* U, int32_t* M, int nfreq, int pc, int pc_pad, int C, int K,
                        void* stream) {
  dim3 grid((pc + 255) / 256, K / 4, nfreq);
  gemm_simt_i8_kernel<<<grid, 256, 0, (cudaStream_t)stream>>>((const int8_t*)V, (const int8_t*)U, M, pc, pc_pad,
                                                              C, K);
  return (int)cudaGetLastError();
}

int launch_gemm_simt(const nova_plan* plan, const void* V, const void* U, float* M, int nfreq, int pc,
                     int pc_pad, int C, int K, void* stream) {
  dim3 grid((pc + BM - 1) / BM, (K + BN - 1) / BN, nfreq);
  if (plan->mode == NOVA_FP32)
    gemm_simt_kernel<float><<<grid, 256, 0, (cudaStream_t)stream>>>((const float*)V, (const float*)U, M, pc,
                                                                    pc_pad, C, K);
  else
    gemm_simt_kernel<__half><<<grid, 256, 0, (cudaStream_t)stream>>>((const __half*)V, (const __half*)U, M,
                                                                     pc, pc_pad, C, K);
  return (int)cudaGetLastError();
}

}  // namespace nova
