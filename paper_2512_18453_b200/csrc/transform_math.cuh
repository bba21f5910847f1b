// Register-level arithmetic shared by the transform kernels: 2-vector helpers and the 1-D
// applications of the B^T and A^T tables, dense or with the even/odd structure of a point
// set that is symmetric about 0.
#pragma once
#include <cuda_fp16.h>
#include <cuda_runtime.h>

#include "nova_internal.h"

namespace nova {
namespace xf {

__device__ __forceinline__ float2 ld2(const __half* p) {
  return __half22float2(*reinterpret_cast<const __half2*>(p));
}
__device__ __forceinline__ float2 ld2(const float* p) { return *reinterpret_cast<const float2*>(p); }
__device__ __forceinline__ void st2(__half* p, float2 v) {
  *reinterpret_cast<__half2*>(p) = __floats2half2_rn(v.x, v.y);
}
__device__ __forceinline__ void st2(float* p, float2 v) { *reinterpret_cast<float2*>(p) = v; }
// The 2-vector forms use Blackwell's packed single-precision instructions (two IEEE fp32
// results per instruction, each rounded exactly like the scalar operation).
__device__ __forceinline__ float2 fma2(float a, float2 b, float2 c) {
  return __ffma2_rn(make_float2(a, a), b, c);
}
__device__ __forceinline__ float2 mul2(float a, float2 b) { return __fmul2_rn(make_float2(a, a), b); }

// Scalar / 2-vector arithmetic used by the output transform (VEC filters per thread).
template <int VEC> struct VecOf;
template <> struct VecOf<1> { using type = float; };
template <> struct VecOf<2> { using type = float2; };
template <typename V> __device__ __forceinline__ V vzero();
template <> __device__ __forceinline__ float vzero<float>() { return 0.f; }
template <> __device__ __forceinline__ float2 vzero<float2>() { return make_float2(0.f, 0.f); }
__device__ __forceinline__ float vmul(float a, float b) { return a * b; }
__device__ __forceinline__ float2 vmul(float a, float2 b) { return mul2(a, b); }
__device__ __forceinline__ float vfma(float a, float b, float c) { return fmaf(a, b, c); }
__device__ __forceinline__ float2 vfma(float a, float2 b, float2 c) { return fma2(a, b, c); }
__device__ __forceinline__ float vadd(float a, float b) { return a + b; }
__device__ __forceinline__ float2 vadd(float2 a, float2 b) { return __fadd2_rn(a, b); }
__device__ __forceinline__ float vsub(float a, float b) { return a - b; }
__device__ __forceinline__ float2 vsub(float2 a, float2 b) { return __fadd2_rn(a, make_float2(-b.x, -b.y)); }
__device__ __forceinline__ float vrelu(float v) { return v < 0.f ? 0.f : v; }
__device__ __forceinline__ float2 vrelu(float2 v) { return make_float2(v.x < 0.f ? 0.f : v.x, v.y < 0.f ? 0.f : v.y); }
__device__ __forceinline__ void vstore(__half* p, float v) { *p = __float2half_rn(v); }
__device__ __forceinline__ void vstore(float* p, float v) { *p = v; }
__device__ __forceinline__ void vstore(__half* p, float2 v) { st2(p, v); }
__device__ __forceinline__ void vstore(float* p, float2 v) { st2(p, v); }


// ---------------------------------------------------------------- 1-D building blocks
// For a point set that is symmetric about 0 (internal order 0, +a, -a, .., infinity) the
// rounded tables satisfy, entry by entry (checked when the plan is built):
//   B^T row 0 has only even columns, row n-1 only odd columns, rows +a / -a have equal even
//   columns and opposite odd columns, and no finite row reaches column n-1;
//   A^T column 0 is e_0, column n-1 is e_{m-1}, columns +a / -a are equal in even rows and
//   opposite in odd rows.
// SYM = true evaluates the same sums with the zeros skipped and the even/odd partial sums of
// a +-pair shared; SYM = false is the dense product.

// Two rows of B^T applied to one n-vector.  Group g = 0 gives rows (0, n-1); g >= 1 gives the
// pair (2g-1, 2g).
template <int N, bool SYM, int G>
__device__ __forceinline__ void bt_two_rows(const Coefs& cf, const float2 (&in)[N], float2& oa, float2& ob) {
  constexpr int RA = (G == 0) ? 0 : 2 * G - 1;
  constexpr int RB = (G == 0) ? N - 1 : 2 * G;
  if constexpr (!SYM) {
    float2 a = mul2(cf.BT[RA][0], in[0]), b = mul2(cf.BT[RB][0], in[0]);
#pragma unroll
    for (int j = 1; j < N; ++j) {
      a = fma2(cf.BT[RA][j], in[j], a);
      b = fma2(cf.BT[RB][j], in[j], b);
    }
    oa = a; ob = b;
  } else if constexpr (G == 0) {
    float2 e = mul2(cf.BT[0][0], in[0]);
#pragma unroll
    for (int j = 2; j < N; j += 2) e = fma2(cf.BT[0][j], in[j], e);
    float2 o = mul2(cf.BT[N - 1][1], in[1]);
#pragma unroll
    for (int j = 3; j < N; j += 2) o = fma2(cf.BT[N - 1][j], in[j], o);
    oa = e; ob = o;
  } else {
    float2 e = mul2(cf.BT[RA][0], in[0]);
#pragma unroll
    for (int j = 2; j < N; j += 2) e = fma2(cf.BT[RA][j], in[j], e);
    float2 o = mul2(cf.BT[RA][1], in[1]);
#pragma unroll
    for (int j = 3; j < N - 1; j += 2) o = fma2(cf.BT[RA][j], in[j], o);
    oa = make_float2(e.x + o.x, e.y + o.y);
    ob = make_float2(e.x - o.x, e.y - o.y);
  }
}

// All n rows of B^T applied to one n-vector.
template <int N, bool SYM>
__device__ __forceinline__ void bt_all_rows(const Coefs& cf, const float2 (&in)[N], float2 (&out)[N]) {
  if constexpr (!SYM) {
#pragma unroll
    for (int p = 0; p < N; ++p) {
      float2 s = mul2(cf.BT[p][0], in[0]);
#pragma unroll
      for (int j = 1; j < N; ++j) s = fma2(cf.BT[p][j], in[j], s);
      out[p] = s;
    }
  } else {
    bt_two_rows<N, true, 0>(cf, in, out[0], out[N - 1]);
    if constexpr (N >= 4) bt_two_rows<N, true, 1>(cf, in, out[1], out[2]);
    if constexpr (N >= 6) bt_two_rows<N, true, 2>(cf, in, out[3], out[4]);
    if constexpr (N >= 8) bt_two_rows<N, true, 3>(cf, in, out[5], out[6]);
    if constexpr (N >= 10) bt_two_rows<N, true, 4>(cf, in, out[7], out[8]);
  }
}

// z[i] = sum_p A^T[i][p] * in[p], i < M.  N = M + r - 1 points: 0, (N - 2) / 2 pairs +-a, infinity.
template <int M, bool SYM, typename V, int N = M + 2>
__device__ __forceinline__ void at_apply(const Coefs& cf, const V (&in)[N], V (&z)[M]) {
  constexpr int NP = (N - 2) / 2;
  if constexpr (!SYM) {
#pragma unroll
    for (int i = 0; i < M; ++i) {
      V s = vmul(cf.AT[i][0], in[0]);
#pragma unroll
      for (int p = 1; p < N; ++p) s = vfma(cf.AT[i][p], in[p], s);
      z[i] = s;
    }
  } else {
    V sm[NP], df[NP];
#pragma unroll
    for (int q = 0; q < NP; ++q) {
      sm[q] = vadd(in[1 + 2 * q], in[2 + 2 * q]);
      df[q] = vsub(in[1 + 2 * q], in[2 + 2 * q]);
    }
#pragma unroll
    for (int i = 0; i < M; ++i) {
      V s = (i & 1) ? vmul(cf.AT[i][1], df[0]) : vmul(cf.AT[i][1], sm[0]);
#pragma unroll
      for (int q = 1; q < NP; ++q)
        s = (i & 1) ? vfma(cf.AT[i][1 + 2 * q], df[q], s) : vfma(cf.AT[i][1 + 2 * q], sm[q], s);
      if (i == 0) s = vadd(s, in[0]);
      if (i == M - 1) s = vadd(s, in[N - 1]);
      z[i] = s;
    }
  }
}

}  // namespace xf
}  // namespace nova
