// Y = A^T M A for one (tile, filter) whose n*n transformed-domain values sit in a shared-memory
// stage (Section 2.1 step 4, 2-D nested form of Appendix B.5), evaluated in float.
// A thread owns VEC consecutive filters of one tile.  VEC = 1: the stage holds 4 filter quads per
// frequency, frequency f = xi*n + nu is 512*f bytes in, and even and odd f differ in the swizzled
// 16-byte chunk (two per-lane bases).  VEC = 2: 8 quads per frequency, 1024*f bytes, one base;
// the arithmetic then runs on packed fp32 pairs (two IEEE results per instruction).  Every load is
// one ld.shared with an immediate offset; the row and pair indices are template parameters for
// that reason.
#pragma once
#include "sm100.cuh"
#include "transform_math.cuh"

namespace nova {
namespace xf {

__device__ __forceinline__ float vmax_lo(float v, float lo) { return v < lo ? lo : v; }
__device__ __forceinline__ float2 vmax_lo(float2 v, float lo) {
  return make_float2(v.x < lo ? lo : v.x, v.y < lo ? lo : v.y);
}

// int32 accumulator bits -> float (round to nearest even), times the dequantisation scale
// (__fmul_rn: the product is rounded on its own, never contracted into a following add)
__device__ __forceinline__ float dequant(float bits, float s) { return __fmul_rn(__int2float_rn(__float_as_int(bits)), s); }
__device__ __forceinline__ float2 dequant(float2 bits, float2 s) {
  return make_float2(__fmul_rn(__int2float_rn(__float_as_int(bits.x)), s.x), __fmul_rn(__int2float_rn(__float_as_int(bits.y)), s.y));
}

// Y[i][j] = sum_xi A^T[i][xi] * z_xi[j], where `rows.template row<XI>(z)` delivers z_xi[j] =
// sum_nu A^T[j][nu] * M[xi][nu] for its (tile, filters).  The row index is a template parameter so
// that whatever the provider loads is addressed by immediates.
template <int M, bool SYM, typename V, int N, typename Rows>
struct RowAccumulator {
  const Coefs& cf;
  const Rows& rows;
  // dense: Y[i][j] += A^T[i][xi] * z_xi[j] for every xi
  template <int XI>
  __device__ __forceinline__ void dense_from(V (&Y)[M][M]) const {
    if constexpr (XI < N) {
      V z[M];
      rows.template row<XI>(z);
#pragma unroll
      for (int i = 0; i < M; ++i)
#pragma unroll
        for (int j = 0; j < M; ++j) Y[i][j] = (XI == 0) ? vmul(cf.AT[i][0], z[j]) : vfma(cf.AT[i][XI], z[j], Y[i][j]);
      dense_from<XI + 1>(Y);
    }
  }
  // symmetric: rows +a / -a (Q, Q+1) share |coefficients|: even output rows take the sum of
  // the two row results, odd output rows the difference
  template <int Q>
  __device__ __forceinline__ void pairs_from(V (&Y)[M][M]) const {
    if constexpr (Q < N - 1) {
      V zp[M], zm[M];
      rows.template row<Q>(zp);
      rows.template row<Q + 1>(zm);
#pragma unroll
      for (int j = 0; j < M; ++j) {
        const V s = vadd(zp[j], zm[j]), d = vsub(zp[j], zm[j]);
#pragma unroll
        for (int i = 0; i < M; ++i)
          Y[i][j] = (Q == 1) ? vmul(cf.AT[i][1], (i & 1) ? d : s) : vfma(cf.AT[i][Q], (i & 1) ? d : s, Y[i][j]);
      }
      pairs_from<Q + 2>(Y);
    }
  }
  __device__ __forceinline__ void run(V (&Y)[M][M]) const {
    if constexpr (!SYM) {
      dense_from<0>(Y);
    } else {
      pairs_from<1>(Y);
      // A^T column 0 is e_0 and column n-1 is e_{m-1}
      V z0[M], zi[M];
      rows.template row<0>(z0);
      rows.template row<N - 1>(zi);
#pragma unroll
      for (int j = 0; j < M; ++j) {
        Y[0][j] = vadd(Y[0][j], z0[j]);
        Y[M - 1][j] = vadd(Y[M - 1][j], zi[j]);
      }
    }
  }
};
template <int M, bool SYM, typename V, int N, typename Rows>
__device__ __forceinline__ void accumulate_rows(const Coefs& cf, const Rows& rows, V (&Y)[M][M]) {
  RowAccumulator<M, SYM, V, N, Rows>{cf, rows}.run(Y);
}

// QUANT: the stage holds the int32 sums of the int8 pipeline; every value is converted to float
// and multiplied by qscale (this thread's filters' s_U[k] * s_V) as it is loaded.
template <int M, bool SYM, int VEC = 1, bool QUANT = false, int R = 3>
struct OutputTile {
  static constexpr int N = M + R - 1;
  using V = typename VecOf<VEC>::type;
  const Coefs& cf;
  uint32_t sb_even, sb_odd;      // VEC = 2 uses sb_even only
  V qscale;

  template <int XI, int NU>
  __device__ __forceinline__ void fill(V (&in)[N]) const {
    if constexpr (NU < N) {
      constexpr int F = XI * N + NU;
      if constexpr (VEC == 1)
        in[NU] = (F & 1) ? sm100::lds_f32<F * 512>(sb_odd) : sm100::lds_f32<F * 512>(sb_even);
      else
        in[NU] = sm100::lds_f32x2<F * 1024>(sb_even);
      if constexpr (QUANT) in[NU] = dequant(in[NU], qscale);
      fill<XI, NU + 1>(in);
    }
  }
  // z[j] = sum_nu A^T[j][nu] * M[xi][nu]
  template <int XI>
  __device__ __forceinline__ void row(V (&z)[M]) const {
    V in[N];
    fill<XI, 0>(in);
    at_apply<M, SYM, V, N>(cf, in, z);
  }
  __device__ __forceinline__ void run(V (&Y)[M][M]) const { accumulate_rows<M, SYM, V, N>(cf, *this, Y); }
};

// Streaming stores of y (written once, not read again by this library): evict-first in the caches,
// so that the lines of M the kernel has yet to read are not pushed out by its own output.
__device__ __forceinline__ void vstore_cs(__half* p, float v) {
  __stcs(reinterpret_cast<unsigned short*>(p), __half_as_ushort(__float2half_rn(v)));
}
__device__ __forceinline__ void vstore_cs(__half* p, float2 v) {
  const __half2 h = __floats2half2_rn(v.x, v.y);
  __stcs(reinterpret_cast<unsigned*>(p), *reinterpret_cast<const unsigned*>(&h));
}
__device__ __forceinline__ void vstore_cs(float* p, float v) { __stcs(p, v); }
__device__ __forceinline__ void vstore_cs(float* p, float2 v) { __stcs(reinterpret_cast<float2*>(p), v); }

// Round Y to the storage type and store the m x m outputs of one (tile, filter): pixel (i, j)
// goes to dst + (i * W + j) * K.  rows / cols = how many of the tile's rows / columns lie inside
// the image (m for an interior tile: no per-store predicate then).  ReLU keeps NaN and +inf.
template <int M, typename T, typename V>
__device__ __forceinline__ void store_tile(const V (&Y)[M][M], T* dst, size_t row_stride, int K, int rows,
                                           int cols, int relu) {
  const float lo = relu ? 0.f : -__int_as_float(0x7f800000);
  if (rows >= M && cols >= M) {
#pragma unroll
    for (int i = 0; i < M; ++i) {
      T* p = dst;
#pragma unroll
      for (int j = 0; j < M; ++j) {
        vstore_cs(p, vmax_lo(Y[i][j], lo));
        p += K;
      }
      dst += row_stride;
    }
  } else {
#pragma unroll
    for (int i = 0; i < M; ++i) {
      if (i < rows) {
        T* p = dst;
#pragma unroll
        for (int j = 0; j < M; ++j) {
          if (j < cols) vstore_cs(p, vmax_lo(Y[i][j], lo));
          p += K;
        }
      }
      dst += row_stride;
    }
  }
}

// max with NaN propagation (either operand NaN -> NaN; +0 > -0), as the pooling kernel's half max
__device__ __forceinline__ float max_nan_f32(float a, float b) {
  float r;
  asm("max.NaN.f32 %0, %1, %2;" : "=f"(r) : "f"(a), "f"(b));
  return r;
}
__device__ __forceinline__ float vmax_nan(float a, float b) { return max_nan_f32(a, b); }
__device__ __forceinline__ float2 vmax_nan(float2 a, float2 b) {
  return make_float2(max_nan_f32(a.x, b.x), max_nan_f32(a.y, b.y));
}

// The same for the 2 x 2 / 2 max-pooled output: the largest of each 2 x 2 window of the tile goes to
// dst + (pi * Wo + pj) * K, with dst, row_stride (= Wo * K), rows and cols those of the POOLED
// tensor (H and W are even and m is even, so a window never straddles tiles or the image edge).
// Max, ReLU and rounding are all monotone, so the result equals pooling the stored outputs.
template <int M, typename T, typename V>
__device__ __forceinline__ void store_tile_pooled(const V (&Y)[M][M], T* dst, size_t row_stride, int K, int rows,
                                                  int cols, int relu) {
  static_assert(M % 2 == 0, "pooling windows must not straddle tiles");
  const float lo = relu ? 0.f : -__int_as_float(0x7f800000);
#pragma unroll
  for (int pi = 0; pi < M / 2; ++pi) {
    if (pi < rows) {
      T* p = dst;
#pragma unroll
      for (int pj = 0; pj < M / 2; ++pj) {
        if (pj < cols)
          vstore_cs(p, vmax_lo(vmax_nan(vmax_nan(Y[2 * pi][2 * pj], Y[2 * pi][2 * pj + 1]),
                                        vmax_nan(Y[2 * pi + 1][2 * pj], Y[2 * pi + 1][2 * pj + 1])), lo));
        p += K;
      }
    }
    dst += row_stride;
  }
}

}  // namespace xf
}  // namespace nova
