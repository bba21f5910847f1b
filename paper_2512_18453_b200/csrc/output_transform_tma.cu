// Output transform Y = A^T M A (Section 2.1 step 4 in its 2-D nested form, Appendix B.5),
// evaluated in float and rounded once to the storage type, with the transformed-domain
// product M staged through shared memory by TMA.
//
// M is stored [n*n][K/4][pc_pad][4] floats (frequency, filter quad, tile, filter in quad).
// One work unit = 8 consecutive tiles x 16 consecutive filters, all n*n frequencies: one TMA
// box of n*n*4 rows of 128 bytes (128-byte swizzle).
//   warp 0      TMA producer, one box per unit into a ring of stages.
//   warps 1-12  three consumer groups of four warps, unit i by group i%3.  Warp w of a group
//               owns tiles w and w+4 of the unit, a lane one (tile, filter): its n*n values sit
//               in conflict-free banks (the swizzle separates tiles w and w+4), and a warp's
//               store of one output pixel covers 16 consecutive filters (32 bytes) of two tiles.
// The arithmetic is transform_math.cuh's (dense, or the shared even/odd sums of a symmetric
// point set).  Every wait is bounded; on expiry the kernel records a status and drains.
#include <cuda.h>
#include <cuda_fp16.h>
#include <cuda_runtime.h>

#include "nova_internal.h"
#include "sm100.cuh"
#include "tma_host.h"
#include "output_math.cuh"
#include "transform_math.cuh"

namespace nova {
namespace {
using namespace sm100;
using namespace xf;

constexpr int kConsGroups = 3;
constexpr int kOtThreads = 32 * (1 + 4 * kConsGroups);

template <int M, int VEC, int R = 3>
struct OtCfg {
  static constexpr int N = M + R - 1;
  static constexpr int NF = N * N;
  static constexpr int kQuads = 4 * VEC;              // filter quads per unit: 16 * VEC filters
  static constexpr int kStageBytes = NF * kQuads * 128;   // NF * kQuads rows of 128 bytes; a multiple of 1024
  // a multiple of the number of consumer groups: a stage is always read by the same group, so
  // no warp can get two phases ahead of a barrier it waits on by parity
  static constexpr int kStages = ((200 * 1024 / kStageBytes) >= 6 ? 6 : 3);
  static_assert(kStages % kConsGroups == 0, "stage ring");
  static constexpr int kBarrierOffset = kStages * kStageBytes;
  static constexpr int kTotal = kBarrierOffset + 256 + 1024;
};

// QUANT: M holds the int32 sums of the int8 pipeline; scale_U[k] * *scale_V dequantises filter k.
// relu: bit 0 = ReLU, bit 1 = the 2 x 2 max-pooled store (y is then [N, H/2, W/2, K]).
template <int M, typename T, bool SYM, int VEC, bool QUANT, int R = 3>
__global__ void __launch_bounds__(kOtThreads, 1)
output_transform_tma_kernel(const __grid_constant__ CUtensorMap tmM, const __grid_constant__ Coefs cf,
                            T* __restrict__ y, int H, int W, int K, int Th, int Tw, long long p0, int pc,
                            int pc_pad, int relu, int* __restrict__ status, const float* __restrict__ scale_U,
                            const float* __restrict__ scale_V, const float* __restrict__ Mbase) {
  using Cfg = OtCfg<M, VEC, R>;
  constexpr int kStages = Cfg::kStages;
  constexpr int kUnitK = 16 * VEC;                    // filters per unit
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
  uint64_t* full_bar = reinterpret_cast<uint64_t*>(smem + Cfg::kBarrierOffset);
  uint64_t* empty_bar = full_bar + kStages;
  volatile int* abort_flag = reinterpret_cast<volatile int*>(empty_bar + kStages);

  const int warp = threadIdx.x >> 5;
  const int lane = threadIdx.x & 31;
  const int KG = (K + kUnitK - 1) / kUnitK;           // filter groups of 16 * VEC
  const int TG = pc_pad >> 3;                         // tile groups of 8 (pc_pad is a multiple of 128)
  // Unit i of this CTA is unit blockIdx.x + i * gridDim.x: ascending tiles chip-wide, i.e. the
  // rows of M the product kernel wrote last (still in L2) first.
  const unsigned num_units = (unsigned)TG * (unsigned)KG;
  const uint32_t n_local = num_units > blockIdx.x ? (num_units - blockIdx.x + gridDim.x - 1) / gridDim.x : 0u;

  if (threadIdx.x == 0) {
    for (int s = 0; s < kStages; ++s) { mbar_init(&full_bar[s], 1); mbar_init(&empty_bar[s], 4); }
    *abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  __syncthreads();
  bool timed_out = false;
  pdl_launch_dependents();       // the set-up above may overlap the tail of the preceding kernel
  pdl_wait();

  if (warp == 0) {
    // ---------------- TMA producer
    for (uint32_t local = 0; local < n_local && !timed_out; ++local) {
      const unsigned u = blockIdx.x + local * gridDim.x;
      const int kg = (int)(u % (unsigned)KG), tg = (int)(u / (unsigned)KG);
      const uint32_t stage = local % kStages, phase = (local / kStages) & 1;
      if (!mbar_wait_warp(&empty_bar[stage], phase ^ 1, abort_flag)) { timed_out = true; break; }
      if (lane == 0) {
        mbar_expect_tx(&full_bar[stage], Cfg::kStageBytes);
        tma_load_3d(smem + (size_t)stage * Cfg::kStageBytes, &tmM, &full_bar[stage], tg * 32, kg * Cfg::kQuads, 0);
      }
      __syncwarp();
    }
  } else {
    // ---------------- consumers
    const int group = (warp - 1) >> 2;
    const int w = (warp - 1) & 3;
    const int t = w + 4 * (lane >> 4);                // tile within the unit's 8
    // filter quad within the unit, filter (pair) in the quad, and the byte offsets of this lane's
    // value(s) inside a frequency's rows (128B swizzle: the 16-byte chunk index is XORed with the
    // row index modulo 8; with 4 rows per frequency even and odd frequencies differ)
    const int kq = (VEC == 1) ? (lane & 15) >> 2 : (lane & 15) >> 1;
    const int kk = (VEC == 1) ? (lane & 3) : (lane & 1) * 2;
    const uint32_t off_even = kq * 128 + ((t ^ kq) << 4) + kk * 4;
    const uint32_t off_odd = kq * 128 + ((t ^ ((kq + 4) & 7)) << 4) + kk * 4;
    for (uint32_t local = group; local < n_local && !timed_out; local += kConsGroups) {
      const unsigned u = blockIdx.x + local * gridDim.x;
      const int kg = (int)(u % (unsigned)KG), tg = (int)(u / (unsigned)KG);
      const uint32_t stage = local % kStages, phase = (local / kStages) & 1;
      if (!mbar_wait_warp(&full_bar[stage], phase, abort_flag)) { timed_out = true; break; }
      const uint32_t sb = smem_u32(smem) + stage * Cfg::kStageBytes;
      const uint32_t sb_even = sb + off_even, sb_odd = sb + off_odd;
      typename VecOf<VEC>::type Y[M][M];
      const int k = kg * kUnitK + (lane & 15) * VEC;
      typename VecOf<VEC>::type qs = {};
      if constexpr (QUANT) {
        const float sv = *scale_V;
        if constexpr (VEC == 1) qs = __fmul_rn(k < K ? scale_U[k] : 0.f, sv);
        else qs = make_float2(__fmul_rn(k < K ? scale_U[k] : 0.f, sv), __fmul_rn(k + 1 < K ? scale_U[k + 1] : 0.f, sv));
      }
      OutputTile<M, SYM, VEC, QUANT, R>{cf, sb_even, sb_odd, qs}.run(Y);
      __syncwarp();
      if (lane == 0) mbar_arrive(&empty_bar[stage]);
      // This unit was the only reader of its box of M (scratch): drop the lines from the L2 so
      // that the ones still dirty there are never written back to device memory.
      {
        const int k4 = K >> 2;
        for (int i = w * 32 + lane; i < Cfg::NF * Cfg::kQuads; i += 128) {
          const int f = i / Cfg::kQuads, kq_abs = kg * Cfg::kQuads + i % Cfg::kQuads;
          if (kq_abs < k4) l2_discard_line(Mbase + (((size_t)f * k4 + kq_abs) * pc_pad + (size_t)tg * 8) * 4);
        }
      }

      const int pl = tg * 8 + t;
      if (pl < pc && k < K) {
        const unsigned p = (unsigned)(p0 + pl);
        const unsigned tw = p % (unsigned)Tw, q2 = p / (unsigned)Tw;
        const unsigned th = q2 % (unsigned)Th, img = q2 / (unsigned)Th;
        const int h0 = M * (int)th, w0 = M * (int)tw;
        if (relu & 2) {              // 2 x 2 / 2 max-pool before the store: y is [N, H/2, W/2, K]
          const int Ho = H >> 1, Wo = W >> 1, ho = h0 >> 1, wo = w0 >> 1;
          T* dst = y + (((size_t)img * Ho + ho) * Wo + wo) * K + k;
          store_tile_pooled<M, T>(Y, dst, (size_t)Wo * K, K, Ho - ho, Wo - wo, relu & 1);
        } else {
          T* dst = y + (((size_t)img * H + h0) * W + w0) * K + k;
          store_tile<M, T>(Y, dst, (size_t)W * K, K, H - h0, W - w0, relu & 1);
        }
      }
    }
  }

  if (timed_out) {
    *abort_flag = 1;
    if (lane == 0) atomicExch(status, NOVA_ERR_DEVICE_TIMEOUT);
  }
}

template <int M, typename T, bool SYM, int VEC, bool QUANT, int R = 3>
int launch_one(const nova_plan* plan, const Geom& g, const CUtensorMap& tmM, const float* Mb, void* y, long long p0, int pc,
               int pc_pad, int relu, const float* scale_U, const float* scale_V, cudaStream_t stream) {
  using Cfg = OtCfg<M, VEC, R>;
  if (cudaError_t e = allow_dynamic_smem(output_transform_tma_kernel<M, T, SYM, VEC, QUANT, R>, Cfg::kTotal); e != cudaSuccess) return (int)e;
  const long long units = (long long)(pc_pad / 8) * ((g.K + 16 * VEC - 1) / (16 * VEC));
  const int grid = (int)(units < plan->sm_count ? units : plan->sm_count);
  return (int)launch_overlapped(output_transform_tma_kernel<M, T, SYM, VEC, QUANT, R>, grid, kOtThreads, Cfg::kTotal,
                                stream, tmM, plan->kcoefs, (T*)y, g.H, g.W, g.K, g.Th, g.Tw, p0, pc, pc_pad, relu,
                                plan->status_dev, scale_U, scale_V, Mb);
}

template <int M, int R = 3>
int launch_m(const nova_plan* plan, const Geom& g, const void* Mb, void* y, long long p0, int pc, int pc_pad,
             int relu, const float* scale_U, const float* scale_V, cudaStream_t stream) {
  EncodeTiledFn enc = tensor_map_encoder();
  if (!enc) return (int)cudaErrorUnknown;
  CUtensorMap tmM;
  const int k4 = g.K / 4;
  cuuint64_t dims[3] = {(cuuint64_t)pc_pad * 4, (cuuint64_t)k4, (cuuint64_t)(g.n * g.n)};
  cuuint64_t strides[2] = {(cuuint64_t)pc_pad * 16, (cuuint64_t)k4 * pc_pad * 16};
  constexpr int VEC = (M + R - 1 <= 8) ? 2 : 1;       // packed fp32 pairs where the registers allow
  cuuint32_t box[3] = {32, 4 * VEC, (cuuint32_t)(g.n * g.n)};
  cuuint32_t estr[3] = {1, 1, 1};
  if (enc(&tmM, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 3, const_cast<void*>(Mb), dims, strides, box, estr,
          CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_NONE,
          CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
    return (int)cudaErrorUnknown;
  if (plan->mode == NOVA_FP32) return (int)cudaErrorInvalidValue;   // the fp32 mode has its own transforms
#define NOVA_OT(TT, SYMV, Q) launch_one<M, TT, SYMV, VEC, Q, R>(plan, g, tmM, (const float*)Mb, y, p0, pc, pc_pad, relu, scale_U, scale_V, stream)
  if (scale_U)                                        // int8 pipeline: M holds int32 sums
    return plan->symmetric ? NOVA_OT(__half, true, true) : NOVA_OT(__half, false, true);
  return plan->symmetric ? NOVA_OT(__half, true, false) : NOVA_OT(__half, false, false);
#undef NOVA_OT
}

}  // namespace

int launch_output_transform_tma(const nova_plan* plan, const Geom& g, const void* Mb, void* y, long long p0,
                                int pc, int pc_pad, int relu, void* stream, const float* scale_U,
                                const float* scale_V) {
  cudaStream_t s = (cudaStream_t)stream;
  if (plan->r == 5) {
    switch (plan->m) {
      case 2: return launch_m<2, 5>(plan, g, Mb, y, p0, pc, pc_pad, relu, scale_U, scale_V, s);
      case 4: return launch_m<4, 5>(plan, g, Mb, y, p0, pc, pc_pad, relu, scale_U, scale_V, s);
      case 6: return launch_m<6, 5>(plan, g, Mb, y, p0, pc, pc_pad, relu, scale_U, scale_V, s);
    }
    return (int)cudaErrorInvalidValue;
  }
  switch (plan->m) {
    case 2: return launch_m<2>(plan, g, Mb, y, p0, pc, pc_pad, relu, scale_U, scale_V, s);
    case 4: return launch_m<4>(plan, g, Mb, y, p0, pc, pc_pad, relu, scale_U, scale_V, s);
    case 6: return launch_m<6>(plan, g, Mb, y, p0, pc, pc_pad, relu, scale_U, scale_V, s);
    case 8: return launch_m<8>(plan, g, Mb, y, p0, pc, pc_pad, relu, scale_U, scale_V, s);
  }
  return (int)cudaErrorInvalidValue;
}

}  // namespace nova
