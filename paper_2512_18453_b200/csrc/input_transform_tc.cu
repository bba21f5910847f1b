// Input-tile transform on the sm_100a tensor cores (Section 2.1 step 1 in its 2-D nested
// form, Appendix B.5): V = B^T d B written as one contraction over the n*n patch elements,
//   V[(xi,nu)][p][c] = sum_{(a,b)} (B^T (x) B^T)[(xi,nu)][(a,b)] * d_p[(a,b)][c],
// half x half -> float, rounded once to half.
//
// The n^2 x n^2 constant matrix is the Kronecker product of the plan's rounded B^T table
// with itself.  A product of two half values needs up to 22 significant bits, so the plan
// stores it as hi + lo (two half matrices, hi = fl16(prod), lo = fl16(prod - hi)) and the
// kernel issues the MMAs of both into the same accumulator: the result is the float
// accumulation of exact products of the rounded coefficients with the inputs, i.e. the
// same quantity the CUDA-core transform evaluates, in a different summation order.
//
// One work unit = two (tile, block of 64 channels) pairs, one per half of the 128 TMEM lanes; the
// pairs are numbered tile-major, so a unit is a tile's two neighbouring channel blocks when C is a
// multiple of 128 and two neighbouring tiles when C = 64 (no lane computes on zero fill).
// The units of a CTA are numbered i = 0, 1, ..; unit i uses ring stage
// i % kStages and TMEM accumulator i % kNumAcc.  Issuing a TMA box or a small MMA costs the
// issuing thread a few hundred cycles, so every role is spread over several warps:
//   warps 0-3   TMA producers, unit i by warp i%4: the n x n x 64-channel patch boxes of the
//               unit (two boxes, one per pair) straight from x [N,H,W,C]; rows/columns
//               outside the image and channels >= C are zero-filled by the TMA unit (the pad-1
//               halo and ragged tiles cost nothing).  A box lands as n*n rows of 128 bytes with
//               the 128-byte swizzle, which is the MN-major operand layout of tcgen05.mma
//               (M = channels).
//   warps 4-7   MMA issuers, unit i by warp 4 + i%4: D[128 channels][n^2 frequencies] (TMEM)
//               = patch (A, MN-major, from the ring) x Kronecker matrix (B, K-major, resident
//               in shared memory for the whole kernel).
//   warps 8-23  epilogue, four groups of four warps (one per TMEM lane quadrant), unit i by
//               group i%4: tcgen05.ld, convert to half, store V[f][p][c] (a lane is a channel:
//               64 contiguous bytes per warp store).
// Every wait is bounded; on expiry the kernel records a status and drains.
#include <cuda.h>
#include <cuda_fp16.h>
#include <cuda_runtime.h>

#include "nova_internal.h"
#include "sm100.cuh"
#include "tma_host.h"

namespace nova {
namespace {
using namespace sm100;

constexpr int kProdWarps = 4;
constexpr int kMmaWarps = 4;
constexpr int kEpiGroups = 4;
constexpr int kTcThreads = 32 * (kProdWarps + kMmaWarps + 4 * kEpiGroups);

template <int M, int R = 3>
struct TcCfg {
  static constexpr int N = M + R - 1;
  static constexpr int PAD = (R - 1) / 2;
  static constexpr int NF = N * N;                       // frequencies = patch elements
  static constexpr int KP = (NF + 15) / 16 * 16;         // contraction length, padded to the MMA K
  static constexpr int NFP = KP;                         // MMA N, padded to a multiple of 16
  static constexpr int KA = (KP + 63) / 64;              // 64-wide K atoms of the K-major operand
  static constexpr int kHalfBytes = KP * 128;            // one 64-channel half of a stage
  static constexpr int kStageBytes = 2 * kHalfBytes;
  static constexpr int kKronBytes = 2 * KA * NFP * 128;  // hi and lo
  static constexpr int kStages = (kStageBytes <= 16384) ? 8 : 4;
  static constexpr int kAccCols = (NFP <= 64) ? 64 : 128;   // TMEM columns per accumulator
  static constexpr int kNumAcc = 512 / kAccCols;            // 8 or 4 accumulators in flight
  static constexpr int kBarrierOffset = kKronBytes + kStages * kStageBytes;
  static constexpr int kTotal = kBarrierOffset + 512 + 1024;
};

// Ring discipline: an mbarrier wait names a phase only by its parity, so a warp that could
// get two phases ahead of a barrier would pass the wait early.  A warp is at most one phase
// ahead of a barrier it waited on for its own previous use of the same slot; therefore every
// slot (stage or accumulator) must always be handled by the same warp (group) of a role:
// the ring lengths are multiples of the number of warps (groups) that share the ring.
template <int M, int R = 3>
struct TcCfgCheck {
  static_assert(TcCfg<M, R>::kStages % kProdWarps == 0 && TcCfg<M, R>::kStages % kMmaWarps == 0, "stage ring");
  static_assert(TcCfg<M, R>::kNumAcc % kMmaWarps == 0 && TcCfg<M, R>::kNumAcc % kEpiGroups == 0, "accumulator ring");
  static constexpr bool ok = true;
};

template <int NR>
__device__ __forceinline__ void tmem_ld16(uint32_t taddr, uint32_t* r) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x16.b32 "
      "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15}, [%16];"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
        "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15])
      : "r"(taddr)
      : "memory");
}

// QMODE 0: V rounded to half.  QMODE 1: nothing is stored; the largest |V| is reduced into *qslot
// (as float bits; first pass of the int8 pipeline's data-derived scale).  QMODE 2: V / *qslot
// rounded to nearest even and saturated to signed 8 bit (the quantiser of the INT8 set-up,
// Section 5.1), as one float multiplication by the reciprocal scale per value.
template <int M, int QMODE, int R = 3>
__global__ void __launch_bounds__(kTcThreads, 1)
input_transform_tc_kernel(const __grid_constant__ CUtensorMap tmX, const __grid_constant__ CUtensorMap tmKron,
                          void* __restrict__ Vout, int C, int Th, int Tw, long long p0, int pc, int pc_pad,
                          int* __restrict__ status, float* __restrict__ qslot) {
  using Cfg = TcCfg<M, R>;
  static_assert(TcCfgCheck<M, R>::ok, "");
  constexpr int kStages = Cfg::kStages;
  constexpr int kNumAcc = Cfg::kNumAcc;
  constexpr int kAccCols = Cfg::kAccCols;
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
  uint8_t* kron = smem;
  uint8_t* ring = smem + Cfg::kKronBytes;
  uint64_t* full_bar = reinterpret_cast<uint64_t*>(smem + Cfg::kBarrierOffset);
  uint64_t* empty_bar = full_bar + kStages;
  uint64_t* tmem_full = empty_bar + kStages;         // [kNumAcc]
  uint64_t* tmem_empty = tmem_full + kNumAcc;        // [kNumAcc]
  uint64_t* kron_bar = tmem_empty + kNumAcc;
  uint32_t* tmem_base_slot = reinterpret_cast<uint32_t*>(kron_bar + 1);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_base_slot + 1);

  const int warp = threadIdx.x >> 5;
  const int lane = threadIdx.x & 31;
  // A unit is two (tile, 64-channel block) pairs, one per half of the 128 TMEM lanes; the pairs are
  // numbered tile-major, so a unit is one tile's two consecutive channel blocks when C is a multiple
  // of 128 and two consecutive tiles when C = 64.  Unit i of this CTA is unit blockIdx.x + i *
  // gridDim.x of the chunk: the chunk's tiles are transformed in ascending order chip-wide, so that
  // the rows of V written last - the ones still in L2 when the product kernel starts - are the
  // highest tiles.
  const unsigned CB64 = (unsigned)(C + 63) / 64;
  const unsigned num_sub = (unsigned)pc * CB64;
  const unsigned num_units = (num_sub + 1) / 2;
  const uint32_t n_local = num_units > blockIdx.x ? (num_units - blockIdx.x + gridDim.x - 1) / gridDim.x : 0u;

  if (threadIdx.x == 0) {
    for (int s = 0; s < kStages; ++s) { mbar_init(&full_bar[s], 1); mbar_init(&empty_bar[s], 1); }
    for (int a = 0; a < kNumAcc; ++a) { mbar_init(&tmem_full[a], 1); mbar_init(&tmem_empty[a], 4); }
    mbar_init(kron_bar, 1);
    *abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == kProdWarps) tmem_alloc(tmem_base_slot, 512);
  // Rows NF .. KP-1 of every stage half are never written by the TMA boxes; the matching
  // Kronecker columns are zero, so the rows only have to be finite: clear them once.
  if constexpr (Cfg::KP > Cfg::NF) {
    constexpr int pad16 = (Cfg::KP - Cfg::NF) * 8;   // 16-byte pieces per half
    for (int i = threadIdx.x; i < kStages * 2 * pad16; i += kTcThreads) {
      const int half = i / pad16, off = i % pad16;
      *reinterpret_cast<uint4*>(ring + (size_t)half * Cfg::kHalfBytes + Cfg::NF * 128 + off * 16) =
          make_uint4(0, 0, 0, 0);
    }
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_base_slot;
  bool timed_out = false;
  // the constant Kronecker table belongs to the plan: it may be fetched while the preceding
  // kernel of the stream is still draining; everything else waits for that kernel
  if (warp == 0 && lane == 0) {
    mbar_expect_tx(kron_bar, Cfg::kKronBytes);
    for (int b = 0; b < 2 * Cfg::KA; ++b)
      tma_load_2d(kron + (size_t)b * Cfg::NFP * 128, &tmKron, kron_bar, 0, b * Cfg::NFP);
  }
  pdl_launch_dependents();
  pdl_wait();

  if (warp < kProdWarps) {
    // ---------------- TMA producers
    for (uint32_t local = warp; local < n_local && !timed_out; local += kProdWarps) {
      const unsigned u = blockIdx.x + local * gridDim.x;
      const uint32_t stage = local % kStages, phase = (local / kStages) & 1;
      if (!mbar_wait_warp(&empty_bar[stage], phase ^ 1, abort_flag)) { timed_out = true; break; }
      if (lane == 0) {
        uint8_t* dst = ring + (size_t)stage * Cfg::kStageBytes;
        const int halves = 2 * u + 1 < num_sub ? 2 : 1;      // the last unit of an odd count has one half
        mbar_expect_tx(&full_bar[stage], halves * Cfg::NF * 128);
        for (int h = 0; h < halves; ++h) {
          const unsigned sidx = 2 * u + h;
          const int cb = (int)(sidx % CB64);
          const unsigned p = (unsigned)p0 + sidx / CB64;
          const int tw = (int)(p % (unsigned)Tw), th = (int)((p / (unsigned)Tw) % (unsigned)Th);
          const int img = (int)(p / ((unsigned)Tw * (unsigned)Th));
          tma_load_4d(dst + h * Cfg::kHalfBytes, &tmX, &full_bar[stage], cb * 64, M * tw - Cfg::PAD, M * th - Cfg::PAD, img);
        }
      }
      __syncwarp();
    }
  } else if (warp < kProdWarps + kMmaWarps) {
    // ---------------- MMA issuers
    constexpr uint32_t idesc = umma_idesc_f16_amn(128, Cfg::NFP);
    if (!mbar_wait_warp(kron_bar, 0, abort_flag)) timed_out = true;
    const uint64_t bd0 = umma_desc_sw128(smem_u32(kron));
    for (uint32_t local = warp - kProdWarps; local < n_local && !timed_out; local += kMmaWarps) {
      const uint32_t acc = local % kNumAcc, acc_phase = (local / kNumAcc) & 1;
      const uint32_t stage = local % kStages, phase = (local / kStages) & 1;
      if (!mbar_wait_warp(&tmem_empty[acc], acc_phase ^ 1, abort_flag)) { timed_out = true; break; }
      if (!mbar_wait_warp(&full_bar[stage], phase, abort_flag)) { timed_out = true; break; }
      tc_fence_after();
      if (lane == 0) {
        const uint32_t sa = smem_u32(ring + (size_t)stage * Cfg::kStageBytes);
        const uint32_t tmem_d = tmem_base + acc * kAccCols;
const uint64_t ad0 = umma_desc_mn_sw128(sa, Cfg::kHalfBytes);
#pragma unroll
        for (int hl = 0; hl < 2; ++hl)
#pragma unroll
          for (int ks = 0; ks < Cfg::KP / 16; ++ks) {
            const uint64_t ad = umma_desc_advance(ad0, ks * 2048);
            const uint64_t bd = umma_desc_advance(bd0, (hl * Cfg::KA + ks / 4) * Cfg::NFP * 128 + (ks % 4) * 32);
            if (hl == 0 && ks == 0) umma_f16_c<false>(tmem_d, ad, bd, idesc);
            else umma_f16_c<true>(tmem_d, ad, bd, idesc);
          }
        umma_commit(&empty_bar[stage]);
        umma_commit(&tmem_full[acc]);
      }
      __syncwarp();
    }
  } else {
    // ---------------- epilogue
    const int quad = warp & 3;                    // the TMEM lane quadrant this warp may read
    const int group = (warp - kProdWarps - kMmaWarps) >> 2;
    const size_t f_stride = (size_t)pc_pad * C;
    float qs = 1.f, amax = 0.f;
    if constexpr (QMODE == 2) {
      qs = *qslot;
      if (qs == 0.f) qs = 1.f;
      qs = __fdiv_rn(1.f, qs);                    // the quantiser multiplies by the reciprocal scale
    }
    for (uint32_t local = group; local < n_local && !timed_out; local += kEpiGroups) {
      const unsigned u = blockIdx.x + local * gridDim.x;
      const unsigned sidx = 2 * u + (quad >> 1);            // this lane quadrant's (tile, channel block) pair
      const int pl = (int)(sidx / CB64);
      const uint32_t acc = local % kNumAcc, acc_phase = (local / kNumAcc) & 1;
      // a pair past the end (odd count) has c >= C: nothing of it is stored or reduced
      const int c = sidx < num_sub ? (int)(sidx % CB64) * 64 + (quad & 1) * 32 + lane : C;
      if (!mbar_wait_warp(&tmem_full[acc], acc_phase, abort_flag)) { timed_out = true; break; }
      tc_fence_after();
      const uint32_t taddr = tmem_base + ((uint32_t)(quad * 32) << 16) + acc * kAccCols;
      __half* dst = reinterpret_cast<__half*>(Vout) + (size_t)pl * C + c;
      int8_t* dst8 = reinterpret_cast<int8_t*>(Vout) + (size_t)pl * C + c;
#pragma unroll
      for (int col0 = 0; col0 < Cfg::NFP; col0 += 64) {
        constexpr int kMaxCols = 64;
        uint32_t r[kMaxCols];
#pragma unroll
        for (int cc = 0; cc < kMaxCols; cc += 16)
          if (col0 + cc < Cfg::NFP) tmem_ld16<16>(taddr + col0 + cc, r + cc);
        tmem_ld_wait();
        if (col0 + 64 >= Cfg::NFP) {              // everything of this accumulator is in registers
          tc_fence_before();
          __syncwarp();
          if (lane == 0) mbar_arrive(&tmem_empty[acc]);
        }
        if constexpr (QMODE == 2) {
          // Four frequencies at a time: a lane packs its channel's four codes into a word, the
          // four lanes of a group transpose the 4 x 4 bytes with two shuffles, and lane i of the
          // group stores frequency i's four consecutive channels as one word (C % 16 == 0, so a
          // group of four channels is inside or outside the tensor as a whole).
          const int li = lane & 3;
          int8_t* d4 = dst8 - li + (size_t)li * f_stride;
#pragma unroll
          for (int cc = 0; cc < kMaxCols; cc += 4)
            if (col0 + cc < Cfg::NF) {
              uint32_t q[4];
#pragma unroll
              for (int j = 0; j < 4; ++j)
                asm("cvt.rni.sat.s8.f32 %0, %1;" : "=r"(q[j]) : "f"(__fmul_rn(__uint_as_float(r[cc + j]), qs)));
              // the low bytes of the four codes, packed with three byte permutations
              const uint32_t w = __byte_perm(__byte_perm(q[0], q[1], 0x0040), __byte_perm(q[2], q[3], 0x0040), 0x5410);
              const uint32_t p1 = __shfl_xor_sync(0xffffffffu, w, 1);
              const uint32_t t = __byte_perm(w, p1, (li & 1) ? 0x3715 : 0x6240);
              const uint32_t p2 = __shfl_xor_sync(0xffffffffu, t, 2);
              const uint32_t o = __byte_perm(t, p2, (li & 2) ? 0x3276 : 0x5410);
              if (c < C) *reinterpret_cast<uint32_t*>(d4) = o;
              d4 += 4 * f_stride;
            }
          dst8 += (size_t)((Cfg::NF - col0 < kMaxCols) ? (Cfg::NF - col0) : kMaxCols) * f_stride;
        } else if (c < C) {
#pragma unroll
          for (int cc = 0; cc < kMaxCols; ++cc)
            if (col0 + cc < Cfg::NF) {
              const float v = __uint_as_float(r[cc]);
              if constexpr (QMODE == 0) {
                *dst = __float2half_rn(v);
                dst += f_stride;
              } else {
                amax = fmaxf(amax, fabsf(v));
              }
            }
        }
      }
    }
    if constexpr (QMODE == 1) {                   // non-negative floats order like their bit patterns
      const unsigned mx = __reduce_max_sync(0xffffffffu, __float_as_uint(amax));
      if (lane == 0) atomicMax(reinterpret_cast<unsigned*>(qslot), mx);
    }
  }

  if (timed_out) {
    *abort_flag = 1;
    if (lane == 0) atomicExch(status, NOVA_ERR_DEVICE_TIMEOUT);
  }
  tc_fence_before();
  __syncthreads();
  if (warp == kProdWarps) {
    tc_fence_after();
    tmem_dealloc(tmem_base, 512);
  }
}

template <int M, int QMODE, int R = 3>
int launch_m(const nova_plan* plan, const Geom& g, const void* x, void* V, long long p0, int pc, int pc_pad,
             float* qslot, cudaStream_t stream) {
  using Cfg = TcCfg<M, R>;
  if (cudaError_t e = allow_dynamic_smem(input_transform_tc_kernel<M, QMODE, R>, Cfg::kTotal); e != cudaSuccess) return (int)e;
  EncodeTiledFn enc = tensor_map_encoder();
  if (!enc) return (int)cudaErrorUnknown;
  CUtensorMap tmX, tmK;
  {
    cuuint64_t dims[4] = {(cuuint64_t)g.C, (cuuint64_t)g.W, (cuuint64_t)g.H, (cuuint64_t)g.N};
    cuuint64_t strides[3] = {(cuuint64_t)g.C * 2, (cuuint64_t)g.W * g.C * 2, (cuuint64_t)g.H * g.W * g.C * 2};
    cuuint32_t box[4] = {64, (cuuint32_t)Cfg::N, (cuuint32_t)Cfg::N, 1};
    cuuint32_t estr[4] = {1, 1, 1, 1};
    if (enc(&tmX, CU_TENSOR_MAP_DATA_TYPE_FLOAT16, 4, const_cast<void*>(x), dims, strides, box, estr,
            CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
      return (int)cudaErrorUnknown;
  }
  {
    cuuint64_t dims[2] = {64, (cuuint64_t)(2 * Cfg::KA * Cfg::NFP)};
    cuuint64_t strides[1] = {128};
    cuuint32_t box[2] = {64, (cuuint32_t)Cfg::NFP};
    cuuint32_t estr[2] = {1, 1};
    if (enc(&tmK, CU_TENSOR_MAP_DATA_TYPE_FLOAT16, 2, plan->kron_dev, dims, strides, box, estr,
            CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
      return (int)cudaErrorUnknown;
  }
  const int sms = plan->sm_count;
  const long long units = ((long long)pc * ((g.C + 63) / 64) + 1) / 2;   // two (tile, 64-channel block) pairs each
  const int grid = (int)(units < sms ? units : sms);
  return (int)launch_overlapped(input_transform_tc_kernel<M, QMODE, R>, grid, kTcThreads, Cfg::kTotal, stream, tmX, tmK,
                                V, g.C, g.Th, g.Tw, p0, pc, pc_pad, plan->status_dev, qslot);
}

}  // namespace

size_t kron_table_halves(int n) {
  const int nf = n * n, kp = (nf + 15) / 16 * 16, ka = (kp + 63) / 64;
  return (size_t)2 * ka * kp * 64;
}

// Host image of the device table: [hi|lo][K atom][frequency row, padded][64 halves].
void build_kron_table(const nova_plan* plan, unsigned short* out) {
  const int n = plan->n, nf = n * n, kp = (nf + 15) / 16 * 16, ka = (kp + 63) / 64;
  for (size_t i = 0; i < kron_table_halves(plan->n); ++i) out[i] = 0;
  for (int xi = 0; xi < n; ++xi)
    for (int nu = 0; nu < n; ++nu)
      for (int a = 0; a < n; ++a)
        for (int b = 0; b < n; ++b) {
          const int f = xi * n + nu, k = a * n + b;
          const double prod = (double)plan->kcoefs.BT[xi][a] * (double)plan->kcoefs.BT[nu][b];
          const __half hi = __double2half(prod);
          const double hid = (double)__half2float(hi);
          __half lo = __float2half(0.f);
          if (hid - hid == 0.0) lo = __double2half(prod - hid);      // hi finite
          const size_t at = ((size_t)(k / 64) * kp + f) * 64 + (k % 64);
          out[at] = __half_as_ushort(hi);
          out[(size_t)ka * kp * 64 + at] = __half_as_ushort(lo);
        }
}

int launch_input_transform_tc(const nova_plan* plan, const Geom& g, const void* x, void* V, long long p0,
                              int pc, int pc_pad, void* stream) {
  cudaStream_t s = (cudaStream_t)stream;
  if (plan->r == 5) {                                 // 5 x 5 filters: n = m + 4 points, halo of 2
    switch (plan->m) {
      case 2: return launch_m<2, 0, 5>(plan, g, x, V, p0, pc, pc_pad, nullptr, s);
      case 4: return launch_m<4, 0, 5>(plan, g, x, V, p0, pc, pc_pad, nullptr, s);
      case 6: return launch_m<6, 0, 5>(plan, g, x, V, p0, pc, pc_pad, nullptr, s);
    }
    return (int)cudaErrorInvalidValue;
  }
  switch (plan->m) {
    case 2: return launch_m<2, 0>(plan, g, x, V, p0, pc, pc_pad, nullptr, s);
    case 4: return launch_m<4, 0>(plan, g, x, V, p0, pc, pc_pad, nullptr, s);
    case 6: return launch_m<6, 0>(plan, g, x, V, p0, pc, pc_pad, nullptr, s);
    case 8: return launch_m<8, 0>(plan, g, x, V, p0, pc, pc_pad, nullptr, s);
  }
  return (int)cudaErrorInvalidValue;
}

// int8 pipeline: pass 0 reduces max|V| into *slot (zeroed by the caller), pass 1 quantises with
// the scale at *slot into Vq [n*n][pc_pad][C] signed bytes.
int launch_input_transform_tc_int8(const nova_plan* plan, const Geom& g, const void* x, void* Vq, float* slot,
                                   int pass, long long p0, int pc, int pc_pad, void* stream) {
  cudaStream_t s = (cudaStream_t)stream;
#define NOVA_TC8(MM) \
  return pass == 0 ? launch_m<MM, 1>(plan, g, x, Vq, p0, pc, pc_pad, slot, s) \
                   : launch_m<MM, 2>(plan, g, x, Vq, p0, pc, pc_pad, slot, s)
  if (plan->r == 5) {
#define NOVA_TC8R5(MM) \
  return pass == 0 ? launch_m<MM, 1, 5>(plan, g, x, Vq, p0, pc, pc_pad, slot, s) \
                   : launch_m<MM, 2, 5>(plan, g, x, Vq, p0, pc, pc_pad, slot, s)
    switch (plan->m) {
      case 2: NOVA_TC8R5(2);
      case 4: NOVA_TC8R5(4);
      case 6: NOVA_TC8R5(6);
    }
#undef NOVA_TC8R5
    return (int)cudaErrorInvalidValue;
  }
  switch (plan->m) {
    case 2: NOVA_TC8(2);
    case 4: NOVA_TC8(4);
    case 6: NOVA_TC8(6);
    case 8: NOVA_TC8(8);
  }
#undef NOVA_TC8
  return (int)cudaErrorInvalidValue;
}

}  // namespace nova
