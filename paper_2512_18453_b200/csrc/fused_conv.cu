// The whole forward convolution (Section 2.1 steps 1, 3, 4 in their 2-D nested form,
// Appendix B.5) as ONE persistent kernel whose CTAs are specialised by role and exchange
// work through rings of transformed tiles that stay in the L2 cache:
//
//   role I  (nI CTAs)      input transform on the tensor cores, x -> V ring   (see input_transform_tc.cu)
//   role G  (the others)   transformed-domain product, V ring x U -> M ring    (see gemm_tcgen05.cu)
//   role O  (every CTA)    output transform, M ring -> y                       (see output_transform_tma.cu)
// Every CTA runs role O on its last nine warps next to role I or role G on the first ones:
// G is bound by the SM's store bandwidth (its epilogue writes 128 KB of M per item while the
// tensor pipe and the issue slots idle), I mostly by latencies, O by instruction issue, so O
// fills the issue slots of every SM while the stores of V and M spread over the chip.
//
// The tiles are grouped in blocks of 128; the rings hold R blocks (row = tile mod 128 R).
// Three counters per block order the roles:
//   v_ready[b]  += 1 by every epilogue warp of role I after its stores of a unit of block b
//   g_done[b]   += 1 by every epilogue warp of role G after its stores of an item of block b
//   o_done[b]   += 1 by every consumer warp of role O after it has read a unit of block b
// and the TMA producer of a role waits, before it loads anything of block b, for
//   role I: g_done[b-R] complete (the V rows are free again);
//   role G: v_ready[b] complete and o_done[b-R] complete (the M rows are free again);
//   role O: g_done[b] complete.
// Every wait names a block that precedes b in each role's own order, every CTA walks its
// role's work in increasing block order (work item = rank + j * role size), and all CTAs are
// co-resident (cooperative launch, one CTA per SM), so the oldest unfinished block can always
// make progress.  All waits are bounded; one that expires sets a flag every CTA polls.
#include <cuda.h>
#include <cuda_fp16.h>
#include <cuda_runtime.h>

#include "nova_internal.h"
#include "sm100.cuh"
#include "output_math.cuh"
#include "transform_math.cuh"

namespace nova {
namespace {
using namespace sm100;
using namespace xf;

constexpr int kFusedThreads = 512;     // 16 warps x 128 registers: 11 of role I or G, then 5 of role O
constexpr int kGWarps = 11;
constexpr int kOWarpBase = 11;
constexpr int BLOCK_M = 128;
constexpr int BLOCK_K = 64;
constexpr uint32_t kCtrSpinLimit = 1u << 20;

struct RingParams {
  uint32_t* v_ready;     // [NB]
  uint32_t* g_done;      // [NB]
  uint32_t* o_done;      // [NB]
  int* abort_all;        // set by any CTA that gives up
  int R;                 // ring length of M in 128-tile blocks
  int RV;                // ring length of V (all blocks when V was produced by an earlier kernel: nI == 0)
  int P;                 // tiles
  int nI, nGO;           // CTAs of role I; the others run roles G and O together
  uint32_t g_target;     // g_done value of a finished block: n^2 * (filter blocks) * 4
};

struct ConvShape {
  int H, W, C, K, Th, Tw, relu;
};

// ---------------------------------------------------------------- counters
__device__ __forceinline__ bool ctr_wait(const uint32_t* ctr, uint32_t target, volatile int* abort_flag,
                                         const int* abort_all) {
  const uint64_t t0 = global_ns();
  for (uint32_t i = 0; i < kCtrSpinLimit; ++i) {
    uint32_t v;
    asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(ctr) : "memory");
    if (v >= target) return true;
    if ((i & 31u) == 31u && (*abort_flag || *reinterpret_cast<const volatile int*>(abort_all) ||
                             global_ns() - t0 > kWaitLimitNs))
      return false;
    __nanosleep(64);
  }
  return false;
}
__device__ __forceinline__ bool ctr_wait_warp(const uint32_t* ctr, uint32_t target, volatile int* abort_flag,
                                              const int* abort_all) {
  uint32_t ok = 1;
  if ((threadIdx.x & 31) == 0) ok = ctr_wait(ctr, target, abort_flag, abort_all) ? 1u : 0u;
  return __shfl_sync(0xffffffffu, ok, 0) != 0;
}
// A counter check whose load was issued one work item ahead (the load is asynchronous until its
// value is used), so that a dependency that is already satisfied costs no round trip to L2 on
// the producer's critical path.  Lane 0 holds the state; gate() returns the verdict to all lanes.
struct CtrGate {
  uint32_t val;
  int block;      // block the prefetched value belongs to (-1: none)
  __device__ __forceinline__ void prefetch(const uint32_t* ctrs, int b) {
    if ((threadIdx.x & 31) == 0) {
      block = b;
      val = 0;
      if (b >= 0) asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(val) : "l"(ctrs + b) : "memory");
    }
  }
  __device__ __forceinline__ bool gate(const uint32_t* ctrs, int b, uint32_t target, volatile int* abort_flag,
                                       const int* abort_all) {
    uint32_t ok = 1;
    if ((threadIdx.x & 31) == 0) {
      ok = (block == b && val >= target) ? 1u : 0u;
      if (!ok) ok = ctr_wait(ctrs + b, target, abort_flag, abort_all) ? 1u : 0u;
    }
    return __shfl_sync(0xffffffffu, ok, 0) != 0;
  }
};

// Called by all lanes of a warp after their global stores (or shared-memory reads) of a unit.
__device__ __forceinline__ void ctr_signal(uint32_t* ctr) {
  __syncwarp();
  if ((threadIdx.x & 31) == 0) {
    __threadfence();
    asm volatile("fence.proxy.async.global;" ::: "memory");
    asm volatile("red.release.gpu.global.add.u32 [%0], 1;" ::"l"(ctr) : "memory");
  }
}
// The same for n units at once.
__device__ __forceinline__ void ctr_signal_n(uint32_t* ctr, uint32_t n) {
  __syncwarp();
  if ((threadIdx.x & 31) == 0) {
    __threadfence();
    asm volatile("fence.proxy.async.global;" ::: "memory");
    asm volatile("red.release.gpu.global.add.u32 [%0], %1;" ::"l"(ctr), "r"(n) : "memory");
  }
}
// "These rows have been read": raised after the data has landed in shared memory (the full
// barrier was observed) and been loaded into registers, so no fence is needed - and none is
// wanted: a fence would wait for the warp's own earlier y stores.
__device__ __forceinline__ void ctr_signal_read(uint32_t* ctr) {
  __syncwarp();
  if ((threadIdx.x & 31) == 0) asm volatile("red.relaxed.gpu.global.add.u32 [%0], 1;" ::"l"(ctr) : "memory");
}
__device__ __forceinline__ void async_proxy_acquire() {
  asm volatile("fence.proxy.async.global;" ::: "memory");
}

__device__ __forceinline__ void tmem_ld16(uint32_t taddr, uint32_t* r) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x16.b32 "
      "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15}, [%16];"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
        "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15])
      : "r"(taddr)
      : "memory");
}
__device__ __forceinline__ void tmem_ld32(uint32_t taddr, uint32_t (&r)[32]) {
  tmem_ld16(taddr, r);
  tmem_ld16(taddr + 16, r + 16);
}

// ---------------------------------------------------------------- configuration
template <int M>
struct ICfg {
  static constexpr int N = M + 2;
  static constexpr int NF = N * N;
  static constexpr int KP = (NF + 15) / 16 * 16;
  static constexpr int NFP = KP;
  static constexpr int KA = (KP + 63) / 64;
  static constexpr int kHalfBytes = KP * 128;
  static constexpr int kStageBytes = 2 * kHalfBytes;
  static constexpr int kKronBytes = 2 * KA * NFP * 128;
  static constexpr int kStages = (kStageBytes <= 16384) ? 4 : 2;
  static constexpr int kAccCols = (NFP <= 64) ? 64 : 128;
  static constexpr int kNumAcc = 512 / kAccCols;
  static constexpr int kProd = 1, kMma = 2, kEpi = 2;       // producer warps, issuer warps, epilogue groups
  // epilogue staging: per group two buffers of [NF frequencies][128 channels] halves
  static constexpr int kOutBufBytes = NF * 256;
  static constexpr int kOutOffset = kKronBytes + kStages * kStageBytes;
  static constexpr int kBytes = kOutOffset + kEpi * 2 * kOutBufBytes;
  // a slot of a ring is always handled by the same warp (group): see the note in input_transform_tc.cu
  static_assert(kStages % kProd == 0 && kStages % kMma == 0 && kNumAcc % kMma == 0 && kNumAcc % kEpi == 0, "rings");
};
template <int M>
struct OCfg {
  static constexpr int N = M + 2;
  static constexpr int NF = N * N;
  static constexpr int VEC = (M <= 6) ? 2 : 1;        // filters per thread: packed fp32 pairs where the registers allow
  static constexpr int kQuads = 4 * VEC;              // filter quads per unit (16 * VEC filters, 8 tiles)
  static constexpr int kStageBytes = NF * kQuads * 128;
  static constexpr int kGroups = 1;                   // one consumer group of four warps
  static constexpr int kStages = 2;
  static constexpr int kBytes = kStages * kStageBytes;
  static_assert(kStages % kGroups == 0, "stage ring");
};
template <int M, int BLOCK_N>
struct GCfg {
  static constexpr int kABytes = BLOCK_M * BLOCK_K * 2;
  static constexpr int kBBytes = BLOCK_N * BLOCK_K * 2;
  static constexpr int kStageBytes = kABytes + kBBytes;
  static constexpr int kStages = 2;                   // what role O leaves of the SM's shared memory
  static constexpr int kBytes = kStages * kStageBytes;
};
constexpr int cmax(int a, int b) { return a > b ? a : b; }
template <int M, int BLOCK_N>
struct FusedCfg {
  // role O's ring sits behind role I's or role G's data, whichever the CTA runs; where both
  // do not fit next to role I (F(8,3)), the role-I CTAs run without role O
  static constexpr bool kOWithI = ICfg<M>::kBytes + OCfg<M>::kBytes <= 220 * 1024;
  static constexpr int kOOffset = kOWithI ? cmax(ICfg<M>::kBytes, GCfg<M, BLOCK_N>::kBytes) : GCfg<M, BLOCK_N>::kBytes;
  static constexpr int kDataBytes = cmax(ICfg<M>::kBytes, kOOffset + OCfg<M>::kBytes);
  static constexpr int kBarrierOffset = kDataBytes;
  static constexpr int kTotal = kBarrierOffset + 512 + 1024;
};

// ---------------------------------------------------------------- role I
// Epilogue pieces with compile-time shared-memory offsets (one instruction per access).
template <int CC, int COL0, int NF>
__device__ __forceinline__ void sts_cols(uint32_t mine, const uint32_t* r) {
  if constexpr (CC < 64) {
    if constexpr (COL0 + CC < NF) {
      sts_b16<(COL0 + CC) * 256>(mine, __half_as_ushort(__float2half_rn(__uint_as_float(r[CC]))));
      sts_cols<CC + 1, COL0, NF>(mine, r);
    }
  }
}
// 64 accumulator columns starting at COL0: TMEM -> registers -> half -> column of the staging tile
template <class Cfg, int COL0>
__device__ __forceinline__ void epi_pass(uint32_t taddr, uint32_t mine) {
  uint32_t r[64];
#pragma unroll
  for (int cc = 0; cc < 64; cc += 16)
    if (COL0 + cc < Cfg::NFP) tmem_ld16(taddr + COL0 + cc, r + cc);
  tmem_ld_wait();
  sts_cols<0, COL0, Cfg::NF>(mine, r);
}
// rows f0, f0+8, f0+16, .. of the staging tile: one 16-byte piece each, to global rows 8 planes apart
template <class Cfg, int J>
__device__ __forceinline__ void copy_out(uint32_t src, __half* dst, size_t stride8, int f0) {
  if constexpr (J < (Cfg::NF + 7) / 8) {
    if (f0 + 8 * J < Cfg::NF) *reinterpret_cast<uint4*>(dst) = lds_v4<J * 8 * 256>(src);
    copy_out<Cfg, J + 1>(src, dst + stride8, stride8, f0);
  }
}

// All threads of the CTA, before the CTA-wide barrier: role I's barriers and the pad rows of its ring.
template <int M>
__device__ __forceinline__ void input_prologue(uint8_t* smem, uint64_t* bars) {
  using Cfg = ICfg<M>;
  constexpr int kStages = Cfg::kStages, kNumAcc = Cfg::kNumAcc;
  uint8_t* ring = smem + Cfg::kKronBytes;
  if (threadIdx.x == 0) {
    uint64_t* full_bar = bars;
    uint64_t* empty_bar = full_bar + kStages;
    uint64_t* tmem_full = empty_bar + kStages;
    uint64_t* tmem_empty = tmem_full + kNumAcc;
    uint64_t* kron_bar = tmem_empty + kNumAcc;
    for (int s = 0; s < kStages; ++s) { mbar_init(&full_bar[s], 1); mbar_init(&empty_bar[s], 1); }
    for (int a = 0; a < kNumAcc; ++a) { mbar_init(&tmem_full[a], 1); mbar_init(&tmem_empty[a], 4); }
    mbar_init(kron_bar, 1);
  }
  if constexpr (Cfg::KP > Cfg::NF) {
    constexpr int pad16 = (Cfg::KP - Cfg::NF) * 8;
    for (int i = threadIdx.x; i < kStages * 2 * pad16; i += kFusedThreads) {
      const int half = i / pad16, off = i % pad16;
      *reinterpret_cast<uint4*>(ring + (size_t)half * Cfg::kHalfBytes + Cfg::NF * 128 + off * 16) =
          make_uint4(0, 0, 0, 0);
    }
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  }
}
constexpr int kIBarriers = 40;      // barrier slots reserved for role I or G; role O's follow
// Warps 0 .. 10 of the CTA; barriers and TMEM are set up by the caller.
template <int M>
__device__ __forceinline__ void role_input(uint8_t* smem, uint64_t* bars, uint32_t tmem_base,
                                           volatile int* abort_flag, const CUtensorMap* tmX,
                                           const CUtensorMap* tmKron, __half* __restrict__ V,
                                           const ConvShape& cs, const RingParams& rp, int rank, bool& timed_out) {
  using Cfg = ICfg<M>;
  constexpr int kStages = Cfg::kStages, kNumAcc = Cfg::kNumAcc, kAccCols = Cfg::kAccCols;
  uint8_t* kron = smem;
  uint8_t* ring = smem + Cfg::kKronBytes;
  uint64_t* full_bar = bars;
  uint64_t* empty_bar = full_bar + kStages;
  uint64_t* tmem_full = empty_bar + kStages;
  uint64_t* tmem_empty = tmem_full + kNumAcc;
  uint64_t* kron_bar = tmem_empty + kNumAcc;

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int C = cs.C;
  const unsigned CB = (unsigned)((C + 127) / 128);
  const unsigned num_units = (unsigned)rp.P * CB;
  const unsigned n_local = (num_units > (unsigned)rank) ? (num_units - rank + rp.nI - 1) / rp.nI : 0u;
  const int RP = rp.RV * 128;
  const uint32_t g_target = rp.g_target;

  if (warp < Cfg::kProd) {
    if (warp == 0 && lane == 0) {
      mbar_expect_tx(kron_bar, Cfg::kKronBytes);
      for (int b = 0; b < 2 * Cfg::KA; ++b)
        tma_load_2d(kron + (size_t)b * Cfg::NFP * 128, tmKron, kron_bar, 0, b * Cfg::NFP);
    }
    for (unsigned local = warp; local < n_local && !timed_out; local += Cfg::kProd) {
      const unsigned u = rank + local * rp.nI;
      const unsigned p = u / CB, cblk = u % CB;
      const unsigned tw = p % (unsigned)cs.Tw, q2 = p / (unsigned)cs.Tw;
      const unsigned th = q2 % (unsigned)cs.Th, img = q2 / (unsigned)cs.Th;
      const int b = (int)(p >> 7);
      if (b >= rp.RV && !ctr_wait_warp(rp.g_done + (b - rp.RV), g_target, abort_flag, rp.abort_all)) {
        timed_out = true; break;
      }
      const uint32_t stage = local % kStages, phase = (local / kStages) & 1;
      if (!mbar_wait_warp(&empty_bar[stage], phase ^ 1, abort_flag)) { timed_out = true; break; }
      if (lane == 0) {
        uint8_t* dst = ring + (size_t)stage * Cfg::kStageBytes;
        mbar_expect_tx(&full_bar[stage], 2 * Cfg::NF * 128);
        tma_load_4d(dst, tmX, &full_bar[stage], (int)cblk * 128, M * (int)tw - 1, M * (int)th - 1, (int)img);
        tma_load_4d(dst + Cfg::kHalfBytes, tmX, &full_bar[stage], (int)cblk * 128 + 64, M * (int)tw - 1,
                    M * (int)th - 1, (int)img);
      }
      __syncwarp();
    }
  } else if (warp < Cfg::kProd + Cfg::kMma) {
    constexpr uint32_t idesc = umma_idesc_f16_amn(128, Cfg::NFP);
    if (!mbar_wait_warp(kron_bar, 0, abort_flag)) timed_out = true;
    const uint64_t bd0 = umma_desc_sw128(smem_u32(kron));
    for (unsigned local = warp - Cfg::kProd; local < n_local && !timed_out; local += Cfg::kMma) {
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
  } else if (warp < Cfg::kProd + Cfg::kMma + 4 * Cfg::kEpi) {
    // Epilogue.  The four warps of a group turn a unit's accumulator (128 channels x NF
    // frequencies, a lane = a channel) into a [NF][128] half tile in shared memory, then all
    // 128 threads copy it out with 16-byte stores: every warp store covers two whole 256-byte
    // rows V[f][row][c0..c0+127].  The block counter is raised (after a fence) when the warp
    // moves on to another block or ends, not per unit.
    const int quad = warp & 3;
    const int ew = warp - Cfg::kProd - Cfg::kMma;          // epilogue warp index
    const int group = ew >> 2;
    const int tg = (ew & 3) * 32 + lane;                   // thread index within the group
    uint8_t* out0 = smem + Cfg::kOutOffset + (size_t)group * 2 * Cfg::kOutBufBytes;
    const size_t f_stride = (size_t)RP * C;
    int pend_block = -1;
    uint32_t pend_count = 0;
    uint32_t n_mine = 0;
    for (unsigned local = group; local < n_local && !timed_out; local += Cfg::kEpi, ++n_mine) {
      const unsigned u = rank + local * rp.nI;
      const unsigned p = u / CB, cblk = u % CB;
      const uint32_t acc = local % kNumAcc, acc_phase = (local / kNumAcc) & 1;
      const int blk = (int)(p >> 7);
      if (blk != pend_block) {
        if (pend_count) ctr_signal_n(rp.v_ready + pend_block, pend_count);
        pend_block = blk;
        pend_count = 0;
      }
      if (!mbar_wait_warp(&tmem_full[acc], acc_phase, abort_flag)) { timed_out = true; break; }
      tc_fence_after();
      const uint32_t taddr = tmem_base + ((uint32_t)(quad * 32) << 16) + acc * kAccCols;
      const uint32_t buf = smem_u32(out0) + (n_mine & 1) * Cfg::kOutBufBytes;
      const uint32_t mine = buf + (quad * 32 + lane) * 2;          // this channel's column of the [NF][128] tile
      epi_pass<Cfg, 0>(taddr, mine);
      if constexpr (Cfg::NFP > 64) epi_pass<Cfg, 64>(taddr, mine);
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(&tmem_empty[acc]);
      asm volatile("bar.sync %0, 128;" ::"r"(1 + group) : "memory");
      {
        const int chunk = tg & 15;                         // 16-byte piece of a 256-byte row
        const int c = (int)cblk * 128 + chunk * 8;
        if (c < C) {
          __half* dst = V + (size_t)(p % (unsigned)RP) * C + c + (size_t)(tg >> 4) * f_stride;
          copy_out<Cfg, 0>(buf + (tg >> 4) * 256 + chunk * 16, dst, 8 * f_stride, tg >> 4);
        }
      }
      ++pend_count;
    }
    if (pend_count && !timed_out) ctr_signal_n(rp.v_ready + pend_block, pend_count);
  }
}

// ---------------------------------------------------------------- role G
template <int M, int BLOCK_N>
__device__ __forceinline__ void gemm_init(uint64_t* bars) {
  constexpr int kStages = GCfg<M, BLOCK_N>::kStages;
  uint64_t* full_bar = bars;
  uint64_t* empty_bar = full_bar + kStages;
  uint64_t* tmem_full = empty_bar + kStages;
  uint64_t* tmem_empty = tmem_full + 2;
  uint64_t* stored_bar = tmem_empty + 2;
  for (int s = 0; s < kStages; ++s) { mbar_init(&full_bar[s], 1); mbar_init(&empty_bar[s], 1); }
  for (int a = 0; a < 2; ++a) {
    mbar_init(&tmem_full[a], 1);
    mbar_init(&tmem_empty[a], 8);
    mbar_init(&stored_bar[a], 8);
  }
}
// Warps 0 .. kGWarps-1 of the CTA; barriers and TMEM are set up by the caller.
template <int M, int BLOCK_N>
__device__ __forceinline__ void role_gemm(uint8_t* smem, uint64_t* bars, uint32_t tmem_base,
                                          volatile int* abort_flag, const CUtensorMap* tmV,
                                          const CUtensorMap* tmU, float* __restrict__ Mo, const ConvShape& cs,
                                          const RingParams& rp, int rank, bool& timed_out) {
  using L = GCfg<M, BLOCK_N>;
  constexpr int NF = (M + 2) * (M + 2);
  constexpr int kStages = L::kStages;
  uint64_t* full_bar = bars;
  uint64_t* empty_bar = full_bar + kStages;
  uint64_t* tmem_full = empty_bar + kStages;
  uint64_t* tmem_empty = tmem_full + 2;
  uint64_t* stored_bar = tmem_empty + 2;           // [2]: the epilogue warps have issued an item's stores

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int C = cs.C, K = cs.K;
  const unsigned NB = (unsigned)((rp.P + 127) >> 7);
  const unsigned num_kb = (unsigned)((K + BLOCK_N - 1) / BLOCK_N);
  const int num_ks = (C + BLOCK_K - 1) / BLOCK_K;
  const unsigned per_block = (unsigned)NF * num_kb;
  const unsigned num_items = NB * per_block;
  const unsigned n_local = (num_items > (unsigned)rank) ? (num_items - rank + rp.nGO - 1) / rp.nGO : 0u;
  const int RP = rp.R * 128;
  const unsigned CB = (unsigned)((C + 127) / 128);
  const uint32_t o_target = 16u * (uint32_t)((K + 16 * OCfg<M>::VEC - 1) / (16 * OCfg<M>::VEC)) * 4u;   // see role O

  if (warp == 0) {
    uint32_t stage = 0, phase = 0;
    CtrGate gate_v{0, -1}, gate_o{0, -1};
    for (unsigned local = 0; local < n_local && !timed_out; ++local) {
      const unsigned it = rank + local * rp.nGO;
      const unsigned pb = it / per_block, rem = it % per_block;
      const unsigned f = rem / num_kb, kb = rem % num_kb;
      int tiles = rp.P - (int)pb * 128;
      tiles = tiles > 128 ? 128 : tiles;
      if (rp.nI > 0 && !gate_v.gate(rp.v_ready, (int)pb, (uint32_t)tiles * CB * 4u, abort_flag, rp.abort_all)) {
        timed_out = true; break;
      }
      if ((int)pb >= rp.R && !gate_o.gate(rp.o_done, (int)pb - rp.R, o_target, abort_flag, rp.abort_all)) {
        timed_out = true; break;
      }
      async_proxy_acquire();
      const int row0 = (int)(pb % (unsigned)rp.RV) * 128;
      for (int ks = 0; ks < num_ks; ++ks) {
        if (!mbar_wait_warp(&empty_bar[stage], phase ^ 1, abort_flag)) { timed_out = true; break; }
        if (lane == 0) {
          uint8_t* sa = smem + stage * L::kStageBytes;
          uint8_t* sb = sa + L::kABytes;
          mbar_expect_tx(&full_bar[stage], L::kStageBytes);
          tma_load_3d(sa, tmV, &full_bar[stage], ks * BLOCK_K, row0, (int)f);
          tma_load_3d(sb, tmU, &full_bar[stage], ks * BLOCK_K, (int)kb * BLOCK_N, (int)f);
        }
        __syncwarp();
        if (++stage == kStages) { stage = 0; phase ^= 1; }
      }
      if (local + 1 < n_local) {                       // look one item ahead
        const int npb = (int)((rank + (local + 1) * rp.nGO) / per_block);
        if (rp.nI > 0) gate_v.prefetch(rp.v_ready, npb);
        gate_o.prefetch(rp.o_done, npb >= rp.R ? npb - rp.R : -1);
      }
    }
  } else if (warp == 1) {
    constexpr uint32_t idesc = umma_idesc_f16(BLOCK_M, BLOCK_N);
    uint32_t stage = 0, phase = 0;
    for (unsigned local = 0; local < n_local && !timed_out; ++local) {
      const uint32_t acc = local & 1, acc_phase = (local >> 1) & 1;
      if (!mbar_wait_warp(&tmem_empty[acc], acc_phase ^ 1, abort_flag)) { timed_out = true; break; }
      tc_fence_after();
      const uint32_t tmem_d = tmem_base + acc * BLOCK_N;
      for (int ks = 0; ks < num_ks; ++ks) {
        if (!mbar_wait_warp(&full_bar[stage], phase, abort_flag)) { timed_out = true; break; }
        tc_fence_after();
        if (lane == 0) {
          const uint32_t sa = smem_u32(smem + stage * L::kStageBytes);
          const uint32_t sb = sa + L::kABytes;
const uint64_t ad0 = umma_desc_sw128(sa), bd0 = umma_desc_sw128(sb);
          umma_f16(tmem_d, ad0, bd0, idesc, ks > 0 ? 1u : 0u);
#pragma unroll
          for (int k = 1; k < BLOCK_K / 16; ++k)
            umma_f16_c<true>(tmem_d, umma_desc_advance(ad0, k * 32), umma_desc_advance(bd0, k * 32), idesc);
          umma_commit(&empty_bar[stage]);
          if (ks == num_ks - 1) umma_commit(&tmem_full[acc]);
        }
        __syncwarp();
        if (++stage == kStages) { stage = 0; phase ^= 1; }
      }
    }
  } else if (warp < 10) {
    // Epilogue: warps 2-5 drain columns [0, BLOCK_N/2), warps 6-9 the other half (each set has
    // one warp per TMEM lane quadrant).  A warp stores straight from registers (16-byte stores,
    // 512 contiguous bytes per warp instruction in the quad-major M layout), then arrives on
    // stored_bar and moves on; warp 10 makes the item's stores visible and raises the counter.
    const int quad = warp & 3;
    const int half = (warp - 2) >> 2;
    const int k4 = K >> 2;
    constexpr int HALF_N = BLOCK_N / 2;
    for (unsigned local = 0; local < n_local && !timed_out; ++local) {
      const unsigned it = rank + local * rp.nGO;
      const unsigned pb = it / per_block, rem = it % per_block;
      const unsigned f = rem / num_kb, kb = rem % num_kb;
      const uint32_t acc = local & 1, acc_phase = (local >> 1) & 1;
      if (!mbar_wait_warp(&tmem_full[acc], acc_phase, abort_flag)) { timed_out = true; break; }
      tc_fence_after();
      const int row = (int)(pb % (unsigned)rp.R) * 128 + quad * 32 + lane;
      const int col_base = (int)kb * BLOCK_N + half * HALF_N;
      const int k_left = K - col_base;
      float* dst = Mo + (((size_t)f * k4 + (size_t)(col_base >> 2)) * RP + row) * 4;
      const size_t q_stride = (size_t)RP * 4;
#pragma unroll 2
      for (int cb = 0; cb < HALF_N; cb += 32) {
        if (cb >= k_left) break;
        uint32_t r[32];
        tmem_ld32(tmem_base + ((uint32_t)(quad * 32) << 16) + acc * BLOCK_N + half * HALF_N + cb, r);
        tmem_ld_wait();
#pragma unroll
        for (int j = 0; j < 8; ++j)
          if (cb + 4 * j < k_left)
            *reinterpret_cast<uint4*>(dst + (size_t)((cb >> 2) + j) * q_stride) =
                make_uint4(r[4 * j], r[4 * j + 1], r[4 * j + 2], r[4 * j + 3]);
      }
      tc_fence_before();
      __syncwarp();
      if (lane == 0) {
        mbar_arrive(&tmem_empty[acc]);
        mbar_arrive(&stored_bar[acc]);
      }
    }
  } else if (warp == 10) {
    // Signalling warp: once all eight epilogue warps have issued an item's stores (barrier,
    // CTA scope), one fence at GPU scope orders them before the counter update.
    for (unsigned local = 0; local < n_local && !timed_out; ++local) {
      const unsigned it = rank + local * rp.nGO;
      const unsigned pb = it / per_block;
      const uint32_t acc = local & 1, acc_phase = (local >> 1) & 1;
      if (!mbar_wait_warp(&stored_bar[acc], acc_phase, abort_flag)) { timed_out = true; break; }
      if (lane == 0) {
        __threadfence();
        asm volatile("fence.proxy.async.global;" ::: "memory");
        asm volatile("red.release.gpu.global.add.u32 [%0], 4;" ::"l"(rp.g_done + pb) : "memory");
      }
      __syncwarp();
    }
  }
}

// ---------------------------------------------------------------- role O
template <int M>
__device__ __forceinline__ void output_init(uint64_t* bars) {
  constexpr int kStages = OCfg<M>::kStages;
  for (int s = 0; s < kStages; ++s) { mbar_init(&bars[s], 1); mbar_init(&bars[kStages + s], 4); }
}
// Warps kOWarpBase .. kOWarpBase+4 of the CTA (`warp` is relative to kOWarpBase): one TMA producer
// and one consumer group of four warps.
template <int M, bool SYM>
__device__ __forceinline__ void role_output(int warp, uint8_t* smem, uint64_t* bars, volatile int* abort_flag,
                                            const CUtensorMap* tmM, const Coefs& cf, __half* __restrict__ y,
                                            const ConvShape& cs, const RingParams& rp, int rank, int size,
                                            bool& timed_out) {
  using Cfg = OCfg<M>;
  constexpr int N = Cfg::N;
  constexpr int kStages = Cfg::kStages;
  uint64_t* full_bar = bars;
  uint64_t* empty_bar = full_bar + kStages;

  const int lane = threadIdx.x & 31;
  const int K = cs.K, H = cs.H, W = cs.W;
  constexpr int VEC = Cfg::VEC;
  const unsigned KG = (unsigned)((K + 16 * VEC - 1) / (16 * VEC));
  const unsigned NB = (unsigned)((rp.P + 127) >> 7);
  const unsigned num_units = NB * 16u * KG;
  const unsigned n_local = (num_units > (unsigned)rank) ? (num_units - rank + size - 1) / size : 0u;
  const int RP = rp.R * 128;
  const uint32_t g_target = rp.g_target;

  if (warp == 0) {
    CtrGate gate_g{0, -1};
    for (unsigned local = 0; local < n_local && !timed_out; ++local) {
      const unsigned u = rank + local * size;
      const unsigned tg = u / KG, kg = u % KG;
      const unsigned b = tg >> 4;
      if (!gate_g.gate(rp.g_done, (int)b, g_target, abort_flag, rp.abort_all)) { timed_out = true; break; }
      async_proxy_acquire();
      const uint32_t stage = local % kStages, phase = (local / kStages) & 1;
      if (!mbar_wait_warp(&empty_bar[stage], phase ^ 1, abort_flag)) { timed_out = true; break; }
      if (lane == 0) {
        mbar_expect_tx(&full_bar[stage], Cfg::kStageBytes);
        tma_load_3d(smem + (size_t)stage * Cfg::kStageBytes, tmM, &full_bar[stage],
                    (int)((tg * 8u) % (unsigned)RP) * 4, (int)kg * Cfg::kQuads, 0);
      }
      __syncwarp();
      if (local + 1 < n_local) gate_g.prefetch(rp.g_done, (int)(((rank + (local + 1) * size) / KG) >> 4));
    }
  } else if (warp <= 4 * Cfg::kGroups) {
    const int group = (warp - 1) >> 2;
    const int w = (warp - 1) & 3;
    const int t = w + 4 * (lane >> 4);
    const int kq = (VEC == 1) ? (lane & 15) >> 2 : (lane & 15) >> 1;
    const int kk = (VEC == 1) ? (lane & 3) : (lane & 1) * 2;
    const uint32_t off_even = kq * 128 + ((t ^ kq) << 4) + kk * 4;
    const uint32_t off_odd = kq * 128 + ((t ^ ((kq + 4) & 7)) << 4) + kk * 4;
    for (unsigned local = group; local < n_local && !timed_out; local += Cfg::kGroups) {
      const unsigned u = rank + local * size;
      const unsigned tg = u / KG, kg = u % KG;
      const uint32_t stage = local % kStages, phase = (local / kStages) & 1;
      if (!mbar_wait_warp(&full_bar[stage], phase, abort_flag)) { timed_out = true; break; }
      const uint32_t sb = smem_u32(smem) + stage * Cfg::kStageBytes;
      const uint32_t sb_even = sb + off_even, sb_odd = sb + off_odd;
      typename VecOf<VEC>::type Y[M][M];
      OutputTile<M, SYM, VEC>{cf, sb_even, sb_odd}.run(Y);
      __syncwarp();
      if (lane == 0) mbar_arrive(&empty_bar[stage]);
      ctr_signal_read(rp.o_done + (tg >> 4));

      const int pl = (int)tg * 8 + t;
      const int k = (int)kg * 16 * VEC + (lane & 15) * VEC;
      if (pl < rp.P && k < K) {
        const unsigned p = (unsigned)pl;
        const unsigned tw = p % (unsigned)cs.Tw, q2 = p / (unsigned)cs.Tw;
        const unsigned th = q2 % (unsigned)cs.Th, img = q2 / (unsigned)cs.Th;
        const int h0 = M * (int)th, w0 = M * (int)tw;
        __half* dst = y + (((size_t)img * H + h0) * W + w0) * K + k;
        store_tile<M, __half>(Y, dst, (size_t)W * K, K, H - h0, W - w0, cs.relu);
      }
    }
  }
}

// ---------------------------------------------------------------- the kernel
template <int M, int BLOCK_N, bool SYM>
__global__ void __launch_bounds__(kFusedThreads, 1)
fused_conv_kernel(const __grid_constant__ CUtensorMap tmX, const __grid_constant__ CUtensorMap tmKron,
                  const __grid_constant__ CUtensorMap tmV, const __grid_constant__ CUtensorMap tmU,
                  const __grid_constant__ CUtensorMap tmM, const __grid_constant__ Coefs cf,
                  __half* __restrict__ V, float* __restrict__ Mo, __half* __restrict__ y,
                  const ConvShape cs, const RingParams rp, int* __restrict__ status) {
  using F = FusedCfg<M, BLOCK_N>;
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
  uint64_t* bars = reinterpret_cast<uint64_t*>(smem + F::kBarrierOffset);
  uint32_t* tmem_base_slot = reinterpret_cast<uint32_t*>(bars + 48);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_base_slot + 1);
  if (threadIdx.x == 0) *abort_flag = 0;
  __syncthreads();

  bool timed_out = false;
  const int b = blockIdx.x;
  const int warp = threadIdx.x >> 5;
  const bool is_input = b < rp.nI;
  constexpr uint32_t kTmemCols = 512;
  if (is_input) input_prologue<M>(smem, bars);
  if (threadIdx.x == 0) {
    if (!is_input) gemm_init<M, BLOCK_N>(bars);
    output_init<M>(bars + kIBarriers);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 1) tmem_alloc(tmem_base_slot, kTmemCols);
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_base_slot;
  // role O: every CTA (except next to role I where the shared memory does not hold both)
  const bool o_here = F::kOWithI || !is_input;
  const int o_rank = F::kOWithI ? b : b - rp.nI;
  const int o_size = F::kOWithI ? (int)gridDim.x : rp.nGO;
  if (warp >= kOWarpBase) {
    if (o_here)
      role_output<M, SYM>(warp - kOWarpBase, smem + F::kOOffset, bars + kIBarriers, abort_flag, &tmM, cf, y, cs, rp,
                          o_rank, o_size, timed_out);
  } else if (is_input) {
    role_input<M>(smem, bars, tmem_base, abort_flag, &tmX, &tmKron, V, cs, rp, b, timed_out);
  } else if (warp < kGWarps) {
    role_gemm<M, BLOCK_N>(smem, bars, tmem_base, abort_flag, &tmV, &tmU, Mo, cs, rp, b - rp.nI, timed_out);
  }
  tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    tc_fence_after();
    tmem_dealloc(tmem_base, kTmemCols);
  }

  if (timed_out) {
    *abort_flag = 1;
    if ((threadIdx.x & 31) == 0) {
      atomicExch(rp.abort_all, 1);
      atomicExch(status, NOVA_ERR_DEVICE_TIMEOUT);
    }
  }
}

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*,
                                  CUtensorMapInterleave, CUtensorMapSwizzle, CUtensorMapL2promotion,
                                  CUtensorMapFloatOOBfill);
EncodeTiledFn encode_fn() {
  static EncodeTiledFn fn = nullptr;
  static bool tried = false;
  if (!tried) {
    tried = true;
    void* p = nullptr;
    cudaDriverEntryPointQueryResult q;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) == cudaSuccess &&
        q == cudaDriverEntryPointSuccess)
      fn = (EncodeTiledFn)p;
  }
  return fn;
}
bool encode(CUtensorMap* map, CUtensorMapDataType dt, int rank, const void* base, const cuuint64_t* dims,
            const cuuint64_t* strides, const cuuint32_t* box, CUtensorMapL2promotion promo,
            CUtensorMapSwizzle swz = CU_TENSOR_MAP_SWIZZLE_128B) {
  EncodeTiledFn enc = encode_fn();
  if (!enc) return false;
  cuuint32_t estr[5] = {1, 1, 1, 1, 1};
  return enc(map, dt, rank, const_cast<void*>(base), dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
             swz, promo, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// nI_req < 0: the plan's (or the default) share of CTAs runs role I and V is a ring of R blocks;
// nI_req == 0: V (all tiles) was produced by an earlier kernel and every CTA runs roles G and O.
template <int M, int BLOCK_N, bool SYM>
int launch_fused_t(const nova_plan* plan, const Geom& g, const void* x, const void* U, void* y, void* Vr,
                   float* Mr, int R, int nI_req, int relu, cudaStream_t stream) {
  using F = FusedCfg<M, BLOCK_N>;
  constexpr int n = M + 2, NF = n * n;
  static bool attr_set = false;
  if (!attr_set) {
    cudaError_t e = cudaFuncSetAttribute(fused_conv_kernel<M, BLOCK_N, SYM>,
                                         cudaFuncAttributeMaxDynamicSharedMemorySize, F::kTotal);
    if (e != cudaSuccess) return (int)e;
    attr_set = true;
  }
  const int NB = (int)((g.P + 127) / 128);
  const int RV = (nI_req == 0) ? NB : R;
  const int RP = R * 128, RPV = RV * 128;
  CUtensorMap tmX, tmK, tmV, tmU, tmM;
  const CUtensorMapDataType f16 = CU_TENSOR_MAP_DATA_TYPE_FLOAT16, f32 = CU_TENSOR_MAP_DATA_TYPE_FLOAT32;
  const CUtensorMapL2promotion p256 = CU_TENSOR_MAP_L2_PROMOTION_L2_256B, p128 = CU_TENSOR_MAP_L2_PROMOTION_L2_128B;
  {
    cuuint64_t dims[4] = {(cuuint64_t)g.C, (cuuint64_t)g.W, (cuuint64_t)g.H, (cuuint64_t)g.N};
    cuuint64_t strides[3] = {(cuuint64_t)g.C * 2, (cuuint64_t)g.W * g.C * 2, (cuuint64_t)g.H * g.W * g.C * 2};
    cuuint32_t box[4] = {64, (cuuint32_t)n, (cuuint32_t)n, 1};
    if (!encode(&tmX, f16, 4, x, dims, strides, box, p256)) return (int)cudaErrorUnknown;
  }
  {
    using IC = ICfg<M>;
    cuuint64_t dims[2] = {64, (cuuint64_t)(2 * IC::KA * IC::NFP)};
    cuuint64_t strides[1] = {128};
    cuuint32_t box[2] = {64, (cuuint32_t)IC::NFP};
    if (!encode(&tmK, f16, 2, plan->kron_dev, dims, strides, box, p256)) return (int)cudaErrorUnknown;
  }
  {
    cuuint64_t dims[3] = {(cuuint64_t)g.C, (cuuint64_t)RPV, (cuuint64_t)NF};
    cuuint64_t strides[2] = {(cuuint64_t)g.C * 2, (cuuint64_t)RPV * g.C * 2};
    cuuint32_t box[3] = {BLOCK_K, BLOCK_M, 1};
    if (!encode(&tmV, f16, 3, Vr, dims, strides, box, p128)) return (int)cudaErrorUnknown;
  }
  {
    cuuint64_t dims[3] = {(cuuint64_t)g.C, (cuuint64_t)g.K, (cuuint64_t)NF};
    cuuint64_t strides[2] = {(cuuint64_t)g.C * 2, (cuuint64_t)g.K * g.C * 2};
    cuuint32_t box[3] = {BLOCK_K, (cuuint32_t)BLOCK_N, 1};
    if (!encode(&tmU, f16, 3, U, dims, strides, box, p256)) return (int)cudaErrorUnknown;
  }
  {
    const int k4 = g.K / 4;
    cuuint64_t dims[3] = {(cuuint64_t)RP * 4, (cuuint64_t)k4, (cuuint64_t)NF};
    cuuint64_t strides[2] = {(cuuint64_t)RP * 16, (cuuint64_t)k4 * RP * 16};
    cuuint32_t box[3] = {32, (cuuint32_t)OCfg<M>::kQuads, (cuuint32_t)NF};
    if (!encode(&tmM, f32, 3, Mr, dims, strides, box, p128)) return (int)cudaErrorUnknown;
  }
  uint32_t* ctr = plan->fused_ctr_dev;
  if (cudaMemsetAsync(ctr, 0, (size_t)(3 * NB + 4) * sizeof(uint32_t), stream) != cudaSuccess)
    return (int)cudaErrorUnknown;
  RingParams rp;
  rp.v_ready = ctr;
  rp.g_done = ctr + NB;
  rp.o_done = ctr + 2 * NB;
  rp.abort_all = reinterpret_cast<int*>(ctr + 3 * NB);
  rp.R = R;
  rp.RV = RV;
  rp.P = (int)g.P;
  const int sms = plan->sm_count;
  int nI = plan->fused_nI;
  if (nI <= 0 || nI >= sms) nI = sms * 43 / 100;      // default share of the SMs for role I
  if (nI_req == 0) nI = 0;
  rp.nI = nI;
  rp.nGO = sms - nI;
  rp.g_target = (uint32_t)NF * (uint32_t)((g.K + BLOCK_N - 1) / BLOCK_N) * 4u;
  ConvShape cs{g.H, g.W, g.C, g.K, g.Th, g.Tw, relu};

  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3((unsigned)sms);
  cfg.blockDim = dim3(kFusedThreads);
  cfg.dynamicSmemBytes = F::kTotal;
  cfg.stream = stream;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeCooperative;        // all CTAs co-resident, or the launch fails
  attr[0].val.cooperative = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  return (int)cudaLaunchKernelEx(&cfg, fused_conv_kernel<M, BLOCK_N, SYM>, tmX, tmK, tmV, tmU, tmM, plan->kcoefs,
                                 (__half*)Vr, Mr, (__half*)y, cs, rp, plan->status_dev);
}

template <int M>
int launch_fused_m(const nova_plan* plan, const Geom& g, const void* x, const void* U, void* y, void* Vr,
                   float* Mr, int R, int nI_req, int relu, cudaStream_t s) {
  if (plan->symmetric) return launch_fused_t<M, 256, true>(plan, g, x, U, y, Vr, Mr, R, nI_req, relu, s);
  return launch_fused_t<M, 256, false>(plan, g, x, U, y, Vr, Mr, R, nI_req, relu, s);
}

}  // namespace

size_t fused_block_bytes(const nova_plan* plan, int C, int K) {
  return (size_t)plan->n * plan->n * 128 * ((size_t)C * 2 + (size_t)K * 4);
}

int launch_fused_conv(const nova_plan* plan, const Geom& g, const void* x, const void* U, void* y, void* ws,
                      int R, int relu, void* stream) {
  cudaStream_t s = (cudaStream_t)stream;
  const size_t v_bytes = ((size_t)plan->n * plan->n * R * 128 * g.C * 2 + 255) / 256 * 256;
  void* Vr = ws;
  float* Mr = reinterpret_cast<float*>(static_cast<char*>(ws) + v_bytes);
  switch (plan->m) {
    case 2: return launch_fused_m<2>(plan, g, x, U, y, Vr, Mr, R, -1, relu, s);
    case 4: return launch_fused_m<4>(plan, g, x, U, y, Vr, Mr, R, -1, relu, s);
    case 6: return launch_fused_m<6>(plan, g, x, U, y, Vr, Mr, R, -1, relu, s);
    case 8: return launch_fused_m<8>(plan, g, x, U, y, Vr, Mr, R, -1, relu, s);
  }
  return (int)cudaErrorInvalidValue;
}

// Product and output transform in one kernel over a V that holds all tiles ([n*n][P_pad][C], written by
// the input-transform kernel before): every CTA runs roles G and O, M is a ring of R blocks.
int launch_fused_product_output(const nova_plan* plan, const Geom& g, const void* x, const void* V, const void* U,
                                void* y, float* Mring, int R, int relu, void* stream) {
  cudaStream_t s = (cudaStream_t)stream;
  void* Vr = const_cast<void*>(V);
  switch (plan->m) {
    case 2: return launch_fused_m<2>(plan, g, x, U, y, Vr, Mring, R, 0, relu, s);
    case 4: return launch_fused_m<4>(plan, g, x, U, y, Vr, Mring, R, 0, relu, s);
    case 6: return launch_fused_m<6>(plan, g, x, U, y, Vr, Mring, R, 0, relu, s);
    case 8: return launch_fused_m<8>(plan, g, x, U, y, Vr, Mring, R, 0, relu, s);
  }
  return (int)cudaErrorInvalidValue;
}

}  // namespace nova
