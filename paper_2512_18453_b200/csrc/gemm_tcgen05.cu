// Transformed-domain product on the sm_100a tensor cores (Section 2.1 step 3
// summed over input channels): for every frequency f,
//   M[f][p][k] = sum_c V[f][p][c] * U[f][k][c],   half x half -> float,
// or, for the int8 pipeline (I8), signed 8-bit x signed 8-bit -> int32 (exact).
//
// Persistent, warp-specialised kernel.  One CTA per SM walks a list of work
// items (f, 128-row block of tiles p, BLOCK_N-wide block of filters k; the filter blocks of a (f, p) pair one after the other):
//   warp 0    TMA producer: 128B-swizzled [rows][64 channels] boxes of V and U
//             into a 4-stage shared-memory ring, completion on mbarriers;
//   warp 1    issues tcgen05.mma (kind::f16, M=128, N=BLOCK_N, K=16) from
//             shared-memory descriptors into one of two TMEM accumulators;
//   warps 2-9 epilogue, warps 2-5 for the first half of the columns and warps
//             6-9 for the second: tcgen05.ld the finished accumulator (one TMEM lane
//             quadrant per warp; a lane is a tile, a column a filter) and
//             store it straight from registers, overlapping the next item's
//             MMAs on the other accumulator.  M is laid out
//             [f][K/4][pc_pad][4]: each 16-byte store instruction of a warp
//             then covers 512 contiguous bytes (32 tiles x 4 filters).
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

constexpr int BLOCK_M = 128;
constexpr int kRowBytes = 128;         // one swizzle row of K per stage: 64 halves or 128 int8
constexpr int kUmmaBytes = 32;         // K bytes one tcgen05.mma contracts (16 halves / 32 int8)
constexpr int kStages = 4;
constexpr int kThreads = 320;          // producer, MMA issuer, 2 x 4 epilogue warps

template <int BLOCK_N>
struct SmemLayout {
  static constexpr int kABytes = BLOCK_M * kRowBytes;
  static constexpr int kBBytes = BLOCK_N * kRowBytes;
  static constexpr int kStageBytes = kABytes + kBBytes;
  static constexpr int kBarrierOffset = kStages * kStageBytes;
  static constexpr int kTotal = kBarrierOffset + 256 + 1024;     // barriers + alignment slack
};

// Measurement aid: sums of clock64() spent in (or around) the waits of one warp.  With ON = false
// every member is empty and the kernel is the production one.
template <bool ON>
struct WaitClock {
  long long sum = 0, t0 = 0;
  __device__ __forceinline__ void start() { if constexpr (ON) t0 = clock64(); }
  __device__ __forceinline__ void stop() { if constexpr (ON) sum += clock64() - t0; }
};

template <int BLOCK_N, bool I8, bool PROF = false>
__global__ void __launch_bounds__(kThreads, 1)
gemm_tcgen05_kernel(const __grid_constant__ CUtensorMap tmV, const __grid_constant__ CUtensorMap tmU,
                    float* __restrict__ Mo, int nfreq, int pc, int pc_pad, int C, int K,
                    int* __restrict__ status, const uint8_t* __restrict__ Vdrop, int f_major, int keep_pct,
                    unsigned long long* __restrict__ prof) {
  using L = SmemLayout<BLOCK_N>;
  constexpr int BLOCK_K = I8 ? kRowBytes : kRowBytes / 2;   // elements of K per stage
  constexpr uint32_t kTmemCols = 2 * BLOCK_N;       // two accumulators; 128, 256 or 512
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
  uint64_t* full_bar = reinterpret_cast<uint64_t*>(smem + L::kBarrierOffset);
  uint64_t* empty_bar = full_bar + kStages;
  uint64_t* tmem_full = empty_bar + kStages;        // [2]
  uint64_t* tmem_empty = tmem_full + 2;             // [2]
  uint32_t* tmem_base_slot = reinterpret_cast<uint32_t*>(tmem_empty + 2);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_base_slot + 1);

  const int warp = threadIdx.x >> 5;
  const int lane = threadIdx.x & 31;
  const int num_pb = (pc + BLOCK_M - 1) / BLOCK_M;
  const int num_kb = (K + BLOCK_N - 1) / BLOCK_N;
  const int num_ks = (C + BLOCK_K - 1) / BLOCK_K;
  // The work list is (row block, frequency), the row block outermost and DESCENDING: the input
  // transform wrote V in ascending tile order, so the highest row blocks are the ones still in
  // L2; and the row blocks this kernel finishes last - the lowest - are the ones the output
  // transform reads first.  With f_major the frequency is outermost instead (see the launcher).
  // Pair i of this CTA is pair blockIdx.x + i * gridDim.x; the CTA runs
  // the pair's filter blocks one after the other (items), so that it is the only reader of the
  // pair's rows of V and knows when they have been read for the last time.
  const long long num_pairs = (long long)nfreq * num_pb;
  const uint32_t pairs_local = num_pairs > blockIdx.x ? (uint32_t)((num_pairs - blockIdx.x + gridDim.x - 1) / gridDim.x) : 0u;
  const uint32_t n_local = pairs_local * (uint32_t)num_kb;
  auto item_of = [&](uint32_t local, int& pb, int& f, int& kb) {
    const unsigned pair = blockIdx.x + (local / (unsigned)num_kb) * gridDim.x;
    if (f_major) { f = (int)(pair / (unsigned)num_pb); pb = num_pb - 1 - (int)(pair % (unsigned)num_pb); }
    else { pb = num_pb - 1 - (int)(pair / (unsigned)nfreq); f = (int)(pair % (unsigned)nfreq); }
    kb = (int)(local % (unsigned)num_kb);
  };

  if (threadIdx.x == 0) {
    for (int s = 0; s < kStages; ++s) { mbar_init(&full_bar[s], 1); mbar_init(&empty_bar[s], 1); }
    for (int a = 0; a < 2; ++a) { mbar_init(&tmem_full[a], 1); mbar_init(&tmem_empty[a], 8); }
    *abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 1) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(
                     smem_u32(tmem_base_slot)),
                 "r"(kTmemCols)
                 : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  __syncthreads();
  asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
  const uint32_t tmem_base = *tmem_base_slot;
  bool timed_out = false;
  // everything above touched no global memory: it may overlap the tail of the preceding kernel
  pdl_launch_dependents();
  pdl_wait();

  if (warp == 0) {
    // ---------------- TMA producer
    WaitClock<PROF> w_empty, total;
    total.start();
    uint32_t stage = 0, phase = 0;
    for (uint32_t local = 0; local < n_local && !timed_out; ++local) {
      int pb, f, kb;
      item_of(local, pb, f, kb);
      for (int ks = 0; ks < num_ks; ++ks) {
        w_empty.start();
        if (!mbar_wait_warp(&empty_bar[stage], phase ^ 1, abort_flag)) { timed_out = true; break; }
        w_empty.stop();
        if (lane == 0) {
          uint8_t* sa = smem + stage * L::kStageBytes;
          uint8_t* sb = sa + L::kABytes;
          mbar_expect_tx(&full_bar[stage], L::kStageBytes);
          tma_load_3d(sa, &tmV, &full_bar[stage], ks * BLOCK_K, pb * BLOCK_M, f);
          tma_load_3d(sb, &tmU, &full_bar[stage], ks * BLOCK_K, kb * BLOCK_N, f);
        }
        __syncwarp();
        if (++stage == kStages) { stage = 0; phase ^= 1; }
      }
    }
    if constexpr (PROF) {
      total.stop();
      if (lane == 0) { prof[blockIdx.x * 8 + 0] = w_empty.sum; prof[blockIdx.x * 8 + 1] = total.sum; }
    }
  } else if (warp == 1) {
    // ---------------- MMA issuer
    constexpr uint32_t idesc = I8 ? umma_idesc_i8(BLOCK_M, BLOCK_N) : umma_idesc_f16(BLOCK_M, BLOCK_N);
    WaitClock<PROF> w_acc, w_ops, total;
    total.start();
    uint32_t stage = 0, phase = 0;
    for (uint32_t local = 0; local < n_local && !timed_out; ++local) {
      const uint32_t acc = local & 1, acc_phase = (local >> 1) & 1;
      w_acc.start();
      if (!mbar_wait_warp(&tmem_empty[acc], acc_phase ^ 1, abort_flag)) { timed_out = true; break; }
      w_acc.stop();
      asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
      const uint32_t tmem_d = tmem_base + acc * BLOCK_N;
      int item_pb, item_f, item_kb;
      item_of(local, item_pb, item_f, item_kb);
      for (int ks = 0; ks < num_ks; ++ks) {
        w_ops.start();
        if (!mbar_wait_warp(&full_bar[stage], phase, abort_flag)) { timed_out = true; break; }
        w_ops.stop();
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
        if (lane == 0) {
          const uint32_t sa = smem_u32(smem + stage * L::kStageBytes);
          const uint32_t sb = sa + L::kABytes;
          const uint64_t ad0 = umma_desc_sw128(sa), bd0 = umma_desc_sw128(sb);
          if constexpr (I8) {
            umma_i8(tmem_d, ad0, bd0, idesc, ks > 0 ? 1u : 0u);
#pragma unroll
            for (int k = 1; k < kRowBytes / kUmmaBytes; ++k)
              umma_i8(tmem_d, umma_desc_advance(ad0, k * kUmmaBytes), umma_desc_advance(bd0, k * kUmmaBytes), idesc, 1u);
          } else {
            umma_f16(tmem_d, ad0, bd0, idesc, ks > 0 ? 1u : 0u);
#pragma unroll
            for (int k = 1; k < kRowBytes / kUmmaBytes; ++k)
              umma_f16_c<true>(tmem_d, umma_desc_advance(ad0, k * kUmmaBytes), umma_desc_advance(bd0, k * kUmmaBytes), idesc);
          }
          umma_commit(&empty_bar[stage]);                 // frees the smem stage when the MMAs retire
          if (ks == num_ks - 1) umma_commit(&tmem_full[acc]);
        }
        __syncwarp();
        // V is scratch and this was the last read of the 128 rows x 128 bytes that have just
        // landed in shared memory: drop those lines from the L2, so that the ones still dirty
        // there (the input transform wrote them moments ago) are never written back.
        if (Vdrop && item_kb == num_kb - 1) {
          const uint8_t* line = Vdrop + (((size_t)item_f * pc_pad + (size_t)item_pb * BLOCK_M) * C) * (I8 ? 1 : 2) +
                                (size_t)ks * kRowBytes;
          const size_t pitch = (size_t)C * (I8 ? 1 : 2);
#pragma unroll
          for (int r = 0; r < BLOCK_M / 32; ++r) l2_discard_line(line + (size_t)(r * 32 + lane) * pitch);
        }
        if (++stage == kStages) { stage = 0; phase ^= 1; }
      }
    }
    if constexpr (PROF) {
      total.stop();
      if (lane == 0) {
        prof[blockIdx.x * 8 + 2] = w_acc.sum; prof[blockIdx.x * 8 + 3] = w_ops.sum; prof[blockIdx.x * 8 + 4] = total.sum;
        prof[blockIdx.x * 8 + 7] = n_local;
      }
    }
  } else {
    // ---------------- epilogue (warps 2..9); a warp may only read TMEM lanes 32*(warp%4)..+31.
    // Rows >= pc of the last row block are zeros (the TMA loads of V fill them) and land in the
    // padding rows pc..pc_pad-1 of M.
    const int quad = warp & 3;
    const int half = (warp - 2) >> 2;                    // which half of the BLOCK_N columns
    constexpr int HALF_N = BLOCK_N / 2;
    const int k4 = K >> 2;
    WaitClock<PROF> w_full, total;
    total.start();
    for (uint32_t local = 0; local < n_local && !timed_out; ++local) {
      int pb, f, kb;
      item_of(local, pb, f, kb);
      const uint32_t acc = local & 1, acc_phase = (local >> 1) & 1;
      w_full.start();
      if (!mbar_wait_warp(&tmem_full[acc], acc_phase, abort_flag)) { timed_out = true; break; }
      w_full.stop();
      asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
      // M is larger than the L2 on the layers that matter, and the output transform reads the row
      // blocks written last (the lowest) first: the share of row blocks that can still be resident
      // then is stored evict-last, the rest evict-first, so that the early blocks, which are lost
      // anyway, do not push out the late ones.
      uint64_t pol;
      if (pb * 100 < num_pb * keep_pct) asm volatile("createpolicy.fractional.L2::evict_last.b64 %0, 1.0;" : "=l"(pol));
      else asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(pol));
      const int row = pb * BLOCK_M + quad * 32 + lane;
      const int col_base = kb * BLOCK_N + half * HALF_N;
      const int k_left = K - col_base;
      float* dst = Mo + (((size_t)f * k4 + (size_t)(col_base >> 2)) * pc_pad + row) * 4;
      const size_t q_stride = (size_t)pc_pad * 4;        // floats between consecutive filter quads
#pragma unroll 1
      for (int cb = 0; cb < HALF_N && cb < k_left; cb += 32) {
        uint32_t r[32];
        tmem_ld32(tmem_base + ((uint32_t)(quad * 32) << 16) + acc * BLOCK_N + half * HALF_N + cb, r);
        asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
#pragma unroll
        for (int j = 0; j < 8; ++j)
          if (cb + 4 * j < k_left)
            asm volatile("st.global.L2::cache_hint.v4.b32 [%0], {%1, %2, %3, %4}, %5;" ::"l"(dst + (size_t)((cb >> 2) + j) * q_stride),
                         "r"(r[4 * j]), "r"(r[4 * j + 1]), "r"(r[4 * j + 2]), "r"(r[4 * j + 3]), "l"(pol) : "memory");
      }
      asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
      __syncwarp();
      if (lane == 0) mbar_arrive(&tmem_empty[acc]);
    }
    if constexpr (PROF) {
      total.stop();
      if (warp == 2 && lane == 0) { prof[blockIdx.x * 8 + 5] = w_full.sum; prof[blockIdx.x * 8 + 6] = total.sum; }
    }
  }

  if (timed_out) {
    *abort_flag = 1;
    if (lane == 0) atomicExch(status, NOVA_ERR_DEVICE_TIMEOUT);
  }
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  __syncthreads();
  if (warp == 1) {
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(kTmemCols)
                 : "memory");
  }
}

// [nfreq][rows][inner] elements of `esize` bytes, frequency stride in elements;
// box = [1][box_rows][box_inner], 128-byte swizzle (box_inner * esize == 128).
bool make_map_3d(CUtensorMap* map, CUtensorMapDataType dt, int esize, const void* base, int inner, int rows,
                 long long freq_stride_elems, int nfreq, int box_inner, int box_rows) {
  EncodeTiledFn enc = tensor_map_encoder();
  if (!enc) return false;
  cuuint64_t dims[3] = {(cuuint64_t)inner, (cuuint64_t)rows, (cuuint64_t)nfreq};
  cuuint64_t strides[2] = {(cuuint64_t)inner * esize, (cuuint64_t)freq_stride_elems * esize};
  cuuint32_t box[3] = {(cuuint32_t)box_inner, (cuuint32_t)box_rows, 1};
  cuuint32_t estr[3] = {1, 1, 1};
  return enc(map, dt, 3, const_cast<void*>(base), dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
             CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
             CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

template <int BLOCK_N, bool I8>
int launch_n(int sms, int l2_bytes, const void* V, const void* U, float* M, int nfreq, int pc, int pc_pad, int C, int K,
             int* status, cudaStream_t stream, unsigned long long* prof = nullptr) {
  using L = SmemLayout<BLOCK_N>;
  if (cudaError_t e = allow_dynamic_smem(gemm_tcgen05_kernel<BLOCK_N, I8>, L::kTotal); e != cudaSuccess) return (int)e;
  CUtensorMap tmV, tmU;
  const CUtensorMapDataType dt = I8 ? CU_TENSOR_MAP_DATA_TYPE_UINT8 : CU_TENSOR_MAP_DATA_TYPE_FLOAT16;
  constexpr int esize = I8 ? 1 : 2;
  constexpr int BLOCK_K = kRowBytes / esize;
  if (!make_map_3d(&tmV, dt, esize, V, C, pc, (long long)pc_pad * C, nfreq, BLOCK_K, BLOCK_M) ||
      !make_map_3d(&tmU, dt, esize, U, C, K, (long long)K * C, nfreq, BLOCK_K, BLOCK_N))
    return (int)cudaErrorUnknown;
  const long long pairs = (long long)nfreq * ((pc + BLOCK_M - 1) / BLOCK_M);
  const int grid = (int)(pairs < sms ? pairs : sms);
  // Work order.  Row-block-major re-streams all of U once per row block; that is free while U
  // stays in the L2 (8 MB at C = K = 256) and costs device-memory reads once it does not (52 MB at
  // C = K = 512 with 100 frequencies: 164 MB read per launch).  Frequency-major lets the CTAs that
  // run at the same time share each U tile in the L2, at the price of the row-block hand-over with
  // the neighbouring kernels.  Measured: 93 -> 84 us per step at C = K = 512, no difference at 256,
  // 7 % slower for a layer with K = 64 and 196 row blocks; hence the threshold on the size of U.
  const bool f_major = (size_t)nfreq * K * C * esize > ((size_t)32 << 20);
  // Share (percent) of the row blocks of M stored evict-last: what two thirds of the L2 can hold
  // (measured at C = K = 256, 25 row blocks, M = 210 MB: 116.3 us per step with none, 114.3 us with
  // 40 %, 117.4 us with all).  In frequency-major order every row block is live all the time: all.
  const double m_bytes = 4.0 * nfreq * (double)pc_pad * K;
  int keep_pct = f_major ? 100 : (int)(100.0 * (2.0 / 3.0) * l2_bytes / m_bytes);
  if (keep_pct > 100) keep_pct = 100;
  // V may be dropped from the L2 after its last read when the pieces read are whole 128-byte lines
  const bool drop = ((size_t)C * esize) % kRowBytes == 0 && (reinterpret_cast<uintptr_t>(V) % kRowBytes) == 0;
  const uint8_t* vdrop = drop ? (const uint8_t*)V : (const uint8_t*)nullptr;
  // the wait-profiling variant exists for the half product with 256-wide filter blocks only
  if constexpr (BLOCK_N == 256 && !I8) {
    if (prof) {
      if (cudaError_t e = allow_dynamic_smem(gemm_tcgen05_kernel<BLOCK_N, I8, true>, L::kTotal); e != cudaSuccess) return (int)e;
      // CTAs beyond this launch's grid must read as "did not run"
      if (cudaError_t e = cudaMemsetAsync(prof, 0, sizeof(unsigned long long) * 8 * sms, stream); e != cudaSuccess) return (int)e;
      return (int)launch_overlapped(gemm_tcgen05_kernel<BLOCK_N, I8, true>, grid, kThreads, L::kTotal, stream, tmV, tmU, M,
                                    nfreq, pc, pc_pad, C, K, status, vdrop, f_major ? 1 : 0, keep_pct, prof);
    }
  }
  return (int)launch_overlapped(gemm_tcgen05_kernel<BLOCK_N, I8>, grid, kThreads, L::kTotal, stream, tmV, tmU, M, nfreq,
                                pc, pc_pad, C, K, status, vdrop, f_major ? 1 : 0, keep_pct, (unsigned long long*)nullptr);
}

}  // namespace

int launch_gemm_tcgen05(const nova_plan* plan, const void* V, const void* U, float* M, int nfreq, int pc,
                        int pc_pad, int C, int K, int* status_dev, void* stream, unsigned long long* prof) {
  cudaStream_t s = (cudaStream_t)stream;
  const int sms = plan->sm_count;
  if (K > 128) return launch_n<256, false>(sms, plan->l2_bytes, V, U, M, nfreq, pc, pc_pad, C, K, status_dev, s, prof);
  if (K > 64) return launch_n<128, false>(sms, plan->l2_bytes, V, U, M, nfreq, pc, pc_pad, C, K, status_dev, s);
  return launch_n<64, false>(sms, plan->l2_bytes, V, U, M, nfreq, pc, pc_pad, C, K, status_dev, s);
}

// The int8 product: V [nfreq][pc_pad][C] and U [nfreq][K][C] signed bytes (C a multiple of 16),
// M as int32 in the same [f][K/4][pc_pad][4] layout.
int launch_gemm_tcgen05_i8(const nova_plan* plan, const void* V, const void* U, int32_t* M, int nfreq, int pc,
                           int pc_pad, int C, int K, int* status_dev, void* stream) {
  cudaStream_t s = (cudaStream_t)stream;
  const int sms = plan->sm_count;
  float* Mf = reinterpret_cast<float*>(M);            // the epilogue moves 32-bit words
  if (K > 128) return launch_n<256, true>(sms, plan->l2_bytes, V, U, Mf, nfreq, pc, pc_pad, C, K, status_dev, s);
  if (K > 64) return launch_n<128, true>(sms, plan->l2_bytes, V, U, Mf, nfreq, pc, pc_pad, C, K, status_dev, s);
  return launch_n<64, true>(sms, plan->l2_bytes, V, U, Mf, nfreq, pc, pc_pad, C, K, status_dev, s);
}

}  // namespace nova
