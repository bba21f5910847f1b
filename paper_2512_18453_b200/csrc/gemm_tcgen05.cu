// Transformed-domain product on the sm_100a tensor cores (Section 2.1 step 3
// summed over input channels): for every frequency f,
//   M[f][p][k] = sum_c V[f][p][c] * U[f][k][c],   half x half -> float.
//
// Persistent, warp-specialised kernel.  One CTA per SM walks a list of work
// items (f, 128-row block of tiles p, BLOCK_N-wide block of filters k):
//   warp 0    TMA producer: 128B-swizzled [rows][64 channels] boxes of V and U
//             into a 4-stage shared-memory ring, completion on mbarriers;
//   warp 1    issues tcgen05.mma (kind::f16, M=128, N=BLOCK_N, K=16) from
//             shared-memory descriptors into one of two TMEM accumulators;
//   warps 2-5 epilogue: tcgen05.ld the finished accumulator (one TMEM lane
//             quadrant per warp), stage it in swizzled shared memory and TMA-
//             store float boxes of M, overlapping the next item's MMAs on the
//             other accumulator.
// Every wait is bounded; on expiry the kernel records a status and drains.
#include <cuda.h>
#include <cuda_fp16.h>
#include <cuda_runtime.h>

#include "nova_internal.h"

namespace nova {
namespace {

constexpr int BLOCK_M = 128;
constexpr int BLOCK_K = 64;            // 64 halves = 128 bytes = one swizzle row
constexpr int UMMA_K = 16;
constexpr int kStages = 4;
constexpr int kThreads = 192;
constexpr uint32_t kSpinLimit = 1u << 24;

__device__ __forceinline__ uint32_t smem_u32(const void* p) {
  return (uint32_t)__cvta_generic_to_shared(p);
}
__device__ __forceinline__ void mbar_init(uint64_t* bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count));
}
__device__ __forceinline__ void mbar_expect_tx(uint64_t* bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(bar)), "r"(bytes)
               : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint64_t* bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(bar)) : "memory");
}
__device__ __forceinline__ bool mbar_test(uint64_t* bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.test_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok)
      : "r"(smem_u32(bar)), "r"(parity)
      : "memory");
  return ok != 0;
}
// Bounded wait.  Returns false if the limit is hit or another role gave up.
__device__ __forceinline__ bool mbar_wait(uint64_t* bar, uint32_t parity, volatile int* abort_flag) {
  for (uint32_t spin = 0; spin < kSpinLimit; ++spin) {
    if (mbar_test(bar, parity)) return true;
    if ((spin & 63u) == 63u && *abort_flag) return false;
  }
  return false;
}

__device__ __forceinline__ void tma_load_3d(void* dst, const CUtensorMap* map, uint64_t* bar, int x,
                                            int y, int z) {
  asm volatile(
      "cp.async.bulk.tensor.3d.shared::cluster.global.tile.mbarrier::complete_tx::bytes"
      " [%0], [%1, {%3, %4, %5}], [%2];"
      ::"r"(smem_u32(dst)), "l"(map), "r"(smem_u32(bar)), "r"(x), "r"(y), "r"(z)
      : "memory");
}

__device__ __forceinline__ void tma_store_3d(const CUtensorMap* map, const void* src, int x, int y, int z) {
  asm volatile("cp.async.bulk.tensor.3d.global.shared::cta.bulk_group [%0, {%2, %3, %4}], [%1];"
               ::"l"(map), "r"(smem_u32(src)), "r"(x), "r"(y), "r"(z)
               : "memory");
}
__device__ __forceinline__ void bulk_commit() { asm volatile("cp.async.bulk.commit_group;" ::: "memory"); }
template <int N>
__device__ __forceinline__ void bulk_wait_read() {
  asm volatile("cp.async.bulk.wait_group.read %0;" ::"n"(N) : "memory");
}
__device__ __forceinline__ void bulk_wait_all() { asm volatile("cp.async.bulk.wait_group 0;" ::: "memory"); }

// Shared-memory matrix descriptor for a K-major operand tile stored as
// [rows][64 halves] with the 128-byte swizzle: 8-row groups are 1024 bytes
// apart (stride byte offset), descriptor version 1, layout type 2.
__device__ __forceinline__ uint64_t umma_desc_sw128(uint32_t saddr) {
  uint64_t d = 0;
  d |= (uint64_t)((saddr & 0x3FFFFu) >> 4);
  d |= (uint64_t)1 << 16;                 // leading byte offset: unused for swizzled K-major
  d |= (uint64_t)(1024 >> 4) << 32;       // stride byte offset
  d |= (uint64_t)1 << 46;                 // descriptor version (sm_100)
  d |= (uint64_t)2 << 61;                 // SWIZZLE_128B
  return d;
}
// Instruction descriptor, kind::f16: D float, A and B half, both K-major.
__host__ __device__ constexpr uint32_t umma_idesc_f16(int M, int N) {
  return (1u << 4) | (0u << 7) | (0u << 10) | (0u << 15) | (0u << 16) | ((uint32_t)(N >> 3) << 17) |
         ((uint32_t)(M >> 4) << 24);
}
__device__ __forceinline__ void umma_f16(uint32_t tmem_d, uint64_t adesc, uint64_t bdesc, uint32_t idesc,
                                         uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
      ::"r"(tmem_d), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate)
      : "memory");
}
__device__ __forceinline__ void umma_commit(uint64_t* bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(
                   smem_u32(bar))
               : "memory");
}
__device__ __forceinline__ void tmem_ld32(uint32_t taddr, uint32_t (&r)[32]) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
      "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
      "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
        "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]),
        "=r"(r[15]), "=r"(r[16]), "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]),
        "=r"(r[22]), "=r"(r[23]), "=r"(r[24]), "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]),
        "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
      : "r"(taddr)
      : "memory");
}

template <int BLOCK_N>
struct SmemLayout {
  static constexpr int kABytes = BLOCK_M * BLOCK_K * 2;
  static constexpr int kBBytes = BLOCK_N * BLOCK_K * 2;
  static constexpr int kStageBytes = kABytes + kBBytes;
  static constexpr int kOutOffset = kStages * kStageBytes;        // epilogue staging
  static constexpr int kOutBytesPerWarp = 2 * 32 * 128;           // two [32 rows][32 floats] boxes
  static constexpr int kBarrierOffset = kOutOffset + 4 * kOutBytesPerWarp;
  static constexpr int kTotal = kBarrierOffset + 256 + 1024;     // barriers + alignment slack
};

template <int BLOCK_N>
__global__ void __launch_bounds__(kThreads, 1)
gemm_tcgen05_kernel(const __grid_constant__ CUtensorMap tmV, const __grid_constant__ CUtensorMap tmU,
                    const __grid_constant__ CUtensorMap tmM, int nfreq, int pc, int C, int K,
                    int* __restrict__ status) {
  using L = SmemLayout<BLOCK_N>;
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
  const long long num_items = (long long)nfreq * num_pb * num_kb;

  if (threadIdx.x == 0) {
    for (int s = 0; s < kStages; ++s) { mbar_init(&full_bar[s], 1); mbar_init(&empty_bar[s], 1); }
    for (int a = 0; a < 2; ++a) { mbar_init(&tmem_full[a], 1); mbar_init(&tmem_empty[a], 4); }
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

  if (warp == 0) {
    // ---------------- TMA producer
    uint32_t stage = 0, phase = 0;
    for (long long it = blockIdx.x; it < num_items && !timed_out; it += gridDim.x) {
      const int kb = (int)(it % num_kb);
      const int pb = (int)((it / num_kb) % num_pb);
      const int f = (int)(it / ((long long)num_kb * num_pb));
      for (int ks = 0; ks < num_ks; ++ks) {
        if (!mbar_wait(&empty_bar[stage], phase ^ 1, abort_flag)) { timed_out = true; break; }
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
  } else if (warp == 1) {
    // ---------------- MMA issuer
    constexpr uint32_t idesc = umma_idesc_f16(BLOCK_M, BLOCK_N);
    uint32_t stage = 0, phase = 0, local = 0;
    for (long long it = blockIdx.x; it < num_items && !timed_out; it += gridDim.x, ++local) {
      const uint32_t acc = local & 1, acc_phase = (local >> 1) & 1;
      if (!mbar_wait(&tmem_empty[acc], acc_phase ^ 1, abort_flag)) { timed_out = true; break; }
      asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
      const uint32_t tmem_d = tmem_base + acc * BLOCK_N;
      for (int ks = 0; ks < num_ks; ++ks) {
        if (!mbar_wait(&full_bar[stage], phase, abort_flag)) { timed_out = true; break; }
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
        if (lane == 0) {
          const uint32_t sa = smem_u32(smem + stage * L::kStageBytes);
          const uint32_t sb = sa + L::kABytes;
#pragma unroll
          for (int k = 0; k < BLOCK_K / UMMA_K; ++k) {
            const uint64_t ad = umma_desc_sw128(sa + k * UMMA_K * 2);
            const uint64_t bd = umma_desc_sw128(sb + k * UMMA_K * 2);
            umma_f16(tmem_d, ad, bd, idesc, (ks > 0 || k > 0) ? 1u : 0u);
          }
          umma_commit(&empty_bar[stage]);                 // frees the smem stage when the MMAs retire
          if (ks == num_ks - 1) umma_commit(&tmem_full[acc]);
        }
        __syncwarp();
        if (++stage == kStages) { stage = 0; phase ^= 1; }
      }
    }
  } else {
    // ---------------- epilogue (warps 2..5); a warp may only read TMEM lanes 32*(warp%4)..+31.
    // Each warp moves its 32 rows in [32 rows][32 floats] boxes: TMEM -> registers ->
    // 128B-swizzled shared memory -> TMA store (which clips rows >= pc and columns >= K).
    const int quad = warp & 3;
    uint8_t* stage_out = smem + L::kOutOffset + (warp - 2) * L::kOutBytesPerWarp;
    uint32_t local = 0, nbox = 0;
    for (long long it = blockIdx.x; it < num_items && !timed_out; it += gridDim.x, ++local) {
      const int kb = (int)(it % num_kb);
      const int pb = (int)((it / num_kb) % num_pb);
      const int f = (int)(it / ((long long)num_kb * num_pb));
      const uint32_t acc = local & 1, acc_phase = (local >> 1) & 1;
      if (!mbar_wait(&tmem_full[acc], acc_phase, abort_flag)) { timed_out = true; break; }
      asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
      const int row0 = pb * BLOCK_M + quad * 32;
      const int k_left = K - kb * BLOCK_N;
#pragma unroll 1
      for (int cb = 0; cb < BLOCK_N && cb < k_left; cb += 32, ++nbox) {
        uint8_t* buf = stage_out + (nbox & 1) * (32 * 128);
        if (lane == 0) bulk_wait_read<1>();          // the store that last read this buffer is done
        __syncwarp();
        uint32_t r[32];
        tmem_ld32(tmem_base + ((uint32_t)(quad * 32) << 16) + acc * BLOCK_N + cb, r);
        asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
        uint8_t* my_row = buf + lane * 128;
#pragma unroll
        for (int j = 0; j < 8; ++j)                  // 16-byte chunk j of row `lane` lives at chunk j ^ (lane & 7)
          *reinterpret_cast<uint4*>(my_row + ((j ^ (lane & 7)) << 4)) =
              make_uint4(r[4 * j], r[4 * j + 1], r[4 * j + 2], r[4 * j + 3]);
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
        __syncwarp();
        if (lane == 0) {
          if (row0 < pc) tma_store_3d(&tmM, buf, kb * BLOCK_N + cb, row0, f);
          bulk_commit();   // one group per box, stored or not, so "at most one pending" always means the other buffer
        }
      }
      asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
      __syncwarp();
      if (lane == 0) mbar_arrive(&tmem_empty[acc]);
    }
    if (lane == 0) bulk_wait_all();
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

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*,
                                  CUtensorMapInterleave, CUtensorMapSwizzle, CUtensorMapL2promotion,
                                  CUtensorMapFloatOOBfill);

EncodeTiledFn get_encode_fn() {
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

// [nfreq][rows][inner] elements of `esize` bytes, frequency stride in elements;
// box = [1][box_rows][box_inner], 128-byte swizzle (box_inner * esize == 128).
bool make_map_3d(CUtensorMap* map, CUtensorMapDataType dt, int esize, const void* base, int inner, int rows,
                 long long freq_stride_elems, int nfreq, int box_inner, int box_rows) {
  EncodeTiledFn enc = get_encode_fn();
  if (!enc) return false;
  cuuint64_t dims[3] = {(cuuint64_t)inner, (cuuint64_t)rows, (cuuint64_t)nfreq};
  cuuint64_t strides[2] = {(cuuint64_t)inner * esize, (cuuint64_t)freq_stride_elems * esize};
  cuuint32_t box[3] = {(cuuint32_t)box_inner, (cuuint32_t)box_rows, 1};
  cuuint32_t estr[3] = {1, 1, 1};
  return enc(map, dt, 3, const_cast<void*>(base), dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
             CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
             CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

template <int BLOCK_N>
int launch_n(const void* V, const void* U, float* M, int nfreq, int pc, int pc_pad, int C, int K,
             int* status, cudaStream_t stream) {
  using L = SmemLayout<BLOCK_N>;
  static bool attr_set = false;
  if (!attr_set) {
    cudaError_t e = cudaFuncSetAttribute(gemm_tcgen05_kernel<BLOCK_N>,
                                         cudaFuncAttributeMaxDynamicSharedMemorySize, L::kTotal);
    if (e != cudaSuccess) return (int)e;
    attr_set = true;
  }
  CUtensorMap tmV, tmU, tmM;
  const CUtensorMapDataType f16 = CU_TENSOR_MAP_DATA_TYPE_FLOAT16, f32 = CU_TENSOR_MAP_DATA_TYPE_FLOAT32;
  if (!make_map_3d(&tmV, f16, 2, V, C, pc, (long long)pc_pad * C, nfreq, BLOCK_K, BLOCK_M) ||
      !make_map_3d(&tmU, f16, 2, U, C, K, (long long)K * C, nfreq, BLOCK_K, BLOCK_N) ||
      !make_map_3d(&tmM, f32, 4, M, K, pc, (long long)pc_pad * K, nfreq, 32, 32))
    return (int)cudaErrorUnknown;
  int dev = 0, sms = 0;
  cudaGetDevice(&dev);
  cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
  const long long items = (long long)nfreq * ((pc + BLOCK_M - 1) / BLOCK_M) * ((K + BLOCK_N - 1) / BLOCK_N);
  const int grid = (int)(items < sms ? items : sms);
  gemm_tcgen05_kernel<BLOCK_N><<<grid, kThreads, L::kTotal, stream>>>(tmV, tmU, tmM, nfreq, pc, C, K, status);
  return (int)cudaGetLastError();
}

}  // namespace

int launch_gemm_tcgen05(const nova_plan* plan, const void* V, const void* U, float* M, int nfreq, int pc,
                        int pc_pad, int C, int K, int* status_dev, void* stream) {
  (void)plan;
  cudaStream_t s = (cudaStream_t)stream;
  if (K > 128) return launch_n<256>(V, U, M, nfreq, pc, pc_pad, C, K, status_dev, s);
  if (K > 64) return launch_n<128>(V, U, M, nfreq, pc, pc_pad, C, K, status_dev, s);
  return launch_n<64>(V, U, M, nfreq, pc, pc_pad, C, K, status_dev, s);
}

}  // namespace nova
