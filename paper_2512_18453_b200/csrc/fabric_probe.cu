// Measurement aid (no counterpart in the paper): how many bytes per second the SMs can move
// to and from the L2 / HBM with the access kinds the convolution kernels use.  The transformed
// input V and the transformed-domain product M of the Winograd pipeline are intermediate tensors
// that cross this path twice each, so its rates - not the HBM or tensor peaks alone - bound the
// un-fused pipeline.  One persistent kernel, one CTA per SM (or fewer), grid-stride over a
// buffer of `bytes`:
//   kind 0  ld.global.v4 by every warp
//   kind 1  st.global.v4 by every warp
//   kind 2  even warps load, odd warps store (each its own half of the index set)
//   kind 3  bulk async copies global -> shared (16 KB pieces, `depth` of them in flight), one issuing thread
//   kind 4  kind 3 plus st.global.v4 from 8 other warps (the product kernel's mix)
//   kind 5  bulk async copies shared -> global (16 KB pieces), one issuing thread per warp
//   kind 6  kind 3 plus kind 5
// Every wait is bounded by the clock; an expired wait sets *status and the kernel drains.
#include <cuda_runtime.h>

#include "nova_internal.h"
#include "sm100.cuh"

namespace nova {
namespace {
using namespace sm100;

constexpr int kPiece = 16384;       // bytes per bulk copy
constexpr int kRing = 12;           // shared-memory slots; `depth` <= kRing of them are used
constexpr int kProbeThreads = 320;  // warp 0 issues bulk loads, warp 1 idles, warps 2..9 load/store

__device__ __forceinline__ void bulk_g2s(void* dst, const void* src, uint32_t bytes, uint64_t* bar) {
  asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
               ::"r"(smem_u32(dst)), "l"(src), "r"(bytes), "r"(smem_u32(bar))
               : "memory");
}
__device__ __forceinline__ void bulk_s2g(void* dst, const void* src, uint32_t bytes) {
  asm volatile("cp.async.bulk.global.shared::cta.bulk_group [%0], [%1], %2;" ::"l"(dst), "r"(smem_u32(src)), "r"(bytes)
               : "memory");
}

__global__ void __launch_bounds__(kProbeThreads, 1)
fabric_probe_kernel(const uint4* __restrict__ src, uint4* __restrict__ dst, size_t bytes, int kind, int iters, int depth,
                    int* __restrict__ status, uint4* __restrict__ sink) {
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
  uint64_t* full = reinterpret_cast<uint64_t*>(smem + (kRing + 1) * kPiece);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(full + kRing);
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  if (threadIdx.x == 0) {
    for (int s = 0; s < kRing; ++s) mbar_init(&full[s], 1);
    *abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  // the source of the shared -> global copies: any initialised bytes
  for (int i = threadIdx.x; i < kPiece / 4; i += blockDim.x) reinterpret_cast<uint32_t*>(smem + kRing * kPiece)[i] = i;
  asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  __syncthreads();

  const size_t n16 = bytes / 16;
  const size_t pieces = bytes / kPiece;
  bool timed_out = false;
  const bool bulk_load = kind == 3 || kind == 4 || kind == 6;
  const bool bulk_store = kind == 5 || kind == 6;
  uint4 acc = make_uint4(0, 0, 0, 0);

  if (warp == 0) {
    if (bulk_load) {
      // ring of kRing pieces; the data is dropped (the next copy overwrites it once its barrier fired)
      uint32_t stage = 0, phase = 0;
      uint32_t issued = 0;
      for (int it = 0; it < iters && !timed_out; ++it)
        for (size_t p = blockIdx.x; p < pieces; p += gridDim.x) {
          if (issued >= (uint32_t)depth) {
            if (!mbar_wait(&full[stage], phase, abort_flag)) { timed_out = true; break; }
            if (stage == depth - 1) phase ^= 1;
          }
          // `stage` was just drained (or never used): refill it
          if (lane == 0) {
            mbar_expect_tx(&full[stage], kPiece);
            bulk_g2s(smem + stage * kPiece, reinterpret_cast<const uint8_t*>(src) + p * kPiece, kPiece, &full[stage]);
          }
          __syncwarp();
          ++issued;
          if (++stage == depth) stage = 0;
        }
      // drain what is still in flight
      const uint32_t pending = issued < (uint32_t)depth ? issued : (uint32_t)depth;
      if (issued < (uint32_t)depth) { stage = 0; phase = 0; }   // the ring never wrapped: oldest is slot 0
      for (uint32_t i = 0; i < pending && !timed_out; ++i) {
        if (!mbar_wait(&full[stage], phase, abort_flag)) { timed_out = true; break; }
        if (stage == depth - 1) phase ^= 1;
        if (++stage == depth) stage = 0;
      }
    }
  } else if (warp >= 2) {
    const int w = warp - 2;                       // 0..7
    if (kind <= 2 || kind == 4) {
      const bool loader = kind == 0 || (kind == 2 && (w & 1) == 0);
      const bool storer = kind == 1 || kind == 4 || (kind == 2 && (w & 1) == 1);
      const size_t stride = (size_t)gridDim.x * 256;
      for (int it = 0; it < iters; ++it)
        for (size_t i = (size_t)blockIdx.x * 256 + (threadIdx.x - 64); i < n16; i += stride) {
          if (loader) {
            uint4 v;
            asm volatile("ld.global.cg.v4.u32 {%0,%1,%2,%3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "l"(src + i));
            acc.x ^= v.x; acc.y ^= v.y; acc.z ^= v.z; acc.w ^= v.w;
          }
          if (storer) dst[i] = make_uint4(it, lane, w, 0);
        }
    } else if (bulk_store) {
      for (int it = 0; it < iters; ++it) {
        for (size_t p = (size_t)blockIdx.x * 8 + w; p < pieces; p += (size_t)gridDim.x * 8) {
          if (lane == 0) {
            bulk_s2g(reinterpret_cast<uint8_t*>(dst) + p * kPiece, smem + kRing * kPiece, kPiece);
            bulk_commit();
            bulk_wait_read<2>();
          }
          __syncwarp();
        }
      }
      if (lane == 0) bulk_wait_done<0>();
    }
  }
  if (acc.x == 0x12345678u && acc.y == 0x9abcdef0u) *sink = acc;
  if (timed_out) {
    *abort_flag = 1;
    if (lane == 0) atomicExch(status, NOVA_ERR_DEVICE_TIMEOUT);
  }
}

}  // namespace
}  // namespace nova

extern "C" int nova_probe_fabric(const nova_plan* p, int kind, const void* src_dev, void* dst_dev, size_t bytes,
                                 int iters, int ctas, int depth, float* ms_host, nova_stream stream) {
  using namespace nova;
  if (!p || !src_dev || !dst_dev || !ms_host || kind < 0 || kind > 6 || iters < 1 || iters > 1000 || ctas < 1 || depth < 1 || depth > kRing ||
      bytes < (size_t)kPiece * 8 || (bytes % kPiece) || bytes > ((size_t)8 << 30) ||
      (reinterpret_cast<uintptr_t>(src_dev) & 127) || (reinterpret_cast<uintptr_t>(dst_dev) & 127))
    return NOVA_ERR_INVALID_ARG;
  if (!p->status_dev) return NOVA_ERR_CUDA;
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess || dev != p->device) return NOVA_ERR_INVALID_ARG;
  if (ctas > p->sm_count) ctas = p->sm_count;
  cudaStream_t s = (cudaStream_t)stream;
  const int smem = (kRing + 1) * kPiece + 256 + 1024;
  if (cudaFuncSetAttribute(fabric_probe_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, smem) != cudaSuccess)
    return NOVA_ERR_CUDA;
  uint4* sink = nullptr;
  if (cudaMalloc((void**)&sink, 64) != cudaSuccess) return NOVA_ERR_CUDA;
  cudaEvent_t e0, e1;
  cudaEventCreate(&e0);
  cudaEventCreate(&e1);
  // one untimed pass, then the timed one
  fabric_probe_kernel<<<ctas, kProbeThreads, smem, s>>>((const uint4*)src_dev, (uint4*)dst_dev, bytes, kind, 1, depth,
                                                       p->status_dev, sink);
  cudaEventRecord(e0, s);
  fabric_probe_kernel<<<ctas, kProbeThreads, smem, s>>>((const uint4*)src_dev, (uint4*)dst_dev, bytes, kind, iters, depth,
                                                       p->status_dev, sink);
  cudaEventRecord(e1, s);
  int st = cudaGetLastError() == cudaSuccess && cudaStreamSynchronize(s) == cudaSuccess ? NOVA_OK : NOVA_ERR_CUDA;
  if (st == NOVA_OK) cudaEventElapsedTime(ms_host, e0, e1);
  cudaEventDestroy(e0);
  cudaEventDestroy(e1);
  cudaFree(sink);
  return st;
}
