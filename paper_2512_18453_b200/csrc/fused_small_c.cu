// Section 2.1 steps 2-4 in ONE kernel for layers with 8 input channels (half mode, 3-tap filters):
// V = B^T d B, M[f] = V[f] U[f]^T and Y = A^T M A for a group of 8 tiles at a time, with V and M
// never leaving the SM.  The first layer of an image network is of this kind (3 colour channels
// padded to 8).  There the three-kernel path is bound by its intermediate tensors alone - the
// n*n*K floats of M per tile are 160 times the bytes of the tile's input patch - while the product
// itself is tiny (8 channels), so it fits the register-level tensor-core instruction: one
// mma.sync m16n8k8 per frequency gives M[f] for 8 tiles x 8 filters, the two results a thread
// holds are the same tile's two adjacent filters, i.e. one packed-fp32 operand of the output
// transform, whose n*n inputs per (tile, filter) are consumed row by row and never all alive.
// (The TMEM-accumulator route of the large-C product kernel cannot do this: n*n frequencies x 8
// filters already exceed an SM's 512 accumulator columns.)
//
// One CTA per SM, 12 warps in two roles with their own register budgets (setmaxnreg); the CTA
// keeps the transformed filters of its 64-filter block in shared memory for its whole life and
// walks groups of 8 consecutive tiles:
//   helper warps (4)   TMA: one n x n x 8-channel box per tile straight from x (out-of-range pixels
//                      read as 0: halo and ragged tiles), issued for the next group as soon as
//                      pass 1 has read this one's;
//                      pass 1: B^T along the patch's rows index a, float, to shared memory;
//                      pass 2: B^T along the columns index b, rounded once to half: V (as soon as
//                      the product warps have released the V buffer);
//                      bulk asynchronous copies of the finished image of y to global memory (a
//                      kilobyte per tile row when K = 64), which drain while the next group is computed
//   product warps (8)  warp w owns filters 8w..8w+7: per row xi of frequencies n mma.sync, then
//                      A^T along nu and the accumulation of Y = sum_xi A^T[.][xi] z_xi, all in
//                      registers (packed fp32); Y rounded to half (and ReLU) into a shared-memory
//                      image of the 8 tiles x 64 filters
// The roles meet at mbarriers (V full / free, image full / free), every wait bounded.
// Rounding points are those of the three-kernel path: tables as the plan holds them, V evaluated
// in float and rounded once to half, products of halves summed in float, Y evaluated in float and
// rounded once to half.
#include <cuda_fp16.h>
#include <cuda_runtime.h>

#include "nova_internal.h"
#include "output_math.cuh"
#include "sm100.cuh"
#include "tma_host.h"

namespace nova {
namespace {
using namespace sm100;
using namespace xf;

constexpr int kProductWarps = 8;   // two warpgroups
constexpr int kHelperWarps = 4;    // one warpgroup
constexpr int kStoreLanes = 16;    // lanes per helper warp that issue the copies of y: 64 threads, one per (tile, output row)
constexpr int kThreads = (kProductWarps + kHelperWarps) * 32;
constexpr int kGroupTiles = 8;     // rows 0..7 of the m16n8k8 product (rows 8..15 are fed zeros)
constexpr int kFilterBlock = 64;   // 8 product warps x 8 filters
// Registers per thread after the role split.  The CTA is alone on its SM (shared memory), so the
// register file holds 256 x 216 + 128 x 72 = 64 512 <= 65 536 whatever the kernel was launched with.
constexpr int kProductRegs = 216;
constexpr int kHelperRegs = 72;

// barrier of the helper warps only
__device__ __forceinline__ void helper_sync() { asm volatile("bar.sync 1, %0;" ::"n"(kHelperWarps * 32) : "memory"); }

template <int M>
struct SmallCLayout {
  static constexpr int N = M + 2;
  static constexpr int kPatchBytes = N * N * 16;                        // one tile: [a][b][8 halves]
  static constexpr int kPatchStride = (kPatchBytes + 127) & ~127;       // TMA destinations: 128-byte aligned
  static constexpr int kUBytes = N * kFilterBlock * 4 * N * 4;          // [xi][filter][channel pair][nu] half2
  static constexpr int kVBytes = N * kGroupTiles * 4 * N * 4;           // [xi][tile][channel pair][nu] half2
  static constexpr int kTTile = N * N * 4 * 8 + 32;                     // [xi][b][channel pair] float2 (+32: banks)
  static constexpr int kTBytes = kGroupTiles * kTTile;
  static constexpr int kYTile = M * M * 128 + 16;                       // [i][j][64 filters] half (+16: banks)
  static constexpr int kYBytes = kGroupTiles * kYTile;
  static constexpr int kOffU = 0;
  static constexpr int kOffPatch = kOffU + kUBytes;
  static constexpr int kOffV = kOffPatch + kGroupTiles * kPatchStride;
  static constexpr int kOffT = kOffV + kVBytes;
  static constexpr int kOffY = kOffT + kTBytes;
  static constexpr int kOffBar = (kOffY + kYBytes + 15) & ~15;
  static constexpr int kTotal = kOffBar + 64 + 4 * 16 * kGroupTiles + 128;  // barriers, four sets of tile records, alignment slack
  static_assert(kTotal <= 227 * 1024, "shared memory of one CTA");
};

struct TileRec {          // where a tile's outputs go; rows = 0 for a tile past the end
  long long ybase;        // element offset of pixel (0, 0), filter 0 of the tile
  int rows, cols;
};

__device__ __forceinline__ void bulk_s2g(void* dst, const void* src, uint32_t bytes) {
  asm volatile("cp.async.bulk.global.shared::cta.bulk_group [%0], [%1], %2;" ::"l"(dst), "r"(smem_u32(src)), "r"(bytes)
               : "memory");
}
template <int OFF>
__device__ __forceinline__ uint2 lds_v2(uint32_t saddr) {
  uint2 v;
  asm volatile("ld.shared.v2.b32 {%0, %1}, [%2+%3];" : "=r"(v.x), "=r"(v.y) : "r"(saddr), "n"(OFF));
  return v;
}
#pragma nv_diag_suppress 550
// D[0..7][0..7] = A[0..7][0..7] * B[0..7][0..7] (halves, float sums) on the warp's tensor-core
// path; rows 8..15 of A are zero and their results are dropped.  A thread (g = lane / 4, t = lane
// % 4) passes A[g][2t, 2t+1] and B[2t, 2t+1][g] and receives D[g][2t, 2t+1].
__device__ __forceinline__ float2 mma_8x8x8(uint32_t a, uint32_t b) {
  float d0, d1, d2, d3;                 // d2, d3: rows 8..15, unused
  asm volatile("mma.sync.aligned.m16n8k8.row.col.f32.f16.f16.f32 {%0, %1, %2, %3}, {%4, %5}, {%6}, {%7, %7, %7, %7};"
               : "=f"(d0), "=f"(d1), "=f"(d2), "=f"(d3)
               : "r"(a), "r"(0u), "r"(b), "f"(0.f));
  return make_float2(d0, d1);
}
#pragma nv_diag_default 550

// z_xi[j] = sum_nu A^T[j][nu] * M[xi][nu] with M[xi][nu] made on the spot from the thread's
// operands of V and U in shared memory.
template <int M, bool SYM>
struct ProductRows {
  static constexpr int N = M + 2;
  using L = SmallCLayout<M>;
  const Coefs& cf;
  uint32_t va, ub;          // shared addresses of this thread's words of V and U at xi = 0, nu = 0
  template <int XI>
  __device__ __forceinline__ void row(float2 (&z)[M]) const {
    float2 in[N];
#pragma unroll
    for (int h = 0; h < N / 2; ++h) {
      const uint2 a = lds_v2<XI * (L::kVBytes / N) + 0>(va + h * 8);
      const uint2 b = lds_v2<XI * (L::kUBytes / N) + 0>(ub + h * 8);
      in[2 * h] = mma_8x8x8(a.x, b.x);
      in[2 * h + 1] = mma_8x8x8(a.y, b.y);
    }
    at_apply<M, SYM, float2, N>(cf, in, z);
  }
};

template <int M, bool SYM>
__global__ void __launch_bounds__(kThreads, 1)
fused_small_c_kernel(const __grid_constant__ Coefs cf, const __grid_constant__ CUtensorMap tmX,
                     const uint32_t* __restrict__ U, __half* __restrict__ y, int H, int W, int K, int Th, int Tw,
                     long long P, int num_kb, int relu, int* __restrict__ status) {
  using L = SmallCLayout<M>;
  constexpr int N = L::N;
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 127) & ~(uintptr_t)127);
  uint32_t* Us = reinterpret_cast<uint32_t*>(smem + L::kOffU);
  uint8_t* patch = smem + L::kOffPatch;
  uint8_t* Vs = smem + L::kOffV;
  uint8_t* Ts = smem + L::kOffT;
  uint8_t* Ys = smem + L::kOffY;
  uint64_t* bars = reinterpret_cast<uint64_t*>(smem + L::kOffBar);
  uint64_t* patch_full = bars;       // the group's boxes have landed                     (TMA)
  uint64_t* v_full = bars + 1;       // V of the group is in shared memory                (helper warps)
  uint64_t* v_free = bars + 2;       // the product warps have read V for the last time   (product warps)
  uint64_t* y_full = bars + 3;       // the image of y is complete                        (product warps)
  uint64_t* y_free = bars + 4;       // the copies to global memory have read the image   (storing warps)
  volatile int* abort_flag = reinterpret_cast<volatile int*>(bars + 5);
  volatile int* helper_stop = abort_flag + 1;
  TileRec* rec = reinterpret_cast<TileRec*>(smem + L::kOffBar + 64);         // [4][8]

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int kb = blockIdx.x % num_kb;                       // this CTA's block of 64 filters
  const int cta = blockIdx.x / num_kb, ctas = gridDim.x / num_kb;
  const long long groups = (P + kGroupTiles - 1) / kGroupTiles;

  if (tid == 0) {
    mbar_init(patch_full, 1);
    mbar_init(v_full, kHelperWarps);
    mbar_init(v_free, kProductWarps);
    mbar_init(y_full, kProductWarps);
    mbar_init(y_free, kHelperWarps);
    *abort_flag = 0;
    *helper_stop = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  __syncthreads();
  pdl_launch_dependents();
  pdl_wait();                                               // x and U may come from the preceding kernels

  if (warp < kProductWarps) {
    // ================= product warps: M[f] = V[f] U[f]^T by mma.sync, Y = A^T M A, image of y
    asm volatile("setmaxnreg.inc.sync.aligned.u32 %0;" ::"n"(kProductRegs));
    // U[f][K][8] (internal frequency order) -> Us[xi][filter][channel pair][nu]; filters >= K read as 0.
    // A thread owns one (filter, channel pair) - of its own warp's 8 filters: n loads in flight, then
    // n contiguous words stored, and only the warp itself reads them back.
    {
      const int t = tid & 3, kl = tid >> 2, k = kb * kFilterBlock + kl;
      const uint32_t* src = U + ((size_t)(k < K ? k : 0) * 4 + t);
      uint32_t* dst = Us + (kl * 4 + t) * N;
#pragma unroll 2
      for (int xi = 0; xi < N; ++xi) {
        uint32_t v[N];
#pragma unroll
        for (int nu = 0; nu < N; ++nu) v[nu] = k < K ? __ldg(src + (size_t)(xi * N + nu) * K * 4) : 0u;
#pragma unroll
        for (int nu = 0; nu < N; nu += 2)
          *reinterpret_cast<uint2*>(dst + xi * kFilterBlock * 4 * N + nu) = make_uint2(v[nu], v[nu + 1]);
      }
      __syncwarp();
    }
    const int g = lane >> 2, t = lane & 3;
    const uint32_t va0 = smem_u32(Vs) + (uint32_t)((g * 4 + t) * N * 4);
    const uint32_t ub0 = smem_u32(Us) + (uint32_t)((((warp * 8 + g) * 4) + t) * N * 4);
    const __half2 lo2 = relu ? __half2half2(__ushort_as_half(0)) : __half2half2(__ushort_as_half(0xfc00));   // 0 or -inf
    uint32_t it = 0;
    for (long long grp = cta; grp < groups; grp += ctas, ++it) {
      if (!mbar_poll(v_full, it & 1, abort_flag)) { *abort_flag = 1; break; }
      float2 Y[M][M];
      const ProductRows<M, SYM> rows{cf, va0, ub0};
      accumulate_rows<M, SYM, float2, N>(cf, rows, Y);
      __syncwarp();
      if (lane == 0) mbar_arrive(v_free);
      // the copies of the previous group must have read the image before it is overwritten
      if (!mbar_wait(y_free, (it & 1) ^ 1, abort_flag)) { *abort_flag = 1; break; }
      // rounded to half, then the ReLU (NaN and +inf pass)
      uint8_t* dst = Ys + g * L::kYTile + warp * 16 + t * 4;
#pragma unroll
      for (int i = 0; i < M; ++i)
#pragma unroll
        for (int j = 0; j < M; ++j)
          *reinterpret_cast<__half2*>(dst + (i * M + j) * 128) = __hmax2_nan(__floats2half2_rn(Y[i][j].x, Y[i][j].y), lo2);
      asm volatile("fence.proxy.async.shared::cta;" ::: "memory");     // the bulk copies read these writes
      __syncwarp();
      if (lane == 0) mbar_arrive(y_full);
    }
  } else {
    // ================= helper warps: boxes of x by TMA, V = B^T d B, copies of the image of y to global memory
    asm volatile("setmaxnreg.dec.sync.aligned.u32 %0;" ::"n"(kHelperRegs));
    const int ht = tid - kProductWarps * 32;                 // 0 .. 127
    const int k_here = min(kFilterBlock, K - kb * kFilterBlock);      // filters of this block that exist
    // Lanes 0 and 1 of every helper warp, one tile each (tile 2 hw + lane of the group): the tile's box
    // into the patch buffer and its output record into record set `set`.  Tiles past the end are not
    // fetched and get an empty record.  (Eight lanes of one warp took 1 500 cycles over it, on the
    // critical path of that warp.)
    const int hw = warp - kProductWarps;
    auto fetch = [&](long long grp, int set) {
      if (lane >= kGroupTiles / kHelperWarps) return;
      const int tl = hw * (kGroupTiles / kHelperWarps) + lane;
      const long long p0 = grp * kGroupTiles;
      if (tl == 0) {
        const int live = (int)((P - p0) < kGroupTiles ? (P - p0) : kGroupTiles);
        mbar_expect_tx(patch_full, (uint32_t)live * L::kPatchBytes);
      }
      TileRec r = {0, 0, 0};
      if (p0 + tl < P) {
        const uint32_t p = (uint32_t)(p0 + tl);               // the launcher keeps P below 2^31
        const uint32_t tw = p % (uint32_t)Tw, q = p / (uint32_t)Tw, th = q % (uint32_t)Th, img = q / (uint32_t)Th;
        tma_load_4d(patch + tl * L::kPatchStride, &tmX, patch_full, 0, (int)(M * tw) - 1, (int)(M * th) - 1, (int)img);
        r.ybase = (((long long)img * H + M * th) * W + M * tw) * K + (long long)kb * kFilterBlock;
        r.rows = min(M, H - (int)(M * th));
        r.cols = min(M, W - (int)(M * tw));
      }
      rec[set * kGroupTiles + tl] = r;
    };
    // The first kStoreLanes lanes of every helper warp, one thread per (tile, output row) of group
    // number `n` of this CTA: bulk copies shared -> global.  A full-width row of a 64-filter layer is
    // one contiguous kilobyte; otherwise one copy per pixel.  (A warp issues such copies lane after
    // lane, some 85 cycles each: hence four warps.)  store_release, a good thousand cycles later, finds
    // the copies' reads of the image complete and hands the image back to the product warps.
    const int st = lane < kStoreLanes ? hw * kStoreLanes + lane : kGroupTiles * M;
    auto store_issue = [&](uint32_t n) {
      const bool ok = mbar_wait(y_full, n & 1, abort_flag);
      if (!ok) *abort_flag = 1;
      if (ok && st < kGroupTiles * M) {
        const int tl = st / M, i = st % M;
        const TileRec r = rec[(n & 3) * kGroupTiles + tl];
        if (i < r.rows) {
          __half* dst = y + r.ybase + (long long)i * W * K;
          const uint8_t* src = Ys + tl * L::kYTile + i * M * 128;
          if (K == kFilterBlock && r.cols == M) {
            bulk_s2g(dst, src, M * 128);
          } else {
            for (int j = 0; j < r.cols; ++j) bulk_s2g(dst + (long long)j * K, src + j * 128, (uint32_t)k_here * 2);
          }
          bulk_commit();
        }
      }
    };
    auto store_release = [&]() {
      bulk_wait_read<0>();
      __syncwarp();
      if (lane == 0) mbar_arrive(y_free);
    };
    if (cta < groups) fetch(cta, 0);
    uint32_t it = 0;
    for (long long grp = cta; grp < groups; grp += ctas, ++it) {
      if (!mbar_wait(patch_full, it & 1, abort_flag)) *abort_flag = 1;
      // ---- pass 1: T[tile][xi][b][cp] = sum_a B^T[xi][a] d[a][b]
      for (int item = ht; item < kGroupTiles * N * 4; item += kHelperWarps * 32) {
        const int cp = item & 3, b = (item >> 2) % N, tl = item / (4 * N);
        const uint8_t* src = patch + tl * L::kPatchStride + b * 16 + cp * 4;
        float2 d[N], o[N];
#pragma unroll
        for (int a = 0; a < N; ++a) d[a] = __half22float2(*reinterpret_cast<const __half2*>(src + a * N * 16));
        bt_all_rows<N, SYM>(cf, d, o);
        float2* dst = reinterpret_cast<float2*>(Ts + tl * L::kTTile) + b * 4 + cp;
#pragma unroll
        for (int xi = 0; xi < N; ++xi) dst[xi * N * 4] = o[xi];
      }
      // One thread samples the abort flag before the barrier and every helper reads that sample
      // after it: the helpers leave the loop together or not at all (a flag read by each thread
      // for itself could change between two reads and strand the others at the next barrier).
      if (ht == 0) *helper_stop = *abort_flag;
      helper_sync();                 // T is complete and the patch buffer is free
      if (*helper_stop) break;
      if (grp + ctas < groups) fetch(grp + ctas, (it + 1) & 3);
      if (it > 1) store_release();   // the copies of group it - 2, issued one iteration ago
      if (!mbar_poll(v_free, (it & 1) ^ 1, abort_flag)) *abort_flag = 1;   // on the critical path
      // ---- pass 2: V[xi][nu] = sum_b T[xi][b] B^T[nu][b], rounded to half
      for (int item = ht; item < kGroupTiles * N * 4; item += kHelperWarps * 32) {
        const int cp = item & 3, tl = (item >> 2) & (kGroupTiles - 1), xi = item >> 5;
        const float2* src = reinterpret_cast<const float2*>(Ts + tl * L::kTTile) + xi * N * 4 + cp;
        float2 d[N], o[N];
#pragma unroll
        for (int b = 0; b < N; ++b) d[b] = src[b * 4];
        bt_all_rows<N, SYM>(cf, d, o);
        uint32_t* dst = reinterpret_cast<uint32_t*>(Vs) + ((xi * kGroupTiles + tl) * 4 + cp) * N;
#pragma unroll
        for (int nu = 0; nu < N; nu += 2) {
          const __half2 h0 = __floats2half2_rn(o[nu].x, o[nu].y), h1 = __floats2half2_rn(o[nu + 1].x, o[nu + 1].y);
          *reinterpret_cast<uint2*>(dst + nu) =
              make_uint2(*reinterpret_cast<const uint32_t*>(&h0), *reinterpret_cast<const uint32_t*>(&h1));
        }
      }
      __syncwarp();
      if (lane == 0) mbar_arrive(v_full);
      if (it > 0) store_issue(it - 1);
      helper_sync();                 // T may be overwritten
    }
    if (!*abort_flag) {
      if (it > 1) store_release();
      if (it > 0) { store_issue(it - 1); store_release(); }
    }
    bulk_wait_read<0>();
  }
  if (*abort_flag && lane == 0) atomicExch(status, NOVA_ERR_DEVICE_TIMEOUT);
}

template <int M, bool SYM>
int go(const nova_plan* plan, const Geom& g, const void* x, const void* U, void* y, int relu, cudaStream_t stream) {
  using L = SmallCLayout<M>;
  EncodeTiledFn enc = tensor_map_encoder();
  if (!enc) return (int)cudaErrorUnknown;
  CUtensorMap tmX;
  cuuint64_t dims[4] = {8, (cuuint64_t)g.W, (cuuint64_t)g.H, (cuuint64_t)g.N};
  cuuint64_t strides[3] = {16, (cuuint64_t)g.W * 16, (cuuint64_t)g.H * g.W * 16};
  cuuint32_t box[4] = {8, (cuuint32_t)L::N, (cuuint32_t)L::N, 1};
  cuuint32_t estr[4] = {1, 1, 1, 1};
  if (enc(&tmX, CU_TENSOR_MAP_DATA_TYPE_FLOAT16, 4, const_cast<void*>(x), dims, strides, box, estr,
          CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
          CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
    return (int)cudaErrorUnknown;
  if (cudaError_t e = allow_dynamic_smem(fused_small_c_kernel<M, SYM>, L::kTotal); e != cudaSuccess) return (int)e;
  const int num_kb = (g.K + kFilterBlock - 1) / kFilterBlock;
  const long long groups = (g.P + kGroupTiles - 1) / kGroupTiles;
  long long per_kb = plan->sm_count / num_kb;
  if (per_kb < 1) per_kb = 1;
  if (per_kb > groups) per_kb = groups;
  return (int)launch_overlapped(fused_small_c_kernel<M, SYM>, (int)(per_kb * num_kb), kThreads, L::kTotal, stream,
                                plan->kcoefs, tmX, (const uint32_t*)U, (__half*)y, g.H, g.W, g.K, g.Th, g.Tw, g.P, num_kb,
                                relu, plan->status_dev);
}

}  // namespace

// x, U and y are 16-byte aligned and K is a multiple of 8 on every path that reaches the launcher.
// Tile indices are 32-bit in the kernel: larger problems stay on the three-kernel path.
bool fused_small_c_applies(const nova_plan* plan, const Geom& g) {
  return plan->mode == NOVA_FP16_F32ACC && plan->r == 3 && g.C == 8 && plan->status_dev != nullptr &&
         g.P < ((long long)1 << 31) - kGroupTiles;
}

int launch_fused_small_c(const nova_plan* plan, const Geom& g, const void* x, const void* U, void* y, int relu,
                         void* stream) {
  cudaStream_t s = (cudaStream_t)stream;
#define NOVA_SMALLC(MV)                                                       \
  return plan->symmetric ? go<MV, true>(plan, g, x, U, y, relu, s) : go<MV, false>(plan, g, x, U, y, relu, s)
  switch (plan->m) {
    case 2: NOVA_SMALLC(2);
    case 4: NOVA_SMALLC(4);
    case 6: NOVA_SMALLC(6);
    case 8: NOVA_SMALLC(8);
  }
#undef NOVA_SMALLC
  return (int)cudaErrorInvalidValue;
}

}  // namespace nova
