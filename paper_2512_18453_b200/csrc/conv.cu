// Host orchestration of the forward convolution and the remaining C ABI.
//
// The tiles of a problem are processed in chunks sized so that the transformed
// input V (operand type) and the transformed-domain product M (float) of one
// chunk fit the caller's scratch: input transform -> product -> output
// transform per chunk, all on the caller's stream, no host synchronisation.
#include <cuda_runtime.h>

#include <mutex>

#include "nova_internal.h"
#include "sm100.cuh"

namespace nova {
namespace {

constexpr size_t kAlign = 256;
constexpr size_t kTargetChunkBytes = (size_t)1 << 30;   // one chunk unless the problem is huge: fewest launches
inline size_t round_up(size_t v, size_t a) { return (v + a - 1) / a * a; }

struct Chunking {
  int pc;            // tiles per chunk
  int pc_pad;        // row stride of V and M inside the workspace
  int chunks;
  size_t v_bytes, m_bytes;
};

size_t per_tile_bytes(const nova_plan* p, const Geom& g) {
  return (size_t)g.n * g.n * ((size_t)g.C * elt_bytes(p->mode) + (size_t)g.K * 4);
}
inline long long round_up_ll(long long v, long long a) { return (v + a - 1) / a * a; }

// Largest chunk, a whole number of 128-tile row blocks, that fits `bytes`.  The scratch rows
// are padded to that multiple: the product kernel writes whole row blocks of M.
bool choose_chunking(const nova_plan* p, const Geom& g, size_t bytes, Chunking* c) {
  const size_t pt = per_tile_bytes(p, g);
  if (bytes < 2 * kAlign + 128 * pt) return false;
  long long pc = (long long)((bytes - 2 * kAlign) / pt) / 128 * 128;
  const long long p_pad = round_up_ll(g.P, 128);
  if (pc > p_pad) pc = p_pad;
  if (pc < 128) return false;
  c->pc = (int)(pc < g.P ? pc : g.P);
  c->pc_pad = (int)pc;
  c->chunks = (int)((g.P + pc - 1) / pc);
  c->v_bytes = round_up((size_t)g.n * g.n * c->pc_pad * g.C * elt_bytes(p->mode), kAlign);
  c->m_bytes = round_up((size_t)g.n * g.n * c->pc_pad * g.K * 4, kAlign);
  return c->v_bytes + c->m_bytes <= bytes;
}

// 3 x 3 filters and 5 x 5 filters (F(2,5), F(4,5), F(6,5)) run the same kernels, instantiated
// for n = m + 2 and n = m + 4.
bool device_plan(const nova_plan* p) { return p && (p->r == kR || p->r == 5); }
bool shape_ok(int N, int H, int W, int C, int K) {
  return N > 0 && H > 0 && W > 0 && C > 0 && K > 0 && (C % 8) == 0 && (K % 8) == 0;
}
bool aligned16(const void* p) { return p && (reinterpret_cast<uintptr_t>(p) & 15) == 0; }

// The plan's status word, its tables and the built-in scratch belong to one device: the device
// entry points refuse to run with another one current.
bool on_plan_device(const nova_plan* p) {
  int dev = -1;
  return p->device >= 0 && cudaGetDevice(&dev) == cudaSuccess && dev == p->device;
}

// The one-kernel path for 8 input channels runs unless a flag asks for a particular kernel of the
// three-kernel path.
bool use_fused_small_c(const nova_plan* p, const Geom& g, int flags) {
  const int forcing = NOVA_GEMM_SIMT | NOVA_GEMM_TCGEN05 | NOVA_TRANSFORM_SIMT | NOVA_PROFILE_WAITS | NOVA_POOL2X2;
  return (flags & forcing) == 0 && fused_small_c_applies(p, g);
}

bool use_tcgen05(const nova_plan* p, int flags) {
  if (p->mode == NOVA_FP32) return false;
  return (flags & NOVA_GEMM_SIMT) == 0;
}

}  // namespace
}  // namespace nova

using namespace nova;

extern "C" size_t nova_filter_transform_bytes(const nova_plan* p, int K, int C) {
  if (!device_plan(p) || K <= 0 || C <= 0) return 0;
  return (size_t)p->n * p->n * K * C * elt_bytes(p->mode);
}

extern "C" int nova_filter_transform(const nova_plan* p, const void* g, int K, int C, void* U,
                                     nova_stream stream) {
  if (!p || !aligned16(g) || !aligned16(U) || K <= 0 || C <= 0 || (K % 8) || (C % 8))
    return NOVA_ERR_INVALID_ARG;
  if (!device_plan(p)) return NOVA_ERR_UNSUPPORTED;
  if (p->device < 0) return NOVA_ERR_CUDA;
  if (!on_plan_device(p)) return NOVA_ERR_INVALID_ARG;
  const int e = p->mode == NOVA_FP32 ? launch_filter_transform_f32(p, g, K, C, U, stream)
                                     : launch_filter_transform(p, g, K, C, U, stream);
  return e == 0 ? NOVA_OK : NOVA_ERR_CUDA;
}

extern "C" size_t nova_conv2d_min_workspace_bytes(const nova_plan* p, int N, int H, int W, int C, int K) {
  if (!device_plan(p) || !shape_ok(N, H, W, C, K)) return 0;
  Geom g = make_geom(p, N, H, W, C, K);
  return (size_t)128 * per_tile_bytes(p, g) + 4 * kAlign;
}

extern "C" size_t nova_conv2d_workspace_bytes(const nova_plan* p, int N, int H, int W, int C, int K) {
  if (!device_plan(p) || !shape_ok(N, H, W, C, K)) return 0;
  Geom g = make_geom(p, N, H, W, C, K);
  const size_t pt = per_tile_bytes(p, g);
  long long pc = (long long)(kTargetChunkBytes / pt) / 128 * 128;
  if (pc < 128) pc = 128;
  if (pc > round_up_ll(g.P, 128)) pc = round_up_ll(g.P, 128);
  return (size_t)pc * pt + 4 * kAlign;
}

extern "C" int nova_conv2d_launch_count(const nova_plan* p, int N, int H, int W, int C, int K,
                                        size_t workspace_bytes, int flags) {
  if (!p || !shape_ok(N, H, W, C, K)) return NOVA_ERR_INVALID_ARG;
  if (!device_plan(p)) return NOVA_ERR_UNSUPPORTED;
  Geom g = make_geom(p, N, H, W, C, K);
  Chunking c;
  if (!choose_chunking(p, g, workspace_bytes, &c)) return NOVA_ERR_WORKSPACE;
  if (use_fused_small_c(p, g, flags)) return 1;
  return 3 * c.chunks;
}

namespace {
int g_last_cuda_error = 0;          // raw code of the last failed CUDA call on the convolution path
// Shared body of nova_conv2d_fwd and nova_conv2d_fwd_timed.  With `ev` non-null,
// four events per chunk bracket the three kernels.
int conv2d_fwd_impl(const nova_plan* p, const void* x, const void* U, void* y, int N, int H, int W, int C,
                    int K, void* ws, size_t ws_bytes, int flags, nova_stream stream, cudaEvent_t* ev) {
  if (!p || !aligned16(x) || !aligned16(U) || !aligned16(y) || !shape_ok(N, H, W, C, K))
    return NOVA_ERR_INVALID_ARG;
  if (!device_plan(p)) return NOVA_ERR_UNSUPPORTED;
  if (!ws || (reinterpret_cast<uintptr_t>(ws) % kAlign)) return NOVA_ERR_WORKSPACE;
  if ((flags & NOVA_GEMM_TCGEN05) && p->mode == NOVA_FP32) return NOVA_ERR_UNSUPPORTED;
  if (p->device < 0) return NOVA_ERR_CUDA;
  if (!on_plan_device(p)) return NOVA_ERR_INVALID_ARG;
  if (flags & NOVA_POOL2X2) {        // the pooled epilogue lives in the TMA-staged half-mode output transform
    if ((H | W) & 1) return NOVA_ERR_INVALID_ARG;
    if (p->mode != NOVA_FP16_F32ACC || !p->status_dev || (flags & NOVA_TRANSFORM_SIMT)) return NOVA_ERR_UNSUPPORTED;
  }
  Geom g = make_geom(p, N, H, W, C, K);
  Chunking c;
  if (!choose_chunking(p, g, ws_bytes, &c)) return NOVA_ERR_WORKSPACE;
  if (use_fused_small_c(p, g, flags)) {
    // steps 2-4 in one kernel, V and M kept on the SM: the workspace is not touched
    if (ev) cudaEventRecord(ev[0], (cudaStream_t)stream);
    if (launch_fused_small_c(p, g, x, U, y, (flags & NOVA_RELU) ? 1 : 0, stream)) return NOVA_ERR_CUDA;
    if (ev) cudaEventRecord(ev[1], (cudaStream_t)stream);
    return NOVA_OK;
  }
  const bool tc = use_tcgen05(p, flags);
  if (tc && !p->status_dev) return NOVA_ERR_CUDA;
  char* Vb = static_cast<char*>(ws);
  float* Mb = reinterpret_cast<float*>(Vb + c.v_bytes);
  const int nfreq = g.n * g.n;
  cudaStream_t s = (cudaStream_t)stream;
  int ci = 0;
  for (long long p0 = 0; p0 < g.P; p0 += c.pc, ++ci) {
    const int pc = (int)((g.P - p0) < c.pc ? (g.P - p0) : c.pc);
    if (ev) cudaEventRecord(ev[4 * ci + 0], s);
    const bool f32 = p->mode == NOVA_FP32;
    const bool tc_in = tc && p->kron_dev && C >= 64 && !(flags & NOVA_TRANSFORM_SIMT);
    if (f32     ? launch_input_transform_f32(p, g, x, Vb, p0, pc, c.pc_pad, stream)
        : tc_in ? launch_input_transform_tc(p, g, x, Vb, p0, pc, c.pc_pad, stream)
                : launch_input_transform(p, g, x, Vb, p0, pc, c.pc_pad, stream))
      return NOVA_ERR_CUDA;
    if (ev) cudaEventRecord(ev[4 * ci + 1], s);
    const int e = tc ? launch_gemm_tcgen05(p, Vb, U, Mb, nfreq, pc, c.pc_pad, C, K, p->status_dev, stream,
                                           (flags & NOVA_PROFILE_WAITS) ? p->prof_dev : nullptr)
                     : launch_gemm_simt(p, Vb, U, Mb, nfreq, pc, c.pc_pad, C, K, stream);
    if (e) return NOVA_ERR_CUDA;
    if (ev) cudaEventRecord(ev[4 * ci + 2], s);
    const int relu = ((flags & NOVA_RELU) ? 1 : 0) | ((flags & NOVA_POOL2X2) ? 2 : 0);   // bit 1: pooled store
    if (f32 ? launch_output_transform_f32(p, g, Mb, y, p0, pc, c.pc_pad, relu, stream)
        : (p->status_dev && !(flags & NOVA_TRANSFORM_SIMT))
            ? launch_output_transform_tma(p, g, Mb, y, p0, pc, c.pc_pad, relu, stream)
            : launch_output_transform(p, g, Mb, y, p0, pc, c.pc_pad, relu, stream))
      return NOVA_ERR_CUDA;
    if (ev) cudaEventRecord(ev[4 * ci + 3], s);
  }
  return NOVA_OK;
}
}  // namespace

extern "C" int nova_conv2d_fwd(const nova_plan* p, const void* x, const void* U, void* y, int N, int H,
                               int W, int C, int K, void* ws, size_t ws_bytes, int flags,
                               nova_stream stream) {
  return conv2d_fwd_impl(p, x, U, y, N, H, W, C, K, ws, ws_bytes, flags, stream, nullptr);
}

extern "C" int nova_conv2d_fwd_timed(const nova_plan* p, const void* x, const void* U, void* y, int N,
                                     int H, int W, int C, int K, void* ws, size_t ws_bytes, int flags,
                                     nova_stream stream, float* kernel_ms) {
  if (!kernel_ms) return NOVA_ERR_INVALID_ARG;
  const int launches = nova_conv2d_launch_count(p, N, H, W, C, K, ws_bytes, flags);
  if (launches < 0) return launches;
  if (launches == 1) {               // the one-kernel path: its time is reported as the product's
    cudaEvent_t e2[2];
    cudaEventCreate(&e2[0]);
    cudaEventCreate(&e2[1]);
    int st1 = conv2d_fwd_impl(p, x, U, y, N, H, W, C, K, ws, ws_bytes, flags, stream, e2);
    if (st1 == NOVA_OK && cudaStreamSynchronize((cudaStream_t)stream) != cudaSuccess) st1 = NOVA_ERR_CUDA;
    kernel_ms[0] = kernel_ms[1] = kernel_ms[2] = 0.f;
    if (st1 == NOVA_OK) cudaEventElapsedTime(&kernel_ms[1], e2[0], e2[1]);
    cudaEventDestroy(e2[0]);
    cudaEventDestroy(e2[1]);
    return st1;
  }
  const int chunks = launches / 3;
  cudaEvent_t* ev = new cudaEvent_t[4 * chunks];
  for (int i = 0; i < 4 * chunks; ++i) cudaEventCreate(&ev[i]);
  int st = conv2d_fwd_impl(p, x, U, y, N, H, W, C, K, ws, ws_bytes, flags, stream, ev);
  if (st == NOVA_OK && cudaStreamSynchronize((cudaStream_t)stream) != cudaSuccess) st = NOVA_ERR_CUDA;
  kernel_ms[0] = kernel_ms[1] = kernel_ms[2] = 0.f;
  if (st == NOVA_OK)
    for (int c = 0; c < chunks; ++c)
      for (int k = 0; k < 3; ++k) {
        float ms = 0.f;
        cudaEventElapsedTime(&ms, ev[4 * c + k], ev[4 * c + k + 1]);
        kernel_ms[k] += ms;
      }
  for (int i = 0; i < 4 * chunks; ++i) cudaEventDestroy(ev[i]);
  delete[] ev;
  return st;
}

// Streams and events of the host-buffer entry point, one set per device, made on first use.
namespace {
constexpr int kHostGroups = 8;
struct HostPipe {
  bool ready = false;
  cudaStream_t in = nullptr, out = nullptr;
  cudaEvent_t start = nullptr, done = nullptr, copied[kHostGroups] = {}, computed[kHostGroups] = {};
};
std::mutex g_pipe_mu;
HostPipe g_pipe[64];

HostPipe* host_pipe() {
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return nullptr;
  HostPipe& hp = g_pipe[dev];
  if (!hp.ready) {
    bool ok = cudaStreamCreateWithFlags(&hp.in, cudaStreamNonBlocking) == cudaSuccess &&
              cudaStreamCreateWithFlags(&hp.out, cudaStreamNonBlocking) == cudaSuccess &&
              cudaEventCreateWithFlags(&hp.start, cudaEventDisableTiming) == cudaSuccess &&
              cudaEventCreateWithFlags(&hp.done, cudaEventDisableTiming) == cudaSuccess;
    for (int i = 0; i < kHostGroups && ok; ++i)
      ok = cudaEventCreateWithFlags(&hp.copied[i], cudaEventDisableTiming) == cudaSuccess &&
           cudaEventCreateWithFlags(&hp.computed[i], cudaEventDisableTiming) == cudaSuccess;
    if (!ok) return nullptr;
    hp.ready = true;
  }
  return &hp;
}
}  // namespace

// The batch is cut into up to eight groups of images (images are independent): group i is copied in
// on one internal stream, convolved on the caller's stream and copied out on another internal
// stream, so that the two copy directions and the kernels overlap.  Everything is ordered after the
// work already in `stream`, and `stream` waits for the last copy out.
extern "C" int nova_conv2d_fwd_host(const nova_plan* p, const void* x_host, const void* U, void* y_host,
                                    int N, int H, int W, int C, int K, void* x_stage, void* y_stage,
                                    void* ws, size_t ws_bytes, int flags, nova_stream stream) {
  if (!p || !x_host || !y_host || !x_stage || !y_stage || !shape_ok(N, H, W, C, K)) return NOVA_ERR_INVALID_ARG;
  if (!device_plan(p)) return NOVA_ERR_UNSUPPORTED;
  cudaStream_t s = (cudaStream_t)stream;
  const size_t x_img = (size_t)H * W * C * elt_bytes(p->mode);
  const bool pooled = (flags & NOVA_POOL2X2) != 0;          // y_host and y_stage then hold [N, H/2, W/2, K]
  const size_t y_img = (size_t)(pooled ? H / 2 : H) * (pooled ? W / 2 : W) * K * elt_bytes(p->mode);
  std::lock_guard<std::mutex> lock(g_pipe_mu);
  HostPipe* hp = host_pipe();
  if (!hp) return NOVA_ERR_CUDA;
  const int groups = N < kHostGroups ? N : kHostGroups;
  const int per = (N + groups - 1) / groups;
  if (cudaEventRecord(hp->start, s) != cudaSuccess || cudaStreamWaitEvent(hp->in, hp->start, 0) != cudaSuccess ||
      cudaStreamWaitEvent(hp->out, hp->start, 0) != cudaSuccess)
    return NOVA_ERR_CUDA;
  for (int gi = 0, n0 = 0; n0 < N; ++gi, n0 += per) {
    const int n = (N - n0) < per ? (N - n0) : per;
    const char* xh = static_cast<const char*>(x_host) + (size_t)n0 * x_img;
    char* xs = static_cast<char*>(x_stage) + (size_t)n0 * x_img;
    char* ys = static_cast<char*>(y_stage) + (size_t)n0 * y_img;
    char* yh = static_cast<char*>(y_host) + (size_t)n0 * y_img;
    if (cudaMemcpyAsync(xs, xh, (size_t)n * x_img, cudaMemcpyHostToDevice, hp->in) != cudaSuccess ||
        cudaEventRecord(hp->copied[gi], hp->in) != cudaSuccess ||
        cudaStreamWaitEvent(s, hp->copied[gi], 0) != cudaSuccess)
      return NOVA_ERR_CUDA;
    const int st = nova_conv2d_fwd(p, xs, U, ys, n, H, W, C, K, ws, ws_bytes, flags, stream);
    if (st != NOVA_OK) return st;
    if (cudaEventRecord(hp->computed[gi], s) != cudaSuccess ||
        cudaStreamWaitEvent(hp->out, hp->computed[gi], 0) != cudaSuccess ||
        cudaMemcpyAsync(yh, ys, (size_t)n * y_img, cudaMemcpyDeviceToHost, hp->out) != cudaSuccess)
      return NOVA_ERR_CUDA;
  }
  if (cudaEventRecord(hp->done, hp->out) != cudaSuccess || cudaStreamWaitEvent(s, hp->done, 0) != cudaSuccess)
    return NOVA_ERR_CUDA;
  return NOVA_OK;
}

// ---------------------------------------------------------------------------
// No-allocation variant.  The scratch is part of the library image; in host
// code `g_static_scratch` is only a handle for the symbol query below, never
// a pointer a kernel could use.
static __device__ __align__(256) unsigned char g_static_scratch[NOVA_STATIC_SCRATCH_BYTES];

namespace {
constexpr int kMaxDevices = 64;
std::mutex g_static_mu;
void* g_static_ptr[kMaxDevices] = {};   // device address of the array, per device ordinal

// Device address of the array on the current device; queried once per device.
int static_scratch_address(void** out) {
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return NOVA_ERR_CUDA;
  std::lock_guard<std::mutex> lock(g_static_mu);
  if (!g_static_ptr[dev]) {
    void* p = nullptr;
    if (cudaGetSymbolAddress(&p, g_static_scratch) != cudaSuccess || !p) return NOVA_ERR_CUDA;
    g_static_ptr[dev] = p;
  }
  *out = g_static_ptr[dev];
  return NOVA_OK;
}
}  // namespace

extern "C" int nova_conv2d_fwd_static(const nova_plan* p, const void* x, const void* U, void* y, int N,
                                      int H, int W, int C, int K, int flags, nova_stream stream) {
  if (!p || !shape_ok(N, H, W, C, K)) return NOVA_ERR_INVALID_ARG;
  if (!device_plan(p)) return NOVA_ERR_UNSUPPORTED;
  if (nova_conv2d_min_workspace_bytes(p, N, H, W, C, K) > NOVA_STATIC_SCRATCH_BYTES)
    return NOVA_ERR_STATIC_LIMIT;
  if (p->device < 0) return NOVA_ERR_CUDA;
  if (!on_plan_device(p)) return NOVA_ERR_INVALID_ARG;   // the scratch looked up below is the current device's
  void* ws = nullptr;
  const int st = static_scratch_address(&ws);
  if (st != NOVA_OK) return st;
  return conv2d_fwd_impl(p, x, U, y, N, H, W, C, K, ws, NOVA_STATIC_SCRATCH_BYTES, flags, stream, nullptr);
}

// ---------------------------------------------------------------------------
// INT8 Winograd-domain pipeline.
namespace {
bool int8_shape_ok(const nova_plan* p, int N, int H, int W, int C, int K) {
  return device_plan(p) && p->mode == NOVA_FP16_F32ACC && shape_ok(N, H, W, C, K) && (C % 16) == 0 && (K % 16) == 0;
}
struct Int8Layout {
  int pad;                  // tiles rounded up to whole 128-row blocks
  size_t v_off, m_off, total;
};
Int8Layout int8_layout(const Geom& g) {
  Int8Layout l;
  l.pad = (int)round_up_ll(g.P, 128);
  l.v_off = kAlign;                                   // the first block holds the scale of V
  l.m_off = l.v_off + round_up((size_t)g.n * g.n * l.pad * g.C, kAlign);
  l.total = l.m_off + round_up((size_t)g.n * g.n * l.pad * g.K * 4, kAlign);
  return l;
}

int conv2d_int8_impl(const nova_plan* p, const void* x, const void* Uq, const float* scale_U, float scale_V,
                     void* y, int N, int H, int W, int C, int K, void* ws, size_t ws_bytes, int flags,
                     nova_stream stream, cudaEvent_t* ev) {
  if (!int8_shape_ok(p, N, H, W, C, K) || !aligned16(x) || !aligned16(Uq) || !aligned16(y) || !scale_U ||
      !(scale_V >= 0.f))
    return p && (p->mode != NOVA_FP16_F32ACC || !device_plan(p)) ? NOVA_ERR_UNSUPPORTED : NOVA_ERR_INVALID_ARG;
  if (!ws || (reinterpret_cast<uintptr_t>(ws) % kAlign)) return NOVA_ERR_WORKSPACE;
  if ((flags & NOVA_POOL2X2) && ((H | W) & 1)) return NOVA_ERR_INVALID_ARG;
  if (!p->status_dev) return NOVA_ERR_CUDA;
  if (!on_plan_device(p)) return NOVA_ERR_INVALID_ARG;
  const Geom g = make_geom(p, N, H, W, C, K);
  if (g.P >= (1ll << 24)) return NOVA_ERR_UNSUPPORTED;
  const Int8Layout l = int8_layout(g);
  if (ws_bytes < l.total) return NOVA_ERR_WORKSPACE;
  char* base = static_cast<char*>(ws);
  float* slot = reinterpret_cast<float*>(base);
  void* Vq = base + l.v_off;
  int32_t* Mb = reinterpret_cast<int32_t*>(base + l.m_off);
  cudaStream_t s = (cudaStream_t)stream;
  const int pc = (int)g.P, nfreq = g.n * g.n;
  int e = 0;
  // The tensor-core transform needs the exact hi + lo table of half-rounded coefficients; plans
  // with float32 coefficients (and narrow layers) use the CUDA-core transform.
  const bool tc_in = p->kron_dev && C >= 64 && !(flags & NOVA_TRANSFORM_SIMT);
  auto transform = [&](int pass) {
    return tc_in ? launch_input_transform_tc_int8(p, g, x, Vq, slot, pass, 0, pc, l.pad, stream)
                 : launch_input_transform_int8(p, g, x, Vq, slot, pass, 0, pc, l.pad, stream);
  };
  if (ev) cudaEventRecord(ev[0], s);
  if (scale_V > 0.f) {
    e = launch_scale_slot(slot, scale_V, 0, stream);
  } else {                                            // s_V = max|V| / 127 over the batch: one more pass
    if (cudaMemsetAsync(slot, 0, sizeof(float), s) != cudaSuccess) return NOVA_ERR_CUDA;
    e = transform(0);
    if (!e) e = launch_scale_slot(slot, 0.f, 1, stream);
  }
  if (!e) e = transform(1);
  if (ev) cudaEventRecord(ev[1], s);
  if (!e)
    e = (flags & NOVA_GEMM_SIMT) ? launch_gemm_simt_i8(Vq, Uq, Mb, nfreq, pc, l.pad, C, K, stream)
                                 : launch_gemm_tcgen05_i8(p, Vq, Uq, Mb, nfreq, pc, l.pad, C, K, p->status_dev, stream);
  if (ev) cudaEventRecord(ev[2], s);
  if (!e)
    e = launch_output_transform_tma(p, g, Mb, y, 0, pc, l.pad,
                                    ((flags & NOVA_RELU) ? 1 : 0) | ((flags & NOVA_POOL2X2) ? 2 : 0), stream, scale_U, slot);
  if (ev) cudaEventRecord(ev[3], s);
  if (e) g_last_cuda_error = e;
  return e ? NOVA_ERR_CUDA : NOVA_OK;
}
}  // namespace

extern "C" size_t nova_filter_transform_int8_bytes(const nova_plan* p, int K, int C) {
  if (!device_plan(p) || K <= 0 || C <= 0) return 0;
  return (size_t)p->n * p->n * K * C;
}

extern "C" int nova_filter_transform_int8(const nova_plan* p, const void* g, int K, int C, int quant, void* Uq,
                                          float* scale_U, nova_stream stream) {
  if (p && (p->mode != NOVA_FP16_F32ACC || !device_plan(p))) return NOVA_ERR_UNSUPPORTED;
  if (!p || !aligned16(g) || !aligned16(Uq) || !scale_U || K <= 0 || C <= 0 || (K % 16) || (C % 16))
    return NOVA_ERR_INVALID_ARG;
  if (quant != NOVA_QUANT_PER_TENSOR && quant != NOVA_QUANT_PER_CHANNEL && quant != NOVA_QUANT_GIVEN)
    return NOVA_ERR_INVALID_ARG;
  if (p->mode != NOVA_FP16_F32ACC || !device_plan(p)) return NOVA_ERR_UNSUPPORTED;
  if (p->device < 0) return NOVA_ERR_CUDA;
  if (!on_plan_device(p)) return NOVA_ERR_INVALID_ARG;
  const int e = launch_filter_transform_int8(p, g, K, C, Uq, scale_U, quant, stream);
  if (e) g_last_cuda_error = e;
  return e ? NOVA_ERR_CUDA : NOVA_OK;
}

extern "C" size_t nova_conv2d_int8_workspace_bytes(const nova_plan* p, int N, int H, int W, int C, int K) {
  if (!int8_shape_ok(p, N, H, W, C, K)) return 0;
  return int8_layout(make_geom(p, N, H, W, C, K)).total;
}

extern "C" int nova_conv2d_fwd_int8(const nova_plan* p, const void* x, const void* Uq, const float* scale_U,
                                    float scale_V, void* y, int N, int H, int W, int C, int K, void* ws,
                                    size_t ws_bytes, int flags, nova_stream stream) {
  return conv2d_int8_impl(p, x, Uq, scale_U, scale_V, y, N, H, W, C, K, ws, ws_bytes, flags, stream, nullptr);
}

extern "C" int nova_conv2d_fwd_int8_timed(const nova_plan* p, const void* x, const void* Uq, const float* scale_U,
                                          float scale_V, void* y, int N, int H, int W, int C, int K, void* ws,
                                          size_t ws_bytes, int flags, nova_stream stream, float* ms) {
  if (!ms) return NOVA_ERR_INVALID_ARG;
  cudaEvent_t ev[4];
  for (auto& e : ev) cudaEventCreate(&e);
  int st = conv2d_int8_impl(p, x, Uq, scale_U, scale_V, y, N, H, W, C, K, ws, ws_bytes, flags, stream, ev);
  if (st == NOVA_OK && cudaStreamSynchronize((cudaStream_t)stream) != cudaSuccess) st = NOVA_ERR_CUDA;
  ms[0] = ms[1] = ms[2] = ms[3] = 0.f;
  if (st == NOVA_OK) {
    for (int k = 0; k < 3; ++k) cudaEventElapsedTime(&ms[k], ev[k], ev[k + 1]);
    cudaEventElapsedTime(&ms[3], ev[0], ev[3]);
  }
  for (auto& e : ev) cudaEventDestroy(e);
  return st;
}

// ---------------------------------------------------------------------------
// Self-test of the failure reporting: one warp waits on an mbarrier phase that nothing completes,
// with the same bounded wait the kernels use but a caller-chosen limit, and reports the expiry
// through the plan's status word.  The wait ends by the clock; nothing faults or hangs.
namespace nova {
static __global__ void wait_timeout_selftest_kernel(int* status, unsigned long long limit_ns, unsigned long long* waited_ns) {
  __shared__ uint64_t bar;
  __shared__ int abort_flag;
  if (threadIdx.x == 0) {
    sm100::mbar_init(&bar, 1);
    abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  __syncthreads();
  const uint64_t t0 = sm100::global_ns();
  const bool ok = sm100::mbar_wait_limited(&bar, 0, &abort_flag, limit_ns, 1u << 16);
  if (threadIdx.x == 0) {
    *waited_ns = sm100::global_ns() - t0;
    if (!ok) atomicExch(status, NOVA_ERR_DEVICE_TIMEOUT);
  }
}
}  // namespace nova

extern "C" int nova_selftest_wait_timeout(const nova_plan* p, unsigned limit_ms, unsigned long long* waited_ns_host,
                                          nova_stream stream) {
  if (!p || !waited_ns_host || limit_ms < 1 || limit_ms > 1000) return NOVA_ERR_INVALID_ARG;
  if (!p->status_dev) return NOVA_ERR_CUDA;
  cudaStream_t s = (cudaStream_t)stream;
  unsigned long long* w = nullptr;
  if (cudaMalloc((void**)&w, sizeof(*w)) != cudaSuccess) return NOVA_ERR_CUDA;
  wait_timeout_selftest_kernel<<<1, 32, 0, s>>>(p->status_dev, (unsigned long long)limit_ms * 1000000ull, w);
  int st = cudaGetLastError() == cudaSuccess ? NOVA_OK : NOVA_ERR_CUDA;
  if (st == NOVA_OK && (cudaMemcpyAsync(waited_ns_host, w, sizeof(*w), cudaMemcpyDeviceToHost, s) != cudaSuccess ||
                        cudaStreamSynchronize(s) != cudaSuccess))
    st = NOVA_ERR_CUDA;
  cudaFree(w);
  return st;
}

extern "C" int nova_plan_wait_profile(const nova_plan* p, double* cycles_host, nova_stream stream) {
  if (!p || !cycles_host) return NOVA_ERR_INVALID_ARG;
  if (!p->prof_dev || p->sm_count <= 0) return NOVA_ERR_CUDA;
  if (!on_plan_device(p)) return NOVA_ERR_INVALID_ARG;
  cudaStream_t s = (cudaStream_t)stream;
  const int n = p->sm_count;
  unsigned long long* h = new unsigned long long[(size_t)n * 8];
  int st = NOVA_OK;
  if (cudaMemcpyAsync(h, p->prof_dev, sizeof(unsigned long long) * n * 8, cudaMemcpyDeviceToHost, s) != cudaSuccess ||
      cudaStreamSynchronize(s) != cudaSuccess)
    st = NOVA_ERR_CUDA;
  if (st == NOVA_OK) {
    int ctas = 0;                                      // CTAs that ran: those with a non-zero item count
    for (int k = 0; k < 8; ++k) cycles_host[k] = 0.0;
    for (int i = 0; i < n; ++i) {
      if (h[(size_t)i * 8 + 7] == 0) continue;
      ++ctas;
      for (int k = 0; k < 8; ++k) cycles_host[k] += (double)h[(size_t)i * 8 + k];
    }
    for (int k = 0; k < 8; ++k) cycles_host[k] = ctas ? cycles_host[k] / ctas : 0.0;
    cycles_host[8] = (double)ctas;
  }
  delete[] h;
  return st;
}

extern "C" int nova_last_cuda_error(void) { return g_last_cuda_error; }

extern "C" int nova_maxpool2x2(const void* x, void* y, int N, int H, int W, int C, int mode,
                               nova_stream stream) {
  if (!aligned16(x) || !aligned16(y) || N <= 0 || H <= 0 || W <= 0 || (H & 1) || (W & 1) || C <= 0 || (C % 8))
    return NOVA_ERR_INVALID_ARG;
  if (mode != NOVA_FP32 && mode != NOVA_FP16_F32ACC) return NOVA_ERR_INVALID_ARG;
  return launch_maxpool2x2(x, y, N, H, W, C, mode, stream) == 0 ? NOVA_OK : NOVA_ERR_CUDA;
}

extern "C" int nova_last_device_status(const nova_plan* p, nova_stream stream) {
  if (!p) return NOVA_ERR_INVALID_ARG;
  if (!p->status_dev) return NOVA_ERR_CUDA;
  cudaStream_t s = (cudaStream_t)stream;
  int v = 0;
  if (cudaMemcpyAsync(&v, p->status_dev, sizeof(int), cudaMemcpyDeviceToHost, s) != cudaSuccess)
    return NOVA_ERR_CUDA;
  if (cudaStreamSynchronize(s) != cudaSuccess) return NOVA_ERR_CUDA;
  if (v != 0) {
    cudaMemsetAsync(p->status_dev, 0, sizeof(int), s);
    cudaStreamSynchronize(s);
  }
  return v;
}
