// Internal declarations shared by the translation units of libnova.
#pragma once
#include <cstddef>
#include <cstdint>
#include "nova.h"

namespace nova {

constexpr int kMaxN = 10;   // n = m + 2 for m = 8
constexpr int kMaxM = 8;
constexpr int kR = 3;        // filter taps of the device path
constexpr int kMaxR = 5;     // filter taps a host-only plan may have

// Coefficient tables as the kernels evaluate them.  Passed by value as a
// __grid_constant__ kernel parameter, i.e. they live in the constant bank and
// fully unrolled loops read them as constant-memory operands.
struct Coefs {
  float BT[kMaxN][kMaxN];
  float AT[kMaxM][kMaxN];
  float G[kMaxN][kMaxR];
};

}  // namespace nova

struct nova_plan {
  int m, r, n;
  int mode, coef;
  nova_rat points[nova::kMaxN];
  double AT[nova::kMaxM * nova::kMaxN];   // m x n row-major
  double G[nova::kMaxN * nova::kMaxR];    // n x r
  double BT[nova::kMaxN * nova::kMaxN];   // n x n
  double kappa2_V;
  double kappa2_mat[3], norm2_mat[3];     // kappa_2 and spectral norm of A, G, B (as scaled)
  nova_rat AT_rat[nova::kMaxM * nova::kMaxN], G_rat[nova::kMaxN * nova::kMaxR], BT_rat[nova::kMaxN * nova::kMaxN];
  int rat_fits;                           // every exact entry fits a 64-bit numerator / denominator
  nova::Coefs coefs;                      // rounded to the coefficient precision, caller's point order
  // The kernels index frequencies in an internal point order: perm[i] is the
  // caller's index of internal point i.  For a symmetric set {0, +-a_1, ..,
  // +-a_q, infinity} the internal order is 0, +a_1, -a_1, .., +a_q, -a_q,
  // infinity, the rounded tables have the even/odd structure the SYM kernel
  // paths rely on (checked entry by entry), and symmetric = 1; otherwise the
  // order is the caller's and the kernels evaluate dense products.
  nova::Coefs kcoefs;
  int perm[nova::kMaxN];
  int symmetric;
  void* kron_dev;                         // device table of the tensor-core input transform (may be null)
  int* status_dev;                        // device status word (null without a device)
  int device;                             // device that owns status_dev
  int sm_count;                           // multiprocessors of that device
  int l2_bytes;                           // size of its L2
  unsigned long long* prof_dev;           // 8 wait counters per multiprocessor (NOVA_PROFILE_WAITS; may be null)
};

namespace nova {

inline size_t elt_bytes(int mode) { return mode == NOVA_FP32 ? 4 : 2; }

// Tile geometry of one problem.
struct Geom {
  int N, H, W, C, K, m, n, Th, Tw;
  long long P;   // total tiles
};
inline Geom make_geom(const nova_plan* p, int N, int H, int W, int C, int K) {
  Geom g;
  g.N = N; g.H = H; g.W = W; g.C = C; g.K = K; g.m = p->m; g.n = p->n;
  g.Th = (H + p->m - 1) / p->m;
  g.Tw = (W + p->m - 1) / p->m;
  g.P = (long long)N * g.Th * g.Tw;
  return g;
}

// Kernel launchers (defined in the .cu files).  All return a cudaError_t as int.
int launch_filter_transform(const nova_plan* plan, const void* g, int K, int C, void* U, void* stream);
int launch_input_transform(const nova_plan* plan, const Geom& g, const void* x, void* V,
                           long long p0, int pc, int pc_pad, void* stream);
int launch_input_transform_tc(const nova_plan* plan, const Geom& g, const void* x, void* V,
                              long long p0, int pc, int pc_pad, void* stream);
size_t kron_table_halves(int n);   // n points
void build_kron_table(const nova_plan* plan, unsigned short* out);
int launch_output_transform(const nova_plan* plan, const Geom& g, const void* M, void* y,
                            long long p0, int pc, int pc_pad, int relu, void* stream);
// scale_U / scale_V non-null: M holds int32 sums of the int8 pipeline, dequantised on load
int launch_output_transform_tma(const nova_plan* plan, const Geom& g, const void* M, void* y,
                                long long p0, int pc, int pc_pad, int relu, void* stream,
                                const float* scale_U = nullptr, const float* scale_V = nullptr);
int launch_filter_transform_int8(const nova_plan* plan, const void* g, int K, int C, void* Uq, float* scales,
                                 int quant, void* stream);
int launch_input_transform_int8(const nova_plan* plan, const Geom& g, const void* x, void* Vq, float* slot,
                                int pass, long long p0, int pc, int pc_pad, void* stream);
int launch_input_transform_tc_int8(const nova_plan* plan, const Geom& g, const void* x, void* Vq, float* slot,
                                   int pass, long long p0, int pc, int pc_pad, void* stream);
int launch_scale_slot(float* slot, float value, int from_absmax, void* stream);
int launch_gemm_tcgen05_i8(const nova_plan* plan, const void* V, const void* U, int32_t* M, int nfreq, int pc,
                           int pc_pad, int C, int K, int* status_dev, void* stream);
int launch_gemm_simt_i8(const void* V, const void* U, int32_t* M, int nfreq, int pc, int pc_pad, int C, int K,
                        void* stream);
// fp32 mode: sums carried in double, one rounding per stored float
int launch_filter_transform_f32(const nova_plan* plan, const void* g, int K, int C, void* U, void* stream);
int launch_input_transform_f32(const nova_plan* plan, const Geom& g, const void* x, void* V, long long p0, int pc,
                               int pc_pad, void* stream);
int launch_output_transform_f32(const nova_plan* plan, const Geom& g, const void* M, void* y, long long p0, int pc,
                                int pc_pad, int relu, void* stream);
int launch_gemm_simt(const nova_plan* plan, const void* V, const void* U, float* M,
                     int nfreq, int pc, int pc_pad, int C, int K, void* stream);
// prof non-null (K > 128, half operands): the wait-profiling variant writes 8 counters per CTA there
int launch_gemm_tcgen05(const nova_plan* plan, const void* V, const void* U, float* M,
                        int nfreq, int pc, int pc_pad, int C, int K, int* status_dev, void* stream,
                        unsigned long long* prof = nullptr);
// Input transform, product and output transform in one kernel for C = 8 (half mode, 3-tap filters)
bool fused_small_c_applies(const nova_plan* plan, const Geom& g);
int launch_fused_small_c(const nova_plan* plan, const Geom& g, const void* x, const void* U, void* y, int relu,
                         void* stream);
int launch_maxpool2x2(const void* x, void* y, int N, int H, int W, int C, int mode, void* stream);

}  // namespace nova
