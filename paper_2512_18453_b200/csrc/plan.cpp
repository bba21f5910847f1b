// Host-side plan builder: exact Toom-Cook construction of A^T, G, B^T from a
// rational point set with the point at infinity (Algorithm 3, "Symbolic
// Cook-Toom Construction"), the exact decomposition check of Section 2.4,
// rounding of the tables, and kappa_2 of the Vandermonde matrix (Section 2.2).
#include <algorithm>
#include <cmath>
#include <cstring>
#include <new>
#include <vector>

#include <cuda_runtime_api.h>

#include "nova_internal.h"

namespace {

typedef __int128 i128;
typedef unsigned __int128 u128;

// ---------------------------------------------------------------- rationals
// Reduced fractions over 128-bit integers; `bad` latches overflow.
struct Rat {
  i128 n = 0, d = 1;
};

i128 iabs(i128 v) { return v < 0 ? -v : v; }
i128 gcd128(i128 a, i128 b) {
  a = iabs(a); b = iabs(b);
  while (b) { i128 t = a % b; a = b; b = t; }
  return a;
}
struct Arith {
  bool bad = false;
  i128 mul(i128 a, i128 b) {
    i128 r;
    if (__builtin_mul_overflow(a, b, &r)) { bad = true; return 0; }
    return r;
  }
  i128 add(i128 a, i128 b) {
    i128 r;
    if (__builtin_add_overflow(a, b, &r)) { bad = true; return 0; }
    return r;
  }
  Rat norm(i128 n, i128 d) {
    if (d == 0) { bad = true; return Rat(); }
    if (d < 0) { n = -n; d = -d; }
    i128 g = gcd128(n, d);
    if (g > 1) { n /= g; d /= g; }
    Rat r; r.n = n; r.d = d;
    return r;
  }
  Rat mul(const Rat& a, const Rat& b) {
    // cross-reduce first to keep the products small
    i128 g1 = gcd128(a.n, b.d), g2 = gcd128(b.n, a.d);
    if (g1 == 0) g1 = 1;
    if (g2 == 0) g2 = 1;
    return norm(mul(a.n / g1, b.n / g2), mul(a.d / g2, b.d / g1));
  }
  Rat div(const Rat& a, const Rat& b) {
    if (b.n == 0) { bad = true; return Rat(); }
    Rat inv; inv.n = b.d; inv.d = b.n;
    if (inv.d < 0) { inv.n = -inv.n; inv.d = -inv.d; }
    return mul(a, inv);
  }
  Rat plus(const Rat& a, const Rat& b) {
    Rat nb = b; nb.n = -nb.n;
    return sub(a, nb);
  }
  Rat sub(const Rat& a, const Rat& b) {
    i128 g = gcd128(a.d, b.d);
    if (g == 0) g = 1;
    i128 bd = b.d / g, ad = a.d / g;
    return norm(add(mul(a.n, bd), -mul(b.n, ad)), mul(a.d, bd));
  }
};

double rat_to_double(const Rat& r) {
  const i128 lim = (i128)1 << 53;
  if (iabs(r.n) < lim && r.d < lim) return (double)(long long)r.n / (double)(long long)r.d;  // one IEEE division: correctly rounded
  return (double)((long double)r.n / (long double)r.d);
}

// ------------------------------------------------------- big integers (check)
// Sign-magnitude, base 2^32, only what the exactness check needs.
struct Big {
  bool neg = false;
  std::vector<uint32_t> w;   // little endian, no leading zeros
  bool zero() const { return w.empty(); }
};
Big big_from(i128 v) {
  Big b;
  b.neg = v < 0;
  u128 u = b.neg ? (u128)(-(v + 1)) + 1 : (u128)v;
  while (u) { b.w.push_back((uint32_t)u); u >>= 32; }
  return b;
}
void trim(Big& b) {
  while (!b.w.empty() && b.w.back() == 0) b.w.pop_back();
  if (b.w.empty()) b.neg = false;
}
int cmp_mag(const Big& a, const Big& b) {
  if (a.w.size() != b.w.size()) return a.w.size() < b.w.size() ? -1 : 1;
  for (size_t i = a.w.size(); i-- > 0;)
    if (a.w[i] != b.w[i]) return a.w[i] < b.w[i] ? -1 : 1;
  return 0;
}
Big add_mag(const Big& a, const Big& b) {
  Big r;
  uint64_t c = 0;
  size_t n = std::max(a.w.size(), b.w.size());
  for (size_t i = 0; i < n; ++i) {
    uint64_t s = c + (i < a.w.size() ? a.w[i] : 0) + (i < b.w.size() ? b.w[i] : 0);
    r.w.push_back((uint32_t)s);
    c = s >> 32;
  }
  if (c) r.w.push_back((uint32_t)c);
  return r;
}
Big sub_mag(const Big& a, const Big& b) {   // |a| >= |b|
  Big r;
  int64_t c = 0;
  for (size_t i = 0; i < a.w.size(); ++i) {
    int64_t s = (int64_t)a.w[i] - (i < b.w.size() ? b.w[i] : 0) + c;
    c = 0;
    if (s < 0) { s += ((int64_t)1 << 32); c = -1; }
    r.w.push_back((uint32_t)s);
  }
  trim(r);
  return r;
}
Big big_add(const Big& a, const Big& b) {
  Big r;
  if (a.neg == b.neg) { r = add_mag(a, b); r.neg = a.neg; }
  else {
    int c = cmp_mag(a, b);
    if (c == 0) return Big();
    if (c > 0) { r = sub_mag(a, b); r.neg = a.neg; }
    else { r = sub_mag(b, a); r.neg = b.neg; }
  }
  trim(r);
  return r;
}
Big big_mul(const Big& a, const Big& b) {
  Big r;
  if (a.zero() || b.zero()) return r;
  r.w.assign(a.w.size() + b.w.size(), 0);
  for (size_t i = 0; i < a.w.size(); ++i) {
    uint64_t c = 0;
    for (size_t j = 0; j < b.w.size(); ++j) {
      uint64_t t = (uint64_t)a.w[i] * b.w[j] + r.w[i + j] + c;
      r.w[i + j] = (uint32_t)t;
      c = t >> 32;
    }
    size_t k = i + b.w.size();
    while (c) { uint64_t t = (uint64_t)r.w[k] + c; r.w[k] = (uint32_t)t; c = t >> 32; ++k; }
  }
  r.neg = a.neg != b.neg;
  trim(r);
  return r;
}

// ------------------------------------------------------------ half rounding
// double -> IEEE binary16 (round to nearest even) -> float, on the host.
float round_through_half(double v) {
  if (std::isnan(v)) return NAN;
  double a = std::fabs(v);
  float sign = std::signbit(v) ? -1.f : 1.f;
  if (a >= 65520.0) return sign * INFINITY;            // halfway between 65504 and 2^16 rounds to inf
  if (a == 0.0) return sign * 0.f;
  int e;
  std::frexp(a, &e);                                    // a = f * 2^e, f in [0.5, 1)
  int exp2 = e - 1;                                     // a in [2^exp2, 2^(exp2+1))
  if (exp2 < -14) exp2 = -14;                           // subnormal spacing 2^-24
  double ulp = std::ldexp(1.0, exp2 - 10);
  double q = std::nearbyint(a / ulp);                   // default rounding mode: to nearest even
  return sign * (float)(q * ulp);
}

// ---------------------------------------------------------------- kappa_2
// One-sided Jacobi SVD of a small rows x n matrix (rows >= n, row-major, leading dimension n);
// returns sigma_max/sigma_min and, if asked, sigma_max.
double cond2(std::vector<double> a, int n, int rows = -1, double* sigma_max = nullptr) {
  if (rows < 0) rows = n;
  for (int sweep = 0; sweep < 60; ++sweep) {
    double off = 0;
    for (int p = 0; p < n - 1; ++p)
      for (int q = p + 1; q < n; ++q) {
        double al = 0, be = 0, ga = 0;
        for (int i = 0; i < rows; ++i) {
          al += a[i * n + p] * a[i * n + p];
          be += a[i * n + q] * a[i * n + q];
          ga += a[i * n + p] * a[i * n + q];
        }
        if (ga == 0) continue;
        off = std::max(off, std::fabs(ga) / std::sqrt(al * be));
        double zeta = (be - al) / (2 * ga);
        double t = (zeta >= 0 ? 1.0 : -1.0) / (std::fabs(zeta) + std::sqrt(1 + zeta * zeta));
        double c = 1 / std::sqrt(1 + t * t), s = c * t;
        for (int i = 0; i < rows; ++i) {
          double x = a[i * n + p], y = a[i * n + q];
          a[i * n + p] = c * x - s * y;
          a[i * n + q] = s * x + c * y;
        }
      }
    if (off < 1e-15) break;
  }
  double smax = 0, smin = INFINITY;
  for (int j = 0; j < n; ++j) {
    double s = 0;
    for (int i = 0; i < rows; ++i) s += a[i * n + j] * a[i * n + j];
    s = std::sqrt(s);
    smax = std::max(smax, s);
    smin = std::min(smin, s);
  }
  if (sigma_max) *sigma_max = smax;
  return smax / smin;
}

// Exact check of the bilinear identity sum_p A^T[i][p] G[p][k] B^T[p][j] == [j == i + k]
// (Section 2.4), over arbitrary-precision integers.
bool identity_holds(int m, int r, int n, const std::vector<Rat>& AT, const std::vector<Rat>& G,
                    const std::vector<Rat>& BT) {
  for (int i = 0; i < m; ++i)
    for (int k = 0; k < r; ++k)
      for (int j = 0; j < n; ++j) {
        Big num, den = big_from(1);
        for (int p = 0; p < n; ++p) {
          const Rat &a = AT[i * n + p], &g = G[p * r + k], &b = BT[p * n + j];
          if (a.n == 0 || g.n == 0 || b.n == 0) continue;
          Big tn = big_mul(big_mul(big_from(a.n), big_from(g.n)), big_from(b.n));
          Big td = big_mul(big_mul(big_from(a.d), big_from(g.d)), big_from(b.d));
          num = big_add(big_mul(num, td), big_mul(tn, den));
          den = big_mul(den, td);
        }
        if (j == i + k) { Big md = den; md.neg = !md.neg; num = big_add(num, md); }
        if (!num.zero()) return false;
      }
  return true;
}

bool fits64(const Rat& v, nova_rat* out) {
  const i128 lim = (i128)1 << 63;
  if (v.n >= lim || v.n < -lim || v.d >= lim) return false;
  out->num = (int64_t)v.n;
  out->den = (int64_t)v.d;
  return true;
}

int create_impl(int m, int r, const nova_rat* points, int n, const nova_rat* scale_G, const nova_rat* scale_B,
                int mode, int coef, nova_plan** out);

int create_impl(int m, int r, const nova_rat* points, int n, const nova_rat* scale_G, const nova_rat* scale_B,
                int mode, int coef, nova_plan** out) {
  if (out) *out = nullptr;
  if (!points || !out) return NOVA_ERR_INVALID_ARG;
  if (m != 2 && m != 4 && m != 6 && m != 8) return NOVA_ERR_INVALID_ARG;
  if (r != 3 && r != 5) return NOVA_ERR_UNSUPPORTED;
  if (n != m + r - 1) return NOVA_ERR_INVALID_ARG;
  if (n > nova::kMaxN) return NOVA_ERR_UNSUPPORTED;   // F(8,5) would need 12 points
  if (mode != NOVA_FP32 && mode != NOVA_FP16_F32ACC) return NOVA_ERR_INVALID_ARG;
  if (coef != NOVA_COEF_ROUND_TO_MODE && coef != NOVA_COEF_FP32) return NOVA_ERR_INVALID_ARG;

  int n_inf = 0;
  for (int i = 0; i < n; ++i) {
    if (points[i].den < 0) return NOVA_ERR_INVALID_ARG;
    if (points[i].den == 0) ++n_inf;
  }
  if (n_inf == 0) return NOVA_ERR_NO_INFINITY;
  if (n_inf > 1 || points[n - 1].den != 0) return NOVA_ERR_MULTIPLE_INFINITY;

  Arith ar;
  const int nf = n - 1;
  Rat al[nova::kMaxN];
  for (int i = 0; i < nf; ++i) al[i] = ar.norm(points[i].num, points[i].den);
  for (int i = 0; i < nf; ++i)
    for (int j = i + 1; j < nf; ++j)
      if (al[i].n == al[j].n && al[i].d == al[j].d) return NOVA_ERR_DUPLICATE_POINT;

  // Lagrange factors F_i = prod_{j != i} (alpha_i - alpha_j)
  Rat F[nova::kMaxN];
  for (int i = 0; i < nf; ++i) {
    Rat f; f.n = 1; f.d = 1;
    for (int j = 0; j < nf; ++j)
      if (j != i) f = ar.mul(f, ar.sub(al[i], al[j]));
    F[i] = f;
  }
  Rat zero, one; one.n = 1;
  std::vector<Rat> AT(m * n, zero), G(n * r, zero), BT(n * n, zero);
  for (int p = 0; p < nf; ++p) {
    Rat pw = one;                                         // alpha_p^i, 0^0 = 1
    for (int i = 0; i < std::max(m, r); ++i) {
      if (i < m) AT[i * n + p] = pw;
      if (i < r) G[p * r + i] = ar.div(pw, F[p]);
      pw = ar.mul(pw, al[p]);
    }
  }
  AT[(m - 1) * n + (n - 1)] = one;
  G[(n - 1) * r + (r - 1)] = one;
  for (int p = 0; p < n; ++p) {                           // row n-1: all finite roots
    std::vector<Rat> poly(1, one);
    for (int j = 0; j < nf; ++j) {
      if (j == p) continue;
      std::vector<Rat> nx(poly.size() + 1, zero);
      for (size_t t = 0; t < poly.size(); ++t) {
        nx[t + 1] = ar.plus(nx[t + 1], poly[t]);          // t * poly
        nx[t] = ar.sub(nx[t], ar.mul(poly[t], al[j]));    // -= poly[t] * alpha_j
      }
      poly.swap(nx);
    }
    for (size_t t = 0; t < poly.size(); ++t) BT[p * n + t] = poly[t];
  }
  // Diagonal rescaling: rows of G by D_G, rows of B^T by D_B, columns of A^T by (D_G D_B)^-1.
  if (scale_G || scale_B) {
    for (int p = 0; p < n; ++p) {
      Rat sg = one, sb = one;
      if (scale_G) { if (scale_G[p].den <= 0 || scale_G[p].num == 0) return NOVA_ERR_INVALID_ARG; sg = ar.norm(scale_G[p].num, scale_G[p].den); }
      if (scale_B) { if (scale_B[p].den <= 0 || scale_B[p].num == 0) return NOVA_ERR_INVALID_ARG; sb = ar.norm(scale_B[p].num, scale_B[p].den); }
      const Rat both = ar.mul(sg, sb);
      for (int k = 0; k < r; ++k) G[p * r + k] = ar.mul(G[p * r + k], sg);
      for (int j = 0; j < n; ++j) BT[p * n + j] = ar.mul(BT[p * n + j], sb);
      for (int i = 0; i < m; ++i) AT[i * n + p] = ar.div(AT[i * n + p], both);
    }
  }
  if (ar.bad) return NOVA_ERR_RATIONAL_OVERFLOW;

  if (!identity_holds(m, r, n, AT, G, BT)) return NOVA_ERR_VERIFY_FAILED;

  nova_plan* pl = new (std::nothrow) nova_plan();
  if (!pl) return NOVA_ERR_INVALID_ARG;
  std::memset(pl, 0, sizeof(*pl));
  pl->m = m; pl->r = r; pl->n = n; pl->mode = mode; pl->coef = coef;
  for (int i = 0; i < n; ++i) pl->points[i] = points[i];
  for (int i = 0; i < m * n; ++i) pl->AT[i] = rat_to_double(AT[i]);
  for (int i = 0; i < n * r; ++i) pl->G[i] = rat_to_double(G[i]);
  for (int i = 0; i < n * n; ++i) pl->BT[i] = rat_to_double(BT[i]);
  pl->rat_fits = 1;
  for (int i = 0; i < m * n; ++i) if (!fits64(AT[i], &pl->AT_rat[i])) pl->rat_fits = 0;
  for (int i = 0; i < n * r; ++i) if (!fits64(G[i], &pl->G_rat[i])) pl->rat_fits = 0;
  for (int i = 0; i < n * n; ++i) if (!fits64(BT[i], &pl->BT_rat[i])) pl->rat_fits = 0;
  {
    std::vector<double> A(n * m), Gd(pl->G, pl->G + n * r), Bd(n * n);
    for (int i = 0; i < m; ++i)
      for (int p = 0; p < n; ++p) A[p * m + i] = pl->AT[i * n + p];          // A = (A^T)^T, n x m
    for (int p = 0; p < n; ++p)
      for (int j = 0; j < n; ++j) Bd[j * n + p] = pl->BT[p * n + j];
    pl->kappa2_mat[0] = cond2(A, m, n, &pl->norm2_mat[0]);
    pl->kappa2_mat[1] = cond2(Gd, r, n, &pl->norm2_mat[1]);
    pl->kappa2_mat[2] = cond2(Bd, n, n, &pl->norm2_mat[2]);
  }

  const bool through_half = (mode == NOVA_FP16_F32ACC && coef == NOVA_COEF_ROUND_TO_MODE);
  auto rnd = [&](double v) { return through_half ? round_through_half(v) : (float)v; };
  for (int i = 0; i < m; ++i)
    for (int p = 0; p < n; ++p) pl->coefs.AT[i][p] = rnd(pl->AT[i * n + p]);
  for (int p = 0; p < n; ++p)
    for (int k = 0; k < r; ++k) pl->coefs.G[p][k] = rnd(pl->G[p * r + k]);
  for (int p = 0; p < n; ++p)
    for (int j = 0; j < n; ++j) pl->coefs.BT[p][j] = rnd(pl->BT[p * n + j]);

  // Internal point order and kernel tables.
  for (int i = 0; i < n; ++i) pl->perm[i] = i;
  pl->symmetric = 0;
  {
    int order[nova::kMaxN], cnt = 0, zero_at = -1;
    bool used[nova::kMaxN] = {};
    for (int i = 0; i < nf; ++i)
      if (al[i].n == 0) zero_at = i;
    bool sym = zero_at >= 0 && (nf % 2) == 1;
    if (sym) {
      order[cnt++] = zero_at;
      used[zero_at] = true;
      for (int i = 0; i < nf && sym; ++i) {
        if (used[i]) continue;
        int mate = -1;
        for (int j = 0; j < nf; ++j)
          if (!used[j] && j != i && al[j].d == al[i].d && al[j].n == -al[i].n) mate = j;
        if (mate < 0) { sym = false; break; }
        const int pos = al[i].n > 0 ? i : mate, neg = al[i].n > 0 ? mate : i;
        order[cnt++] = pos;
        order[cnt++] = neg;
        used[i] = used[mate] = true;
      }
      if (sym) order[cnt++] = n - 1;
    }
    if (sym && cnt == n)
      for (int i = 0; i < n; ++i) pl->perm[i] = order[i];
    nova::Coefs& k = pl->kcoefs;
    for (int i = 0; i < m; ++i)
      for (int p = 0; p < n; ++p) k.AT[i][p] = pl->coefs.AT[i][pl->perm[p]];
    for (int p = 0; p < n; ++p) {
      for (int kk = 0; kk < r; ++kk) k.G[p][kk] = pl->coefs.G[pl->perm[p]][kk];
      for (int j = 0; j < n; ++j) k.BT[p][j] = pl->coefs.BT[pl->perm[p]][j];
    }
    // The SYM kernel paths skip the structural zeros and share even/odd partial sums of a
    // +-pair; they are used only if the rounded tables have exactly that structure.
    if (sym && cnt == n) {
      bool ok = true;
      for (int j = 0; j < n; ++j) {
        if ((j & 1) && k.BT[0][j] != 0.f) ok = false;
        if (!(j & 1) && k.BT[n - 1][j] != 0.f) ok = false;
      }
      for (int i = 0; i < m; ++i) {
        if (k.AT[i][0] != (i == 0 ? 1.f : 0.f)) ok = false;
        if (k.AT[i][n - 1] != (i == m - 1 ? 1.f : 0.f)) ok = false;
      }
      for (int q = 1; q + 1 < n - 1; q += 2) {
        if (k.BT[q][n - 1] != 0.f || k.BT[q + 1][n - 1] != 0.f) ok = false;
        for (int j = 0; j < n; ++j)
          if (k.BT[q + 1][j] != ((j & 1) ? -k.BT[q][j] : k.BT[q][j])) ok = false;
        for (int i = 0; i < m; ++i)
          if (k.AT[i][q + 1] != ((i & 1) ? -k.AT[i][q] : k.AT[i][q])) ok = false;
      }
      pl->symmetric = ok ? 1 : 0;
    }
  }

  std::vector<double> V(nf * nf);
  for (int i = 0; i < nf; ++i) {
    double a = rat_to_double(al[i]), pw = 1.0;
    for (int j = 0; j < nf; ++j) { V[i * nf + j] = pw; pw *= a; }
  }
  pl->kappa2_V = cond2(V, nf);

  // One device status word, if a device is present (host-only use is allowed).
  pl->status_dev = nullptr;
  pl->device = -1;
  int ndev = 0;
  if (cudaGetDeviceCount(&ndev) == cudaSuccess && ndev > 0) {
    int dev = 0;
    if (cudaGetDevice(&dev) == cudaSuccess) {
      int* w = nullptr;
      if (cudaMalloc((void**)&w, sizeof(int)) == cudaSuccess) {
        cudaMemset(w, 0, sizeof(int));
        pl->status_dev = w;
        pl->device = dev;
        cudaDeviceGetAttribute(&pl->sm_count, cudaDevAttrMultiProcessorCount, dev);
        cudaDeviceGetAttribute(&pl->l2_bytes, cudaDevAttrL2CacheSize, dev);
      }
      if (pl->status_dev && pl->sm_count > 0) {
        unsigned long long* pd = nullptr;
        const size_t nb = (size_t)pl->sm_count * 8 * sizeof(unsigned long long);
        if (cudaMalloc((void**)&pd, nb) == cudaSuccess) {
          cudaMemset(pd, 0, nb);
          pl->prof_dev = pd;
        }
      }
      // Kronecker table of the tensor-core input transform (half mode, half-rounded tables).
      if (pl->status_dev && mode == NOVA_FP16_F32ACC && coef == NOVA_COEF_ROUND_TO_MODE) {
        std::vector<unsigned short> img(nova::kron_table_halves(n));
        nova::build_kron_table(pl, img.data());
        void* kd = nullptr;
        if (cudaMalloc(&kd, img.size() * 2) == cudaSuccess) {
          if (cudaMemcpy(kd, img.data(), img.size() * 2, cudaMemcpyHostToDevice) == cudaSuccess) pl->kron_dev = kd;
          else cudaFree(kd);
        }
      }
    }
  }
  (void)cudaGetLastError();
  *out = pl;
  return NOVA_OK;
}

}  // namespace

extern "C" int nova_plan_create(int m, int r, const nova_rat* points, int n, int mode, int coef,
                                nova_plan** out) {
  return create_impl(m, r, points, n, nullptr, nullptr, mode, coef, out);
}

extern "C" int nova_plan_create_scaled(int m, int r, const nova_rat* points, int n, const nova_rat* scale_G,
                                       const nova_rat* scale_B, int mode, int coef, nova_plan** out) {
  return create_impl(m, r, points, n, scale_G, scale_B, mode, coef, out);
}

extern "C" int nova_snap_to_rational(double x, int max_den, nova_rat* out) {
  if (!out || max_den < 1 || max_den > 4096 || !std::isfinite(x)) return NOVA_ERR_INVALID_ARG;
  // Candidates lie in [-5, 5], so clamping x to [-6, 6] changes no answer; and an |x| below
  // 2^-30 is closer to 0 than to the smallest non-zero candidate (>= 2^-12) with no tie possible.
  if (x > 6) x = 6;
  if (x < -6) x = -6;
  if (std::fabs(x) < std::ldexp(1.0, -30)) { out->num = 0; out->den = 1; return NOVA_OK; }
  // x = X / 2^s exactly, |X| < 2^53, s <= 83.  |x - a/b| = |X b - a 2^s| / (b 2^s); two
  // candidates compare by cross-multiplication, which stays below 2^111.
  int e;
  const double fr = std::frexp(x, &e);
  i128 X = (i128)(long long)std::ldexp(fr, 53);
  int s = 53 - e;
  while (s < 0) { X *= 2; ++s; }
  // For a denominator b the closest numerator is one of the two integers around x b (exactly:
  // floor(X b / 2^s) and its successor), clamped to [-5b, 5b]; the winner over all b is found by
  // cross-multiplication.  Ties follow the order of the definition's enumeration (Algorithm 2:
  // b ascending, then a ascending, strict "<"): the smaller b, then the smaller a, stays.
  long long best_a = 0, best_b = 1;
  i128 best_num = -1;
  for (long long b = 1; b <= max_den; ++b) {
    const i128 Xb = X * b;
    i128 fl = Xb >> s;                                  // arithmetic shift: floor for negative values too
    long long cand[2] = {(long long)fl, (long long)fl + 1};
    for (int t = 0; t < 2; ++t) {
      long long a = cand[t];
      if (a < -5 * b) a = -5 * b;
      if (a > 5 * b) a = 5 * b;
      if (t == 1 && a == cand[0]) continue;             // both clamped to the same end
      cand[t] = a;
      i128 num = Xb - ((i128)a << s);
      if (num < 0) num = -num;
      if (best_num < 0 || num * best_b < best_num * b) { best_num = num; best_a = a; best_b = b; }
    }
  }
  const long long g = (long long)gcd128(best_a, best_b);
  out->num = best_a / (g ? g : 1);
  out->den = best_b / (g ? g : 1);
  return NOVA_OK;
}

extern "C" int nova_symmetric_search(int n_finite, int max_den, int max_abs, nova_rat* points_out,
                                     double* kappa2_out) {
  if (!points_out || n_finite < 2 || n_finite >= nova::kMaxN || max_den < 1 || max_den > 64 || max_abs < 1 ||
      max_abs > 5)
    return NOVA_ERR_INVALID_ARG;
  // candidates: the positive fractions a/b in lowest terms, b <= max_den, a/b <= max_abs, ascending
  std::vector<std::pair<int, int>> cand;
  for (int b = 1; b <= max_den; ++b)
    for (int a = 1; a <= max_abs * b; ++a)
      if (gcd128(a, b) == 1) cand.push_back({a, b});
  std::sort(cand.begin(), cand.end(), [](const std::pair<int, int>& x, const std::pair<int, int>& y) {
    return (long long)x.first * y.second < (long long)y.first * x.second;
  });
  const int pairs = n_finite / 2, nc = (int)cand.size();
  if (pairs > nc) return NOVA_ERR_INVALID_ARG;
  double combos = 1;
  for (int i = 0; i < pairs; ++i) combos = combos * (nc - i) / (i + 1);
  if (combos > 4e6) return NOVA_ERR_UNSUPPORTED;       // keep the enumeration to seconds
  std::vector<int> idx(pairs), best_idx;
  for (int i = 0; i < pairs; ++i) idx[i] = i;
  double best = INFINITY;
  std::vector<double> V(n_finite * n_finite), pts(n_finite);
  for (;;) {
    int k = 0;
    if (n_finite & 1) pts[k++] = 0.0;
    for (int i = 0; i < pairs; ++i) {
      const double p = (double)cand[idx[i]].first / (double)cand[idx[i]].second;
      pts[k++] = p;
      pts[k++] = -p;
    }
    for (int i = 0; i < n_finite; ++i) {
      double pw = 1.0;
      for (int j = 0; j < n_finite; ++j) { V[i * n_finite + j] = pw; pw *= pts[i]; }
    }
    const double kap = cond2(V, n_finite);
    if (kap < best) { best = kap; best_idx = idx; }
    int i = pairs - 1;                                  // next combination in lexicographic order
    while (i >= 0 && idx[i] == nc - pairs + i) --i;
    if (i < 0) break;
    ++idx[i];
    for (int j = i + 1; j < pairs; ++j) idx[j] = idx[j - 1] + 1;
  }
  int k = 0;
  if (n_finite & 1) { points_out[k].num = 0; points_out[k].den = 1; ++k; }
  for (int i = 0; i < pairs; ++i) {
    const std::pair<int, int>& c = cand[best_idx[i]];
    points_out[k].num = c.first; points_out[k].den = c.second; ++k;
    points_out[k].num = -c.first; points_out[k].den = c.second; ++k;
  }
  points_out[k].num = 1;
  points_out[k].den = 0;                                // the point at infinity, last
  if (kappa2_out) *kappa2_out = best;
  return NOVA_OK;
}

extern "C" int nova_plan_create_f64(int m, int r, const double* finite_points, int n_finite, int max_den,
                                    int mode, int coef, nova_plan** out) {
  if (out) *out = nullptr;
  if (!finite_points || !out || n_finite < 1 || n_finite >= nova::kMaxN) return NOVA_ERR_INVALID_ARG;
  nova_rat pts[nova::kMaxN];
  for (int i = 0; i < n_finite; ++i) {
    const int st = nova_snap_to_rational(finite_points[i], max_den, &pts[i]);
    if (st != NOVA_OK) return st;
  }
  pts[n_finite].num = 1;
  pts[n_finite].den = 0;
  return create_impl(m, r, pts, n_finite + 1, nullptr, nullptr, mode, coef, out);
}

extern "C" int nova_verify_decomposition(int m, int r, int n, const nova_rat* AT, const nova_rat* G,
                                         const nova_rat* BT) {
  if (!AT || !G || !BT || m < 1 || r < 1 || n != m + r - 1 || n > 64) return NOVA_ERR_INVALID_ARG;
  Arith ar;
  std::vector<Rat> a(m * n), g(n * r), b(n * n);
  auto conv = [&](const nova_rat* src, std::vector<Rat>& dst) {
    for (size_t i = 0; i < dst.size(); ++i) {
      if (src[i].den <= 0) return false;
      dst[i] = ar.norm(src[i].num, src[i].den);
    }
    return true;
  };
  if (!conv(AT, a) || !conv(G, g) || !conv(BT, b)) return NOVA_ERR_INVALID_ARG;
  return identity_holds(m, r, n, a, g, b) ? NOVA_OK : NOVA_ERR_VERIFY_FAILED;
}

extern "C" int nova_plan_get_matrices_rational(const nova_plan* p, nova_rat* AT, nova_rat* G, nova_rat* BT) {
  if (!p) return NOVA_ERR_INVALID_ARG;
  if (!p->rat_fits) return NOVA_ERR_RATIONAL_OVERFLOW;
  if (AT) std::memcpy(AT, p->AT_rat, sizeof(nova_rat) * p->m * p->n);
  if (G) std::memcpy(G, p->G_rat, sizeof(nova_rat) * p->n * p->r);
  if (BT) std::memcpy(BT, p->BT_rat, sizeof(nova_rat) * p->n * p->n);
  return NOVA_OK;
}

extern "C" int nova_plan_kappa_matrices(const nova_plan* p, double* kappa2, double* norm2) {
  if (!p) return NOVA_ERR_INVALID_ARG;
  for (int i = 0; i < 3; ++i) {
    if (kappa2) kappa2[i] = p->kappa2_mat[i];
    if (norm2) norm2[i] = p->norm2_mat[i];
  }
  return NOVA_OK;
}

extern "C" void nova_plan_destroy(nova_plan* plan) {
  if (!plan) return;
  if (plan->status_dev) cudaFree(plan->status_dev);
  if (plan->kron_dev) cudaFree(plan->kron_dev);
  if (plan->prof_dev) cudaFree(plan->prof_dev);
  delete plan;
}

extern "C" int nova_plan_get_matrices(const nova_plan* p, double* AT, double* G, double* BT) {
  if (!p) return NOVA_ERR_INVALID_ARG;
  if (AT) std::memcpy(AT, p->AT, sizeof(double) * p->m * p->n);
  if (G) std::memcpy(G, p->G, sizeof(double) * p->n * p->r);
  if (BT) std::memcpy(BT, p->BT, sizeof(double) * p->n * p->n);
  return NOVA_OK;
}

extern "C" int nova_plan_get_device_tables(const nova_plan* p, float* AT, float* G, float* BT) {
  if (!p) return NOVA_ERR_INVALID_ARG;
  for (int i = 0; i < p->m; ++i)
    for (int q = 0; q < p->n; ++q)
      if (AT) AT[i * p->n + q] = p->coefs.AT[i][q];
  for (int q = 0; q < p->n; ++q)
    for (int k = 0; k < p->r; ++k)
      if (G) G[q * p->r + k] = p->coefs.G[q][k];
  for (int q = 0; q < p->n; ++q)
    for (int j = 0; j < p->n; ++j)
      if (BT) BT[q * p->n + j] = p->coefs.BT[q][j];
  return NOVA_OK;
}

extern "C" int nova_plan_frequency_order(const nova_plan* p, int* perm, int* symmetric) {
  if (!p) return NOVA_ERR_INVALID_ARG;
  if (perm)
    for (int i = 0; i < p->n; ++i) perm[i] = p->perm[i];
  if (symmetric) *symmetric = p->symmetric;
  return NOVA_OK;
}

extern "C" int nova_plan_kappa(const nova_plan* p, double* k) {
  if (!p || !k) return NOVA_ERR_INVALID_ARG;
  *k = p->kappa2_V;
  return NOVA_OK;
}

extern "C" const char* nova_status_string(int s) {
  switch (s) {
    case NOVA_OK: return "ok";
    case NOVA_ERR_INVALID_ARG: return "invalid argument";
    case NOVA_ERR_NO_INFINITY: return "point set has no point at infinity";
    case NOVA_ERR_MULTIPLE_INFINITY: return "point at infinity must appear exactly once, last";
    case NOVA_ERR_DUPLICATE_POINT: return "finite points must be distinct";
    case NOVA_ERR_RATIONAL_OVERFLOW: return "exact rational arithmetic overflowed 127 bits";
    case NOVA_ERR_VERIFY_FAILED: return "exact decomposition identity failed";
    case NOVA_ERR_UNSUPPORTED: return "unsupported configuration";
    case NOVA_ERR_CUDA: return "CUDA call failed or no device";
    case NOVA_ERR_DEVICE_TIMEOUT: return "a bounded device-side wait expired";
    case NOVA_ERR_WORKSPACE: return "workspace too small or misaligned";
    case NOVA_ERR_STATIC_LIMIT: return "problem exceeds the built-in scratch of the no-allocation entry point";
    default: return "unknown status";
  }
}
