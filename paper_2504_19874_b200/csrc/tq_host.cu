// Host-side set-up of TurboQuant's global parameters: the Lloyd-Max codebook of Eq. (4)
// for the coordinate density of Lemma 1, and the seeded Gaussian / orthogonal matrices of
// Section 3.1 and Definition 1.  Everything here is fp64 and runs once per (d, b, seed).
#include "tq_internal.h"

#include <algorithm>
#include <atomic>
#include <cmath>
#include <cstdlib>
#include <cstring>
#include <vector>

namespace tq {

static thread_local char g_err[512] = "";

static std::atomic<unsigned long long> g_launches{0};
void count_launches(int k) { g_launches.fetch_add((unsigned long long)k, std::memory_order_relaxed); }

bool log_enabled() {
  static const bool on = [] {
    const char* v = std::getenv("TQ_LOG");
    return v != nullptr && v[0] != '\0' && !(v[0] == '0' && v[1] == '\0');
  }();
  return on;
}

void set_error(const char* fmt, ...) {
  va_list ap;
  va_start(ap, fmt);
  vsnprintf(g_err, sizeof(g_err), fmt, ap);
  va_end(ap);
}

// ---------------------------------------------------------------------------------------
// Lemma 1 with x = sin(theta): f_X(x) dx = K cos^(d-2)(theta) dtheta, smooth for every d >= 2.
// Cell mass by composite Gauss-Legendre in theta; cell first moment in closed form:
//   int x f_X dx = -K (1 - x^2)^((d-1)/2) / (d - 1) = -K cos^(d-1)(theta) / (d - 1).
// ---------------------------------------------------------------------------------------
namespace {

struct GaussLegendre {
  static constexpr int kOrder = 20;
  double x[kOrder], w[kOrder];
  GaussLegendre() {
    // Newton iteration on the Legendre polynomial P_n.
    const int n = kOrder;
    for (int i = 0; i < n; ++i) {
      double z = std::cos(M_PI * (i + 0.75) / (n + 0.5));
      double dp = 1.0;
      for (int it = 0; it < 100; ++it) {
        double p0 = 1.0, p1 = z;
        for (int k = 2; k <= n; ++k) {
          double p2 = ((2.0 * k - 1.0) * z * p1 - (k - 1.0) * p0) / k;
          p0 = p1;
          p1 = p2;
        }
        dp = n * (z * p1 - p0) / (z * z - 1.0);
        double dz = p1 / dp;
        z -= dz;
        if (std::fabs(dz) < 1e-16) break;
      }
      x[i] = z;
      w[i] = 2.0 / ((1.0 - z * z) * dp * dp);
    }
  }
};

double cos_power_integral(double t0, double t1, double expo, const GaussLegendre& gl) {
  // int_{t0}^{t1} cos(theta)^expo dtheta, split into panels no wider than the peak's width.
  if (t1 <= t0) return 0.0;
  const double width = 0.5 / std::sqrt(expo + 1.0);
  int panels = (int)std::ceil((t1 - t0) / width);
  panels = std::max(1, std::min(panels, 4096));
  const double h = (t1 - t0) / panels;
  double tot = 0.0;
  for (int p = 0; p < panels; ++p) {
    const double a = t0 + p * h, mid = a + 0.5 * h;
    double s = 0.0;
    for (int i = 0; i < GaussLegendre::kOrder; ++i) {
      const double th = mid + 0.5 * h * gl.x[i];
      const double c = std::cos(th);
      s += gl.w[i] * (expo == 0.0 ? 1.0 : std::exp(expo * std::log(c)));
    }
    tot += 0.5 * h * s;
  }
  return tot;
}

}  // namespace

int lloyd_max(int d, int bits, double* c_out) {
  const int k = 1 << bits;
  if (k == 1) {
    c_out[0] = 0.0;
    return TQ_OK;
  }
  static const GaussLegendre gl;
  const double expo = d - 2.0;
  // Beyond theta_max the density is below 1e-40 of its peak; never past pi/2.
  const double theta_max = (d > 2) ? std::min(M_PI / 2, std::sqrt(190.0 / expo)) : M_PI / 2;
  const double sigma = 1.0 / std::sqrt((double)d);
  std::vector<double> c(k), t(k + 1), nc(k);
  for (int i = 0; i < k; ++i) {
    double v = (2.0 * i + 1.0 - k) / k * 2.5 * sigma;
    c[i] = std::max(-0.95, std::min(0.95, v));
  }
  // Mass and first moment share the constant K, which cancels in the centroid.
  for (int it = 0; it < 200000; ++it) {
    t[0] = -theta_max;
    t[k] = theta_max;
    for (int i = 1; i < k; ++i) t[i] = std::asin(0.5 * (c[i - 1] + c[i]));
    for (int i = 0; i < k; ++i) {
      const double mass = cos_power_integral(t[i], t[i + 1], expo, gl);
      const double ca = std::cos(t[i]), cb = std::cos(t[i + 1]);
      const double ga = (i == 0) ? 0.0 : std::exp((expo + 1.0) * std::log(ca));
      const double gb = (i == k - 1) ? 0.0 : std::exp((expo + 1.0) * std::log(cb));
      nc[i] = (ga - gb) / (expo + 1.0) / mass;
    }
    double delta = 0.0;
    for (int i = 0; i < k; ++i) {
      const double sym = 0.5 * (nc[i] - nc[k - 1 - i]);  // the density is even
      delta = std::max(delta, std::fabs(sym - c[i]));
      c[i] = sym;
    }
    if (delta < 1e-14) {
      for (int i = 0; i < k; ++i) c_out[i] = c[i];
      return TQ_OK;
    }
  }
  set_error("tq_codebook: Lloyd-Max did not converge for d=%d bits=%d", d, bits);
  return TQ_ERR_NOT_CONVERGED;
}

// p_l = mass of the l-th cell (boundaries halfway between neighbouring centroids) under the density of Lemma 1:
// the probability of index value l (entropy-coding paragraph of Section 3.1).
int cell_masses(int d, int levels, const float* centroids, double* p_out) {
  static const GaussLegendre gl;
  const double expo = d - 2.0;
  std::vector<double> t(levels + 1);
  t[0] = -M_PI / 2;
  t[levels] = M_PI / 2;
  for (int i = 1; i < levels; ++i) {
    const double b = 0.5 * ((double)centroids[i - 1] + (double)centroids[i]);
    if (!(b > -1.0 && b < 1.0) || !(centroids[i] > centroids[i - 1])) {
      set_error("cell_masses: centroids must be strictly ascending inside (-1, 1)");
      return TQ_ERR_INVALID_ARG;
    }
    t[i] = std::asin(b);
  }
  double tot = 0.0;
  for (int i = 0; i < levels; ++i) {
    p_out[i] = cos_power_integral(t[i], t[i + 1], expo, gl);
    tot += p_out[i];
  }
  for (int i = 0; i < levels; ++i) p_out[i] /= tot;
  return TQ_OK;
}

// ---------------------------------------------------------------------------------------
// Counter-based Gaussian draws (documented in tq.h so that anyone can reproduce a matrix).
// ---------------------------------------------------------------------------------------
static inline uint64_t mix64(uint64_t x) {
  x ^= x >> 30;
  x *= 0xBF58476D1CE4E5B9ull;
  x ^= x >> 27;
  x *= 0x94D049BB133111EBull;
  x ^= x >> 31;
  return x;
}

static inline double gaussian_at(uint64_t seed_mixed, uint64_t e) {
  const uint64_t G = 0x9E3779B97F4A7C15ull;
  const uint64_t h1 = mix64(seed_mixed + (2 * e) * G);
  const uint64_t h2 = mix64(seed_mixed + (2 * e + 1) * G);
  const double u1 = ((double)(h1 >> 11) + 0.5) * 0x1.0p-53;
  const double u2 = (double)(h2 >> 11) * 0x1.0p-53;
  return std::sqrt(-2.0 * std::log(u1)) * std::cos(2.0 * M_PI * u2);
}

void gaussian_matrix(int d, uint64_t seed, double* out /* row-major d*d */) {
  const uint64_t sm = mix64(seed + 0x9E3779B97F4A7C15ull);
#pragma omp parallel for schedule(static)
  for (int64_t e = 0; e < (int64_t)d * d; ++e) out[e] = gaussian_at(sm, (uint64_t)e);
}

// Householder QR of the d x d matrix whose COLUMNS are col[j] (each contiguous, length d).
// Returns Q (columns, contiguous) with the sign convention R_kk > 0.
static void householder_q(int d, std::vector<double>& a /* d*d, column j at a[j*d] */,
                          std::vector<double>& q) {
  std::vector<double> vs((size_t)d * d, 0.0);  // reflector k stored at vs[k*d + k ..]
  std::vector<double> rdiag(d);
  for (int k = 0; k < d; ++k) {
    double* x = &a[(size_t)k * d];
    double nrm2 = 0.0;
    for (int i = k; i < d; ++i) nrm2 += x[i] * x[i];
    const double nrm = std::sqrt(nrm2);
    double* v = &vs[(size_t)k * d];
    if (nrm == 0.0) {
      rdiag[k] = 0.0;
      continue;
    }
    const double alpha = (x[k] >= 0.0) ? -nrm : nrm;  // R_kk
    rdiag[k] = alpha;
    double vn2 = 0.0;
    for (int i = k; i < d; ++i) {
      v[i] = x[i] - (i == k ? alpha : 0.0);
      vn2 += v[i] * v[i];
    }
    const double inv = 1.0 / std::sqrt(vn2);
    for (int i = k; i < d; ++i) v[i] *= inv;
#pragma omp parallel for schedule(static)
    for (int j = k + 1; j < d; ++j) {
      double* y = &a[(size_t)j * d];
      double dot = 0.0;
      for (int i = k; i < d; ++i) dot += v[i] * y[i];
      dot *= 2.0;
      for (int i = k; i < d; ++i) y[i] -= dot * v[i];
    }
  }
  // Q = H_0 H_1 ... H_{d-1}: apply the reflectors in reverse order to the identity.
  q.assign((size_t)d * d, 0.0);
  for (int j = 0; j < d; ++j) q[(size_t)j * d + j] = 1.0;
  for (int k = d - 1; k >= 0; --k) {
    const double* v = &vs[(size_t)k * d];
#pragma omp parallel for schedule(static)
    for (int j = k; j < d; ++j) {
      double* y = &q[(size_t)j * d];
      double dot = 0.0;
      for (int i = k; i < d; ++i) dot += v[i] * y[i];
      dot *= 2.0;
      for (int i = k; i < d; ++i) y[i] -= dot * v[i];
    }
  }
  for (int j = 0; j < d; ++j)
    if (rdiag[j] < 0.0) {
      double* y = &q[(size_t)j * d];
      for (int i = 0; i < d; ++i) y[i] = -y[i];
    }
}

}  // namespace tq

using namespace tq;

extern "C" const char* tq_last_error(void) { return g_err; }

extern "C" uint64_t tq_launch_count(void) { return g_launches.load(std::memory_order_relaxed); }

extern "C" size_t tq_idx_row_bytes(int d, int bits) {
  if (d <= 0 || bits <= 0) return 0;
  size_t raw = ((size_t)d * bits + 7) / 8;
  if (raw >= 16) return (raw + 15) / 16 * 16;
  size_t p = 4;
  while (p < raw) p *= 2;
  return p;
}

extern "C" size_t tq_qjl_row_bytes(int d) { return tq_idx_row_bytes(d, 1); }

extern "C" int tq_codebook(int d, int bits, float* centroids, float* boundaries) {
  if (!centroids) {
    set_error("tq_codebook: centroids is NULL");
    return TQ_ERR_INVALID_ARG;
  }
  if (d < 2 || d > TQ_MAX_D || bits < 0 || bits > 4) {
    set_error("tq_codebook: unsupported d=%d bits=%d (d in 2..%d, bits in 0..4)", d, bits, TQ_MAX_D);
    return TQ_ERR_UNSUPPORTED;
  }
  double c[16];
  int rc = lloyd_max(d, bits, c);
  if (rc != TQ_OK) return rc;
  const int k = 1 << bits;
  for (int i = 0; i < k; ++i) centroids[i] = (float)c[i];
  if (boundaries)
    for (int i = 0; i + 1 < k; ++i) boundaries[i] = 0.5f * (centroids[i] + centroids[i + 1]);
  return TQ_OK;
}

extern "C" int tq_rotation(int d, uint64_t seed, int kind, float* out) {
  if (!out) {
    set_error("tq_rotation: out is NULL");
    return TQ_ERR_INVALID_ARG;
  }
  if (d < 1 || d > TQ_MAX_D || (kind != TQ_ORTHOGONAL && kind != TQ_GAUSSIAN)) {
    set_error("tq_rotation: unsupported d=%d kind=%d", d, kind);
    return TQ_ERR_UNSUPPORTED;
  }
  std::vector<double> g((size_t)d * d);
  gaussian_matrix(d, seed, g.data());
  if (kind == TQ_GAUSSIAN) {
    for (size_t e = 0; e < g.size(); ++e) out[e] = (float)g[e];
    return TQ_OK;
  }
  std::vector<double> cols((size_t)d * d), q;
  for (int i = 0; i < d; ++i)
    for (int j = 0; j < d; ++j) cols[(size_t)j * d + i] = g[(size_t)i * d + j];
  householder_q(d, cols, q);
  for (int i = 0; i < d; ++i)
    for (int j = 0; j < d; ++j) out[(size_t)i * d + j] = (float)q[(size_t)j * d + i];
  return TQ_OK;
}
