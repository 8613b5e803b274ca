// Host-side entry points: rotation generator, Lloyd-Max codebooks, derived tables, size queries.
#include <algorithm>
#include <atomic>
#include <cmath>
#include <cstring>
#include <vector>

#include "pq_common.cuh"

namespace {

const double kPi = 3.14159265358979323846264338327950288;

// ---- counter-based Gaussian generator (splitmix64 + Box-Muller) --------------------------
inline uint64_t splitmix64(uint64_t x) {
  x += 0x9E3779B97F4A7C15ull;
  x = (x ^ (x >> 30)) * 0xBF58476D1CE4E5B9ull;
  x = (x ^ (x >> 27)) * 0x94D049BB133111EBull;
  return x ^ (x >> 31);
}
inline double uniform01(uint64_t seed, uint64_t idx) {  // in (0, 1)
  const uint64_t bits = splitmix64(splitmix64(seed) ^ (idx * 0xD6E8FEB86659FD93ull + 0x2545F4914F6CDD1Dull));
  return ((double)(bits >> 11) + 0.5) * (1.0 / 9007199254740992.0);
}
inline double gaussian(uint64_t seed, uint64_t idx) {
  const double u1 = uniform01(seed, 2 * idx), u2 = uniform01(seed, 2 * idx + 1);
  return std::sqrt(-2.0 * std::log(u1)) * std::cos(2.0 * kPi * u2);
}

// ---- Lemma 2 densities and Simpson quadrature --------------------------------------------
inline double density_unnorm(int level, double psi) {
  if (level == 1) return 1.0;
  const int k = 1 << (level - 1);
  return std::pow(std::sin(2.0 * psi), k - 1);
}
// Integrals of f and psi*f over [lo, hi] by composite Simpson (the integrand is a polynomial
// in sin/cos, so 4096 panels are far beyond float64 accuracy).
inline void cell_moments(int level, double lo, double hi, double* m0, double* m1) {
  const int n = 4096;
  const double h = (hi - lo) / n;
  double s0 = 0.0, s1 = 0.0;
  for (int i = 0; i <= n; ++i) {
    const double p = lo + h * i;
    const double w = (i == 0 || i == n) ? 1.0 : ((i & 1) ? 4.0 : 2.0);
    const double f = density_unnorm(level, p);
    s0 += w * f;
    s1 += w * f * p;
  }
  *m0 = s0 * h / 3.0;
  *m1 = s1 * h / 3.0;
}

// ---- level-1 decision table for an arbitrary codebook ---------------------------------------
// The plane is cut into octants by the signs of a, b and |b| > |a|; inside octant o the angle is
// psi = B_o + D_o * phi with phi = atan(t), t = min(|a|,|b|) / max(|a|,|b|) in [0, 1].  The 16 rays that separate
// the level-1 cells (the 15 boundaries and the ray at 0 = 2 pi between code 15 and code 0) are expressed in the
// octant's own coordinate continued past its edges, t_c = tan(D_o (beta - B_o)), for every ray within
// [-pi/4, atan 2] of the octant's first edge: a point whose computed t is off by less than 1 is, in this
// coordinate, still on the same side of every ray it was not moved across.
// A cell stores one value tau and two codes such that for EVERY t of the cell
//   (1) |t - tau| is at most the distance from t to every ray (in t_c), and
//   (2) the code is `lo` for t < tau and `hi` for t > tau,
// so the kernel decides with one comparison and certifies with one distance.  A cell that cannot offer both
// (two rays inside or next to it) stores NaN and every decision in it is taken in float64.
struct L1Ray {
  double t;
  int below, above;  // codes on the sides t_c < t and t_c > t
};

int l1_code_of_angle(const double* bnd, double psi) {
  int c = 0;
  for (int k = 0; k < 15; ++k) c += psi > bnd[k];
  return c;
}

bool build_l1_cells(const double* bnd, uint2 (*cells)[pq::kL1Cells]) {
  const double kHalfPi = 0.5 * kPi;
  for (int o = 0; o < 8; ++o) {
    const int sb = (o >> 2) & 1, sa = (o >> 1) & 1, sw = o & 1;
    double B, D;
    if (!sa && !sb) { B = sw ? kHalfPi : 0.0; D = sw ? -1.0 : 1.0; }
    else if (sa && !sb) { B = sw ? kHalfPi : kPi; D = sw ? 1.0 : -1.0; }
    else if (sa && sb) { B = sw ? 3.0 * kHalfPi : kPi; D = sw ? -1.0 : 1.0; }
    else { B = sw ? 3.0 * kHalfPi : 2.0 * kPi; D = sw ? 1.0 : -1.0; }
    std::vector<L1Ray> rays;
    for (int j = 0; j < 16; ++j) {
      const double ang = j == 0 ? 0.0 : bnd[j - 1];
      double phi = std::remainder(D * (ang - B), 2.0 * kPi);  // in [-pi, pi]
      if (phi < -0.25 * kPi - 0.02 || phi > std::atan(2.0) + 0.02) continue;
      const int below = (j + 15) & 15, above = j;  // codes at smaller / larger psi
      rays.push_back({std::tan(phi), D > 0 ? below : above, D > 0 ? above : below});
    }
    for (int c = 0; c < pq::kL1Cells; ++c) {
      // the kernel's cell index is floor(m / 8), m = t * kL1CellScale * 8 rounded to an integer
      const double scale = (double)pq::kL1CellScale;
      const double lo = std::fmax(0.0, (c - 1.0 / 16.0) / scale - 1e-6), hi = std::fmin(1.0, (c + 15.0 / 16.0) / scale + 1e-6);
      const double w = hi - lo;
      int n_in = 0, in_idx = -1;
      double dA = 1e30, dB = 1e30;  // distance from the cell to the nearest ray below / above it
      for (size_t i = 0; i < rays.size(); ++i) {
        if (rays[i].t >= lo && rays[i].t <= hi) { ++n_in; in_idx = (int)i; }
        else if (rays[i].t < lo) dA = std::fmin(dA, lo - rays[i].t);
        else dB = std::fmin(dB, rays[i].t - hi);
      }
      float tau;
      int code_lo, code_hi;
      if (n_in == 0) {
        // no ray inside: a virtual tau outside the cell whose distance stays below both neighbours' for every t
        const double mA = std::fmin(dA, dB - w), mB = std::fmin(dB, dA - w);
        const double t = mA >= mB ? lo - std::fmin(mA, 1.0) : hi + std::fmin(mB, 1.0);
        const double mid = 0.5 * (lo + hi);
        double psi = B + D * std::atan(mid);
        if (psi >= 2.0 * kPi) psi -= 2.0 * kPi;
        if (psi < 0.0) psi += 2.0 * kPi;
        code_lo = code_hi = l1_code_of_angle(bnd, psi);
        tau = (float)std::fmin(1.0, std::fmax(0.0, t));
        if ((mA >= mB ? mA : mB) <= 0.0) tau = std::nanf("");  // a ray touches the cell from both sides
      } else if (n_in == 1) {
        const double tm = rays[in_idx].t;
        const double far = std::fmax(tm - lo, hi - tm);  // largest distance from a t of the cell to the ray
        tau = (dA >= far && dB >= far) ? (float)tm : std::nanf("");
        code_lo = rays[in_idx].below;
        code_hi = rays[in_idx].above;
      } else {
        tau = std::nanf("");
        code_lo = code_hi = 0;
      }
      uint32_t bits;
      std::memcpy(&bits, &tau, 4);
      cells[o][c] = make_uint2(bits, ((uint32_t)code_lo << 28) | ((uint32_t)code_hi << 24));
    }
    // Check the two properties on a grid of every cell (the table is small; a wrong entry would be a silent
    // wrong code).
    for (int c = 0; c < pq::kL1Cells; ++c) {
      float tau;
      std::memcpy(&tau, &cells[o][c].x, 4);
      if (tau != tau) continue;
      const double scale = (double)pq::kL1CellScale;
      const double lo = std::fmax(0.0, (c - 1.0 / 16.0) / scale), hi = std::fmin(1.0, (c + 15.0 / 16.0) / scale);
      for (int i = 0; i <= 4; ++i) {
        const double t = lo + (hi - lo) * i / 4.0, dist = std::fabs(t - (double)tau);
        double nearest = 1e30;
        for (const L1Ray& r : rays) nearest = std::fmin(nearest, std::fabs(t - r.t));
        if (dist > nearest + 1e-7) return false;
        if (dist < 1e-6) continue;
        double psi = B + D * std::atan(t);
        if (psi >= 2.0 * kPi) psi -= 2.0 * kPi;
        if (psi < 0.0) psi += 2.0 * kPi;
        const int want = l1_code_of_angle(bnd, psi);
        const int got = (int)((cells[o][c].y >> (t > (double)tau ? 24 : 28)) & 15u);
        if (want != got) return false;
      }
    }
  }
  return true;
}

}  // namespace

namespace pq {
static thread_local cudaError_t g_last_cuda_error = cudaSuccess;
void note_cuda_error(cudaError_t e) { g_last_cuda_error = e; }
// The kernels' Paging from a caller's pq_paging (validated).
int32_t paging_from(const pq_paging* p, int head_dim, Paging* out) {
  if (p == nullptr || p->page_table_dev == nullptr) return PQ_ERR_INVALID_ARG;
  if (p->page_tokens <= 0 || p->pages_per_seq <= 0 || p->n_pages <= 0) return PQ_ERR_INVALID_ARG;
  if (p->page_tokens % (head_dim == 128 ? 128 : kTokenBlock)) return PQ_ERR_INVALID_ARG;
  if ((int64_t)p->page_tokens * p->pages_per_seq >= (1ll << 31)) return PQ_ERR_UNSUPPORTED;
  if ((uintptr_t)p->page_table_dev & 3) return PQ_ERR_ALIGNMENT;
  out->table = p->page_table_dev; out->page_tokens = p->page_tokens; out->pages_per_seq = p->pages_per_seq;
  out->n_pages = p->n_pages;
  return PQ_OK;
}

static std::atomic<int> g_debug_wait_failure{0};
bool take_debug_wait_failure(int which) {
  int armed = which;
  return g_debug_wait_failure.compare_exchange_strong(armed, 0);
}
}  // namespace pq

extern "C" {

const char* pq_last_cuda_error(void) {
  return pq::g_last_cuda_error == cudaSuccess ? "" : cudaGetErrorString(pq::g_last_cuda_error);
}

const char* pq_status_string(int32_t status) {
  switch (status) {
    case PQ_OK: return "ok";
    case PQ_ERR_INVALID_ARG: return "invalid argument";
    case PQ_ERR_UNSUPPORTED: return "unsupported configuration";
    case PQ_ERR_ALIGNMENT: return "device pointer not 16-byte aligned";
    case PQ_ERR_CAPACITY: return "cache capacity exceeded";
    case PQ_ERR_CUDA: return "CUDA runtime error";
    case PQ_ERR_TIMEOUT: return "bounded device wait timed out";
    case PQ_ERR_NONFINITE: return "non-finite input";
    case PQ_ERR_EMPTY: return "attention over an empty sequence";
    case PQ_ERR_SCRATCH: return "built-in scratch buffer too small for this problem";
    default: return "unknown status";
  }
}

int32_t pq_token_block(void) { return pq::kTokenBlock; }

int32_t pq_debug_fail_next_wait(int32_t which) {
  if (which < 0 || which > 4) return PQ_ERR_INVALID_ARG;
  pq::g_debug_wait_failure.store(which);
  return PQ_OK;
}

int32_t pq_make_structured_rotation(int32_t d, int32_t kind, const int8_t* signs_host, float* S_host) {
  if (S_host == nullptr || d <= 0) return PQ_ERR_INVALID_ARG;
  if (kind != PQ_ROTATION_IDENTITY && kind != PQ_ROTATION_HADAMARD) return PQ_ERR_INVALID_ARG;
  if (d > 4096) return PQ_ERR_UNSUPPORTED;
  if (kind == PQ_ROTATION_IDENTITY) {
    for (int i = 0; i < d; ++i)
      for (int j = 0; j < d; ++j) S_host[(size_t)i * d + j] = i == j ? 1.f : 0.f;
    return PQ_OK;
  }
  if (d & (d - 1)) return PQ_ERR_UNSUPPORTED;
  if (signs_host == nullptr) return PQ_ERR_INVALID_ARG;
  for (int i = 0; i < d; ++i)
    if (signs_host[i] != 1 && signs_host[i] != -1) return PQ_ERR_INVALID_ARG;
  // entry (i, j) of the Sylvester matrix: -1 to the number of bit positions set in both indices
  const double c = 1.0 / std::sqrt((double)d);
  for (int i = 0; i < d; ++i)
    for (int j = 0; j < d; ++j) {
      unsigned both = (unsigned)i & (unsigned)j;
      int odd = 0;
      for (; both; both &= both - 1) odd ^= 1;
      S_host[(size_t)i * d + j] = (float)((odd ? -c : c) * (double)signs_host[i]);
    }
  return PQ_OK;
}

int32_t pq_make_rotation(int32_t d, uint64_t seed, float* S_host) {
  pq::NvtxRange nvtx_range("pq_make_rotation");
  if (S_host == nullptr || d <= 0) return PQ_ERR_INVALID_ARG;
  if (d > 4096) return PQ_ERR_UNSUPPORTED;
  std::vector<double> A((size_t)d * d), Q((size_t)d * d, 0.0), v(d), w(d), rdiag(d);
  for (int64_t i = 0; i < (int64_t)d * d; ++i) A[i] = gaussian(seed, (uint64_t)i);
  for (int i = 0; i < d; ++i) Q[(size_t)i * d + i] = 1.0;
  // Householder QR: A = Q R.  Reflector k zeroes column k below the diagonal.
  for (int k = 0; k < d; ++k) {
    double norm = 0.0;
    for (int i = k; i < d; ++i) norm += A[(size_t)i * d + k] * A[(size_t)i * d + k];
    norm = std::sqrt(norm);
    const double x0 = A[(size_t)k * d + k];
    const double alpha = x0 >= 0.0 ? -norm : norm;
    rdiag[k] = alpha;
    double vnorm = 0.0;
    for (int i = k; i < d; ++i) {
      v[i] = A[(size_t)i * d + k] - (i == k ? alpha : 0.0);
      vnorm += v[i] * v[i];
    }
    if (vnorm == 0.0) continue;
    const double beta = 2.0 / vnorm;
    // A <- (I - beta v v^T) A on rows k..d-1
    for (int j = k; j < d; ++j) {
      double s = 0.0;
      for (int i = k; i < d; ++i) s += v[i] * A[(size_t)i * d + j];
      w[j] = s * beta;
    }
    for (int i = k; i < d; ++i)
      for (int j = k; j < d; ++j) A[(size_t)i * d + j] -= v[i] * w[j];
    // Q <- Q (I - beta v v^T) on columns k..d-1
    for (int i = 0; i < d; ++i) {
      double s = 0.0;
      for (int j = k; j < d; ++j) s += Q[(size_t)i * d + j] * v[j];
      s *= beta;
      for (int j = k; j < d; ++j) Q[(size_t)i * d + j] -= s * v[j];
    }
  }
  for (int i = 0; i < d; ++i)
    for (int j = 0; j < d; ++j) S_host[(size_t)i * d + j] = (float)(Q[(size_t)i * d + j] * (rdiag[j] < 0.0 ? -1.0 : 1.0));
  return PQ_OK;
}

int32_t pq_fit_codebooks(const int32_t* bits, double* centroids_host, double* boundaries_host) {
  pq::NvtxRange nvtx_range("pq_fit_codebooks");
  if (bits == nullptr || centroids_host == nullptr || boundaries_host == nullptr) return PQ_ERR_INVALID_ARG;
  if (bits[0] != 4 || bits[1] != 2 || bits[2] != 2 || bits[3] != 2) return PQ_ERR_UNSUPPORTED;
  for (int level = 1; level <= PQ_N_LEVELS; ++level) {
    const int n = 1 << bits[level - 1];
    const double lo = 0.0, hi = level == 1 ? 2.0 * kPi : 0.5 * kPi;
    double* theta = centroids_host + pq::cen_off(level);
    double* beta = boundaries_host + pq::bnd_off(level);
    for (int k = 0; k < n; ++k) theta[k] = lo + (k + 0.5) * (hi - lo) / n;
    for (int it = 0; it < 100000; ++it) {
      double delta = 0.0;
      for (int k = 0; k + 1 < n; ++k) beta[k] = 0.5 * (theta[k] + theta[k + 1]);
      for (int k = 0; k < n; ++k) {
        const double a = k == 0 ? lo : beta[k - 1], b = k == n - 1 ? hi : beta[k];
        double m0, m1;
        cell_moments(level, a, b, &m0, &m1);
        const double t = m1 / m0;
        delta = std::fmax(delta, std::fabs(t - theta[k]));
        theta[k] = t;
      }
      if (delta < 1e-15) break;
    }
    for (int k = 0; k + 1 < n; ++k) beta[k] = 0.5 * (theta[k] + theta[k + 1]);
  }
  return PQ_OK;
}

int32_t pq_fit_codebooks_from_histograms(const uint64_t* hist, int32_t n_bins, const double* init, double* cen,
                                         double* bnd) {
  if (hist == nullptr || cen == nullptr || bnd == nullptr || n_bins < 16 || n_bins > PQ_HIST_MAX_BINS) return PQ_ERR_INVALID_ARG;
  double start[PQ_N_CENTROIDS];
  if (init == nullptr) {
    // the analytic codebook costs tens of milliseconds of quadrature: computed once per process
    struct Analytic {
      double cen[PQ_N_CENTROIDS], bnd[PQ_N_BOUNDARIES];
      int32_t status;
      Analytic() {
        const int32_t bits[PQ_N_LEVELS] = {4, 2, 2, 2};
        status = pq_fit_codebooks(bits, cen, bnd);
      }
    };
    static const Analytic analytic;  // thread-safe initialisation
    if (analytic.status != PQ_OK) return analytic.status;
    std::memcpy(start, analytic.cen, sizeof(start));
  } else {
    std::memcpy(start, init, sizeof(start));
  }
  std::vector<double> centre(n_bins), w0(n_bins + 1), w1(n_bins + 1);
  for (int level = 1; level <= PQ_N_LEVELS; ++level) {
    const int n = level == 1 ? 16 : 4;
    const double hi = level == 1 ? 2.0 * kPi : 0.5 * kPi, width = hi / n_bins;
    const uint64_t* h = hist + (size_t)(level - 1) * n_bins;
    double* theta = cen + pq::cen_off(level);
    double* beta = bnd + pq::bnd_off(level);
    for (int k = 0; k < n; ++k) {
      theta[k] = start[pq::cen_off(level) + k];
      if (!(theta[k] >= 0.0 && theta[k] <= hi) || (k > 0 && !(theta[k] > theta[k - 1]))) return PQ_ERR_INVALID_ARG;
    }
    // prefix sums of the weights and of weight x centre: a cell's mean is two differences
    w0[0] = w1[0] = 0.0;
    for (int i = 0; i < n_bins; ++i) {
      centre[i] = (i + 0.5) * width;
      w0[i + 1] = w0[i] + (double)h[i];
      w1[i + 1] = w1[i] + (double)h[i] * centre[i];
    }
    for (int iter = 0; iter < 10000; ++iter) {
      bool moved = false;
      int first = 0;  // first bin of cell k
      double next[16];
      for (int k = 0; k < n; ++k) {
        // the cell ends before the first bin whose centre lies above the boundary between k and k + 1
        int last = n_bins;
        if (k + 1 < n) {
          const double b = 0.5 * (theta[k] + theta[k + 1]);
          last = (int)(std::upper_bound(centre.begin() + first, centre.end(), b) - centre.begin());
        }
        const double m0 = w0[last] - w0[first], m1 = w1[last] - w1[first];
        next[k] = m0 > 0.0 ? m1 / m0 : theta[k];
        first = last;
      }
      for (int k = 0; k < n; ++k) {
        moved = moved || next[k] != theta[k];
        theta[k] = next[k];
      }
      if (!moved) break;
    }
    for (int k = 0; k + 1 < n; ++k) beta[k] = 0.5 * (theta[k] + theta[k + 1]);
  }
  return PQ_OK;
}

int64_t pq_tables_bytes(void) { return (int64_t)sizeof(pq::Tables); }

int32_t pq_build_tables(const double* cen, const double* bnd, void* tables_host) {
  if (cen == nullptr || bnd == nullptr || tables_host == nullptr) return PQ_ERR_INVALID_ARG;
  for (int level = 1; level <= PQ_N_LEVELS; ++level) {
    const int n = level == 1 ? 16 : 4;
    const double hi = level == 1 ? 2.0 * kPi : 0.5 * kPi;
    for (int k = 0; k < n; ++k) {
      const double c = cen[pq::cen_off(level) + k];
      if (!(c >= 0.0 && c <= hi)) return PQ_ERR_INVALID_ARG;
      if (k > 0 && !(c > cen[pq::cen_off(level) + k - 1])) return PQ_ERR_INVALID_ARG;
    }
    for (int k = 0; k + 1 < n; ++k) {
      const double b = bnd[pq::bnd_off(level) + k];
      if (!(b > 0.0 && b < hi)) return PQ_ERR_INVALID_ARG;
      if (k > 0 && !(b > bnd[pq::bnd_off(level) + k - 1])) return PQ_ERR_INVALID_ARG;
    }
  }
  pq::Tables t;
  std::memset(&t, 0, sizeof(t));
  bool uniform = true;
  for (int k = 0; k < PQ_N_BOUNDARIES; ++k) {
    t.bnd[k] = bnd[k];
    t.bnd_cos[k] = std::cos(bnd[k]);
    t.bnd_sin[k] = std::sin(bnd[k]);
    t.bnd_cosf[k] = (float)t.bnd_cos[k];
    t.bnd_sinf[k] = (float)t.bnd_sin[k];
  }
  for (int k = 0; k < 9; ++k) {
    const double tn = std::tan(bnd[15 + k]);
    t.bnd_tan2[k] = tn * tn;
  }
  for (int k = 0; k < 15; ++k) {
    t.bnd_upper[k] = bnd[k] <= kPi ? 1 : 0;
    t.n_upper += t.bnd_upper[k];
    if (std::fabs(bnd[k] - (k + 1) * kPi / 8.0) > 1e-12) uniform = false;
  }
  bool symmetric = true;
  for (int l = 0; l < 3; ++l)
    if (std::fabs(t.bnd_tan2[3 * l + 1] - 1.0) > 1e-9 || std::fabs(t.bnd_tan2[3 * l] * t.bnd_tan2[3 * l + 2] - 1.0) > 1e-9)
      symmetric = false;
  t.flags = (uniform ? pq::kFlagUniformL1 : 0u) | (symmetric ? pq::kFlagSymmetricUpper : 0u);
  for (int k = 0; k < PQ_N_CENTROIDS; ++k) {
    t.cen_cos[k] = (float)std::cos(cen[k]);
    t.cen_sin[k] = (float)std::sin(cen[k]);
  }
  auto h2 = [](double lo, double hi) -> uint32_t {
    const __half a = __double2half(lo), b = __double2half(hi);
    uint16_t ua, ub;
    std::memcpy(&ua, &a, 2);
    std::memcpy(&ub, &b, 2);
    return (uint32_t)ua | ((uint32_t)ub << 16);
  };
  auto split = [&](double va, double vb, uint32_t* hi, uint32_t* lo) {
    const double ha = (double)__half2float(__double2half(va)), hb = (double)__half2float(__double2half(vb));
    *hi = h2(va, vb);
    *lo = h2(va - ha, vb - hb);
  };
  for (int c = 0; c < 16; ++c) split(std::cos(cen[c]), std::sin(cen[c]), &t.l1_hi[c], &t.l1_lo[c]);
  for (int e = 0; e < 256; ++e) {
    const uint32_t ha = t.l1_hi[e & 15], hb = t.l1_hi[e >> 4], la = t.l1_lo[e & 15], lb = t.l1_lo[e >> 4];
    t.t1p_hi[e] = make_uint2((ha & 0xFFFFu) | (hb << 16), (ha >> 16) | (hb & 0xFFFF0000u));
    t.t1p_lo[e] = make_uint2((la & 0xFFFFu) | (lb << 16), (la >> 16) | (lb & 0xFFFF0000u));
  }
  double uc[12], us[12];  // cos / sin of the centroids of levels 2, 3, 4
  for (int k = 0; k < 12; ++k) {
    uc[k] = std::cos(cen[16 + k]);
    us[k] = std::sin(cen[16 + k]);
  }
  for (int s = 0; s < 4; ++s)
    for (int i = 0; i < 64; ++i) {
      const int k2 = i & 3, k3 = 4 + ((i >> 2) & 3), k4 = 8 + (i >> 4);
      const double t4 = (s >> 1) ? us[k4] : uc[k4];
      const double t3 = (s & 1) ? us[k3] : uc[k3];
      split(t4 * t3 * uc[k2], t4 * t3 * us[k2], &t.u_tab[s][i].x, &t.u_tab[s][i].y);
    }
  if (!build_l1_cells(bnd, t.l1_cells)) return PQ_ERR_INVALID_ARG;
  std::memcpy(tables_host, &t, sizeof(t));
  return PQ_OK;
}

int64_t pq_cache_bytes(int32_t head_dim, int32_t batch, int32_t n_kv_heads, int32_t capacity) {
  if (!(head_dim == 16 || head_dim == 32 || head_dim == 64 || head_dim == 128)) return PQ_ERR_UNSUPPORTED;
  if (batch <= 0 || n_kv_heads <= 0 || capacity <= 0) return PQ_ERR_INVALID_ARG;
  const pq::Layout L = pq::make_layout(head_dim, capacity);
  return (int64_t)batch * n_kv_heads * L.head_bytes;
}

int64_t pq_paged_cache_bytes(int32_t head_dim, int32_t n_kv_heads, int32_t page_tokens, int32_t n_pages) {
  if (!(head_dim == 16 || head_dim == 32 || head_dim == 64 || head_dim == 128)) return PQ_ERR_UNSUPPORTED;
  if (n_kv_heads <= 0 || page_tokens <= 0 || n_pages <= 0) return PQ_ERR_INVALID_ARG;
  if (page_tokens % (head_dim == 128 ? 128 : pq::kTokenBlock)) return PQ_ERR_INVALID_ARG;
  const pq::Layout L = pq::make_layout(head_dim, page_tokens);
  return (int64_t)n_pages * n_kv_heads * L.head_bytes;
}

}  // extern "C"
