// Host side of the nested gradient code: construction of the component codes
// (Algorithm 1), the layered task schedule (Section III) and the stopping rule
// (Sections II-D / III).  Everything here is plain fp64 in a fixed operation order,
// compiled without fused multiply-add contraction, so results are bit-reproducible.
#include <algorithm>
#include <cmath>
#include <cstring>
#include <limits>
#include <new>
#include <numeric>

#include "ngc_internal.h"

namespace {

// SplitMix64 (Steele, Lea, Flood 2014): k-th output of the stream seeded with `seed`.
inline uint64_t splitmix64_at(uint64_t seed, uint64_t k) {
  uint64_t z = seed + k * 0x9E3779B97F4A7C15ull;
  z = (z ^ (z >> 30)) * 0xBF58476D1CE4E5B9ull;
  z = (z ^ (z >> 27)) * 0x94D049BB133111EBull;
  return z ^ (z >> 31);
}

// Entry (r, c) of the zero-row-sum matrix H of tolerance s: dyadic uniform in [-1, 1).
inline double h_entry(uint64_t seed, int s, int r, int c) {
  const uint64_t k = 1ull + (((uint64_t)s << 20) | ((uint64_t)r << 10) | (uint64_t)c);
  const uint64_t u = splitmix64_at(seed, k) >> 11;
  return (double)u / 4503599627370496.0 - 1.0;
}

// Solves the s x s system M z = b by Gaussian elimination with partial pivoting
// (first row of maximal magnitude), row-wise elimination, back substitution last to first.
void solve_small(int s, std::vector<double> &M, std::vector<double> &b, std::vector<double> &z) {
  for (int p = 0; p < s; ++p) {
    double best = std::fabs(M[p * s + p]);
    int q = p;
    for (int r = p + 1; r < s; ++r) {
      const double v = std::fabs(M[r * s + p]);
      if (v > best) { best = v; q = r; }
    }
    if (q != p) {
      for (int c = 0; c < s; ++c) std::swap(M[p * s + c], M[q * s + c]);
      std::swap(b[p], b[q]);
    }
    for (int r = p + 1; r < s; ++r) {
      const double f = M[r * s + p] / M[p * s + p];
      for (int c = p + 1; c < s; ++c) M[r * s + c] = M[r * s + c] - f * M[p * s + c];
      b[r] = b[r] - f * b[p];
    }
  }
  for (int p = s - 1; p >= 0; --p) {
    double acc = b[p];
    for (int c = p + 1; c < s; ++c) acc = acc - M[p * s + c] * z[c];
    z[p] = acc / M[p * s + p];
  }
}

// Coefficients of B_s in windowed storage: coef[i*(s+1)+t] = B[i, (i+t) mod n].
void build_coefficients(int n, int s, uint64_t seed, std::vector<double> &coef) {
  coef.assign((size_t)n * (s + 1), 0.0);
  if (s == 0) {
    for (int i = 0; i < n; ++i) coef[i] = 1.0;
    return;
  }
  std::vector<double> H((size_t)s * n);
  for (int r = 0; r < s; ++r) {
    double acc = 0.0;
    for (int c = 0; c < n - 1; ++c) {
      H[(size_t)r * n + c] = h_entry(seed, s, r, c);
      acc = acc + H[(size_t)r * n + c];
    }
    H[(size_t)r * n + n - 1] = -acc;
  }
  std::vector<double> M((size_t)s * s), b(s), z(s);
  for (int i = 0; i < n; ++i) {
    for (int r = 0; r < s; ++r) {
      for (int t = 0; t < s; ++t) M[r * s + t] = H[(size_t)r * n + (i + 1 + t) % n];
      b[r] = -H[(size_t)r * n + i];
    }
    solve_small(s, M, b, z);
    coef[(size_t)i * (s + 1)] = 1.0;
    for (int t = 0; t < s; ++t) coef[(size_t)i * (s + 1) + 1 + t] = z[t];
  }
}

// Householder QR with column pivoting of the dense n x n matrix A (row-major), rank r = n - s.
// Produces an orthonormal basis N (n x s) of the left null space {v : A^T v = 0} and the
// minimum-norm solution a0 of A^T a = 1.  Used by the device solve, which turns every
// straggler pattern into an s x s system instead of an n x (n-s) one.
void left_null_space(int n, int s, const std::vector<double> &A_in, std::vector<double> &N,
                     std::vector<double> &a0) {
  std::vector<double> A(A_in);          // becomes R (upper triangle)
  std::vector<double> Q((size_t)n * n, 0.0);
  for (int i = 0; i < n; ++i) Q[(size_t)i * n + i] = 1.0;
  std::vector<int> perm(n);
  std::iota(perm.begin(), perm.end(), 0);
  std::vector<double> v(n);
  const int r = n - s;
  for (int p = 0; p < r; ++p) {
    // pivot: remaining column of largest norm
    int best = p;
    double bestn = -1.0;
    for (int c = p; c < n; ++c) {
      double nn = 0.0;
      for (int i = p; i < n; ++i) nn += A[(size_t)i * n + c] * A[(size_t)i * n + c];
      if (nn > bestn) { bestn = nn; best = c; }
    }
    if (best != p) {
      for (int i = 0; i < n; ++i) std::swap(A[(size_t)i * n + p], A[(size_t)i * n + best]);
      std::swap(perm[p], perm[best]);
    }
    double alpha = std::sqrt(bestn);
    if (alpha == 0.0) continue;
    if (A[(size_t)p * n + p] > 0.0) alpha = -alpha;
    double vnorm2 = 0.0;
    for (int i = p; i < n; ++i) {
      v[i] = A[(size_t)i * n + p];
      if (i == p) v[i] -= alpha;
      vnorm2 += v[i] * v[i];
    }
    if (vnorm2 == 0.0) continue;
    for (int c = p; c < n; ++c) {            // A <- (I - 2 v v^T / v^T v) A
      double dot = 0.0;
      for (int i = p; i < n; ++i) dot += v[i] * A[(size_t)i * n + c];
      const double f = 2.0 * dot / vnorm2;
      for (int i = p; i < n; ++i) A[(size_t)i * n + c] -= f * v[i];
    }
    for (int row = 0; row < n; ++row) {      // Q <- Q (I - 2 v v^T / v^T v)
      double dot = 0.0;
      for (int i = p; i < n; ++i) dot += Q[(size_t)row * n + i] * v[i];
      const double f = 2.0 * dot / vnorm2;
      for (int i = p; i < n; ++i) Q[(size_t)row * n + i] -= f * v[i];
    }
  }
  N.assign((size_t)n * s, 0.0);
  for (int i = 0; i < n; ++i)
    for (int c = 0; c < s; ++c) N[(size_t)i * s + c] = Q[(size_t)i * n + r + c];
  // A P = Q R  =>  A^T a = 1  <=>  R^T (Q^T a) = P^T 1 = 1.  Forward-substitute the leading r x r block.
  std::vector<double> w(r);
  for (int i = 0; i < r; ++i) {
    double acc = 1.0;
    for (int c = 0; c < i; ++c) acc -= A[(size_t)c * n + i] * w[c];
    w[i] = acc / A[(size_t)i * n + i];
  }
  a0.assign(n, 0.0);
  for (int i = 0; i < n; ++i) {
    double acc = 0.0;
    for (int c = 0; c < r; ++c) acc += Q[(size_t)i * n + c] * w[c];
    a0[i] = acc;
  }
  (void)perm;
}

}  // namespace

int ngc_host_build_plan(ngc_plan_s *p) {
  const int n = p->n;
  p->lv.resize(p->L);
  for (int l = 0; l < p->L; ++l) {
    ngc_level_t &lv = p->lv[l];
    lv.s = p->levels[l];
    build_coefficients(n, lv.s, p->seed, lv.coef);
    if (lv.s == 0) {
      lv.a0.assign(n, 1.0);
      lv.N.clear();
      continue;
    }
    std::vector<double> dense((size_t)n * n, 0.0);
    for (int i = 0; i < n; ++i)
      for (int t = 0; t <= lv.s; ++t) dense[(size_t)i * n + (i + t) % n] = lv.coef[(size_t)i * (lv.s + 1) + t];
    left_null_space(n, lv.s, dense, lv.N, lv.a0);
    double worst = 0.0;
    for (int j = 0; j < n; ++j) {
      double acc = 0.0;
      for (int i = 0; i < n; ++i) acc += dense[(size_t)i * n + j] * lv.a0[i];
      worst = std::max(worst, std::fabs(acc - 1.0));
      for (int c = 0; c < lv.s; ++c) {
        double t = 0.0;
        for (int i = 0; i < n; ++i) t += dense[(size_t)i * n + j] * lv.N[(size_t)i * lv.s + c];
        worst = std::max(worst, std::fabs(t));
      }
    }
    lv.plan_residual = worst;
  }
  const int sL = p->levels.back();
  p->order.resize((size_t)n * (sL + 1));
  for (int i = 0; i < n; ++i)
    for (int t = 0; t <= sL; ++t) p->order[(size_t)i * (sL + 1) + t] = (i + t) % n;
  p->tasks_per_layer.resize(p->L);
  for (int l = 0; l < p->L; ++l) p->tasks_per_layer[l] = p->levels[l] + 1;
  return NGC_OK;
}

extern "C" {

int64_t ngc_num_params(const ngc_model_t *m) {
  if (!m || m->d <= 0) return -1;
  switch (m->kind) {
    case NGC_LSQ:
    case NGC_LOGISTIC:
      return m->d;
    case NGC_SOFTMAX:
      return m->n_classes > 0 ? (int64_t)m->d * m->n_classes : -1;
    case NGC_MLP:
      if (m->n_classes <= 0 || m->hidden <= 0) return -1;
      return (int64_t)m->d * m->hidden + m->hidden + (int64_t)m->hidden * m->n_classes + m->n_classes;
    default:
      return -1;
  }
}

int ngc_plan(int n_workers, int n_levels, const int *s_levels, int n_partitions, uint64_t seed, double gamma,
             double eps, ngc_plan_t **out) {
  if (!out) return NGC_ERR_INVALID;
  *out = nullptr;
  if (n_workers < 1 || n_workers > NGC_MAX_N || n_levels < 1 || n_levels > NGC_MAX_LEVELS || !s_levels)
    return NGC_ERR_INVALID;
  if (n_partitions < n_workers || n_partitions % n_workers != 0) return NGC_ERR_INVALID;
  for (int l = 0; l < n_levels; ++l) {
    if (s_levels[l] < 0 || s_levels[l] >= n_workers || s_levels[l] > NGC_MAX_S) return NGC_ERR_INVALID;
    if (l > 0 && s_levels[l] <= s_levels[l - 1]) return NGC_ERR_INVALID;
  }
  if (!(gamma >= 0.0) || !(eps >= 0.0)) return NGC_ERR_INVALID;
  ngc_plan_s *p = new (std::nothrow) ngc_plan_s();
  if (!p) return NGC_ERR_NOMEM;
  p->n = n_workers;
  p->k = n_partitions;
  p->q = n_partitions / n_workers;
  p->L = n_levels;
  p->seed = seed;
  p->gamma = gamma;
  p->eps = eps;
  p->levels.assign(s_levels, s_levels + n_levels);
  const int rc = ngc_host_build_plan(p);
  if (rc != NGC_OK) {
    delete p;
    return rc;
  }
  *out = p;
  return NGC_OK;
}

int ngc_plan_B(const ngc_plan_t *p, int layer, const double **coef, int *width) {
  if (!p || !coef || !width || layer < 0 || layer >= p->L) return NGC_ERR_INVALID;
  *coef = p->lv[layer].coef.data();
  *width = p->lv[layer].s + 1;
  return NGC_OK;
}

int ngc_plan_schedule(const ngc_plan_t *p, const int32_t **order, const int32_t **tasks_per_layer) {
  if (!p || !order || !tasks_per_layer) return NGC_ERR_INVALID;
  *order = p->order.data();
  *tasks_per_layer = p->tasks_per_layer.data();
  return NGC_OK;
}

int ngc_set_coded_dtype(ngc_plan_t *p, int dtype) {
  if (!p || !(dtype == -1 || dtype == NGC_F32 || dtype == NGC_F64)) return NGC_ERR_INVALID;
  p->coded_dtype_override = dtype;
  return NGC_OK;
}

int ngc_coded_dtype(const ngc_plan_t *p, const ngc_model_t *m) {
  if (!p || !m) return NGC_ERR_INVALID;
  if (p->coded_dtype_override >= 0) return p->coded_dtype_override;
  return (m->kind == NGC_LSQ || m->kind == NGC_LOGISTIC) ? NGC_F64 : NGC_F32;
}

int ngc_select(const ngc_plan_t *p, const double *times, ngc_step_info_t *info) {
  if (!p || !times || !info) return NGC_ERR_INVALID;
  const int n = p->n, nt = p->levels.back() + 1;
  for (int i = 0; i < n * nt; ++i)
    if (!(times[i] >= 0.0)) return NGC_ERR_INVALID;  // negative or NaN
  std::vector<double> C((size_t)n * nt);
  for (int i = 0; i < n; ++i) {
    double acc = 0.0;
    for (int m = 0; m < nt; ++m) {
      acc = acc + times[(size_t)i * nt + m];
      C[(size_t)i * nt + m] = acc;
    }
  }
  const double inf = std::numeric_limits<double>::infinity();
  int best_l = -1;
  double best_D = inf;
  std::vector<double> col(n);
  for (int l = 0; l < p->L; ++l) {
    const int s = p->levels[l];
    for (int i = 0; i < n; ++i) col[i] = C[(size_t)i * nt + s];
    std::sort(col.begin(), col.end());
    const double D = col[n - s - 1];
    if (D < best_D) { best_D = D; best_l = l; }
  }
  if (best_l < 0) return NGC_ERR_UNDECODABLE;
  const int s = p->levels[best_l];
  std::vector<int> idx(n);
  std::iota(idx.begin(), idx.end(), 0);
  std::stable_sort(idx.begin(), idx.end(),
                   [&](int a, int b) { return C[(size_t)a * nt + s] < C[(size_t)b * nt + s]; });
  std::vector<int> S(idx.begin(), idx.begin() + (n - s));
  std::sort(S.begin(), S.end());
  std::memset(info, 0, sizeof(*info));
  info->layer = best_l;
  info->sigma = s;
  info->nS = n - s;
  for (int t = 0; t < n - s; ++t) info->S[t] = S[t];
  info->latency = p->gamma + p->eps + best_D;
  for (int i = 0; i < n; ++i) {
    int done = 0;
    for (int m = 0; m < nt; ++m)
      if (C[(size_t)i * nt + m] <= best_D) done = m + 1;
    info->tasks_done[i] = done;
  }
  return NGC_OK;
}

int ngc_sample_times(uint64_t seed, int n, int tasks, double shift, double rate, double p_fail, double *out) {
  if (!out || n < 1 || tasks < 1 || !(rate > 0.0) || !(shift >= 0.0) || !(p_fail >= 0.0 && p_fail <= 1.0))
    return NGC_ERR_INVALID;
  const double inf = std::numeric_limits<double>::infinity();
  for (int i = 0; i < n; ++i) {
    const double uf = (double)(splitmix64_at(seed, 1ull + (uint64_t)i * (tasks + 1)) >> 11) / 9007199254740992.0;
    const bool dead = uf < p_fail;
    for (int m = 0; m < tasks; ++m) {
      const uint64_t bits = splitmix64_at(seed, 2ull + (uint64_t)i * (tasks + 1) + m) >> 11;
      const double u = ((double)bits + 0.5) / 9007199254740992.0;  // (0, 1)
      out[(size_t)i * tasks + m] = dead ? inf : shift - std::log(u) / rate;
    }
  }
  return NGC_OK;
}

// ---- Section IV closed forms ----------------------------------------------------------------------
namespace {
// Binomial coefficients as doubles, Pascal's rule.
struct Binom {
  std::vector<double> c;
  int n;
  explicit Binom(int n_) : c((size_t)(n_ + 1) * (n_ + 1), 0.0), n(n_) {
    for (int a = 0; a <= n; ++a) {
      c[(size_t)a * (n + 1)] = 1.0;
      for (int b = 1; b <= a; ++b)
        c[(size_t)a * (n + 1) + b] = c[(size_t)(a - 1) * (n + 1) + b - 1] + (b <= a - 1 ? c[(size_t)(a - 1) * (n + 1) + b] : 0.0);
    }
  }
  double operator()(int a, int b) const { return (b < 0 || b > a) ? 0.0 : c[(size_t)a * (n + 1) + b]; }
};

// Eq. 3 with the Erlang tail summed over k = 0..u-1: P(u tasks done by t).
double tasks_cdf(int u, double t, double lam, double rho, double gamma, double eps) {
  if (u == 0) return 1.0;
  const double x = t - (gamma + eps + u * rho);
  if (x <= 0.0) return 0.0;
  double term = 1.0, tail = 1.0;
  for (int k = 1; k < u; ++k) {
    term *= lam * x / k;
    tail += term;
  }
  return 1.0 - tail * std::exp(-lam * x);
}
bool latency_args_ok(int n, int s, double lam, double rho, double gamma, double eps, double pf) {
  return n >= 1 && n <= NGC_MAX_N && s >= 0 && s < n && lam > 0.0 && rho >= 0.0 && gamma >= 0.0 && eps >= 0.0 &&
         pf >= 0.0 && pf <= 1.0;
}
}  // namespace

double ngc_latency_cdf_gc(int n, int sigma, double t, double lam, double rho, double gamma, double eps, double pf) {
  if (!latency_args_ok(n, sigma, lam, rho, gamma, eps, pf)) return -1.0;
  const Binom C(n);
  const double F = tasks_cdf(sigma + 1, t, lam, rho, gamma, eps);
  double total = 0.0;
  for (int kappa = 0; kappa <= sigma; ++kappa) {
    const int alive = n - kappa;
    double cond = 0.0;
    for (int tau = n - sigma; tau <= alive; ++tau) cond += C(alive, tau) * std::pow(F, tau) * std::pow(1.0 - F, alive - tau);
    total += cond * C(n, kappa) * std::pow(pf, kappa) * std::pow(1.0 - pf, n - kappa);
  }
  return total;
}

double ngc_latency_cdf_ngc(int n, int s_max, double t, double lam, double rho, double gamma, double eps, double pf) {
  if (!latency_args_ok(n, s_max, lam, rho, gamma, eps, pf)) return -1.0;
  const Binom C(n);
  const int top = s_max + 1;
  std::vector<double> F(top + 2), q(top + 1);
  for (int u = 0; u <= top + 1; ++u) F[u] = tasks_cdf(u, t, lam, rho, gamma, eps);
  for (int u = 0; u < top; ++u) q[u] = F[u] - F[u + 1];  // exactly u tasks done
  q[top] = F[top];                                        // s_max + 1 (or more) done
  double total = 0.0;
  for (int kappa = 0; kappa <= s_max; ++kappa) {
    const int alive = n - kappa;
    // w[c] = weight of the configurations in which c alive workers have finished at least u tasks and no
    // component has been decodable so far (at most n - v workers with >= v tasks, for every v >= u)
    std::vector<double> w(alive + 1, 0.0), w2(alive + 1);
    for (int c = 0; c <= std::min(alive, n - top); ++c) w[c] = C(alive, c) * std::pow(q[top], c);
    for (int u = top - 1; u >= 1; --u) {
      std::fill(w2.begin(), w2.end(), 0.0);
      const int cap = std::min(alive, n - u);
      for (int c = 0; c <= alive; ++c) {
        if (w[c] == 0.0) continue;
        for (int i = 0; c + i <= cap; ++i) w2[c + i] += w[c] * C(alive - c, i) * std::pow(q[u], i);
      }
      w.swap(w2);
    }
    double not_decodable = 0.0;
    for (int c = 0; c <= alive; ++c) not_decodable += w[c] * std::pow(q[0], alive - c);
    total += (1.0 - not_decodable) * C(n, kappa) * std::pow(pf, kappa) * std::pow(1.0 - pf, n - kappa);
  }
  return total;
}

const char *ngc_strerror(int status) {
  switch (status) {
    case NGC_OK: return "ok";
    case NGC_ERR_INVALID: return "invalid argument";
    case NGC_ERR_UNDECODABLE: return "no component code becomes decodable for this straggler pattern";
    case NGC_ERR_SINGULAR: return "decoding vector residual above threshold";
    case NGC_ERR_CUDA: return "CUDA runtime error";
    case NGC_ERR_TIMEOUT: return "bounded device-side wait gave up";
    case NGC_ERR_NOMEM: return "out of host memory";
    case NGC_ERR_TOO_LARGE: return "problem exceeds the fixed scratch array of ngc_grad_encode_static";
    default: return "unknown status";
  }
}

}  // extern "C"
