// Performance models and strategy selector (host arithmetic only).
//
//   Eq. 2-3  T_decomp(d) = (d-1) * T_stage * eta(d) + T_comp/d + T_comm/d,
//            T_stage = max(T_comp, T_comm)/d, eta(d) = alpha + beta*d
//   Eq. 4-5  d* = P2(sqrt((1 - alpha + rho)/beta)) kept only if it beats d = 1
//   Eq. 7-8  T_fusion = (n-1)*max(T_comp/n, T_comm/(n-1)) + T_comp/n
//                       + (n-1)*(alpha_f + beta_f*m)
//   Algorithm 1: IntraFusion if T_fusion < T_decomp(d*), else InterDecom.
//
// rho: Eq. 5 prints 1/lambda, the stationary point of Eq. 2 when T_comp >=
// T_comm.  Differentiating Eq. 2 in general gives
// d^2 = ((T_comp+T_comm)/max(T_comp,T_comm) - alpha)/beta, i.e. rho =
// min(lambda, 1/lambda); that is the default, the literal form is selectable.
#include <cmath>

#include "internal.h"

namespace compass {
namespace {

constexpr int kCandidates[4] = {2, 4, 8, 16};   // Table IV, decomposition degrees

double decomp_time(double tc, double tm, double alpha, double beta, int d) {
  const double dd = double(d);
  const double t_stage = (tc > tm ? tc : tm) / dd;
  return (dd - 1.0) * t_stage * (alpha + beta * dd) + tc / dd + tm / dd;
}

// Nearest power of two on a log scale: between 2^e and 2^(e+1) the boundary is
// their geometric mean; exact ties go down.
int nearest_pow2(double x) {
  int e = 0;
  double low = std::frexp(x, &e);   // x = low * 2^e, low in [0.5, 1)
  (void)low;
  e -= 1;                           // 2^e <= x < 2^(e+1)
  const double lo = std::ldexp(1.0, e), hi = std::ldexp(1.0, e + 1);
  const double pick = (x * x <= lo * hi) ? lo : hi;
  if (pick < 1.0) return 1;
  if (pick > 1073741824.0) return 1 << 30;
  return int(pick);
}

// Argument of P2 in Eq. 5, or a negative value when it does not exist.
double d_continuous(double tc, double tm, double alpha, double beta, bool as_printed) {
  if (!(tc > 0.0) || !(tm > 0.0) || !(beta > 0.0)) return -1.0;
  const double lambda = tc / tm;
  const double inv = 1.0 / lambda;
  const double rho = as_printed ? inv : (lambda < inv ? lambda : inv);
  const double radicand = (1.0 - alpha + rho) / beta;
  if (!(radicand > 0.0)) return -1.0;
  return std::sqrt(radicand);
}

// Eq. 5 clamped to the admissible candidates; 0 if there is none.
int d_candidate(double tc, double tm, double alpha, double beta, int d_max, bool as_printed, double* d_cont) {
  int n = 0;
  while (n < 4 && kCandidates[n] <= d_max) ++n;
  const double x = d_continuous(tc, tm, alpha, beta, as_printed);
  if (d_cont) *d_cont = x;
  if (n == 0) return 0;
  if (x < 0.0) {
    int best = kCandidates[0];
    for (int i = 1; i < n; ++i)
      if (decomp_time(tc, tm, alpha, beta, kCandidates[i]) < decomp_time(tc, tm, alpha, beta, best)) best = kCandidates[i];
    return best;
  }
  if (!(x < 1.0e6)) return kCandidates[n - 1];   // far beyond the candidate set, or overflowed to infinity
  int d = nearest_pow2(x);
  if (d < kCandidates[0]) d = kCandidates[0];
  if (d > kCandidates[n - 1]) d = kCandidates[n - 1];
  return d;
}

int optimal_degree(double tc, double tm, double alpha, double beta, int d_max, bool as_printed, double* d_cont) {
  if (d_cont) *d_cont = -1.0;
  if (!(tm > 0.0)) return 1;
  const int cand = d_candidate(tc, tm, alpha, beta, d_max, as_printed, d_cont);
  if (cand == 0) return 1;
  return decomp_time(tc, tm, alpha, beta, cand) < decomp_time(tc, tm, alpha, beta, 1) ? cand : 1;   // Eq. 4
}

double fusion_time(double tc, double tm, int n, double alpha_f, double beta_f, double m_volume) {
  const double comp_chunk = tc / n;
  const double comm_chunk = n > 1 ? tm / (n - 1) : 0.0;
  double t = 0.0;
  for (int i = 2; i <= n; ++i) t += comp_chunk > comm_chunk ? comp_chunk : comm_chunk;   // overlapped stages
  t += comp_chunk;                                                                          // exposed first chunk
  t += double(n - 1) * (alpha_f + beta_f * m_volume);                                       // Eq. 8
  return t;
}

// Least squares y = a + b*x.
bool ols(const double* x, const double* y, size_t n, double* a, double* b) {
  if (n == 0) return false;
  double mx = 0, my = 0;
  for (size_t i = 0; i < n; ++i) {
    mx += x[i];
    my += y[i];
  }
  mx /= double(n);
  my /= double(n);
  double sxx = 0, sxy = 0;
  for (size_t i = 0; i < n; ++i) {
    sxx += (x[i] - mx) * (x[i] - mx);
    sxy += (x[i] - mx) * (y[i] - my);
  }
  if (sxx == 0.0) {
    *a = my;
    *b = 0.0;
    return true;
  }
  *b = sxy / sxx;
  *a = my - *b * mx;
  return true;
}

int largest_degree(int64_t rows_per_rank) {
  int d = 1;
  while (d < 16 && rows_per_rank % (2 * d) == 0) d *= 2;
  return d;
}

}  // namespace
}  // namespace compass

using namespace compass;

extern "C" int compass_model_decomp_time(double t_comp, double t_comm, double alpha, double beta, int d, double* out) {
  if (out == nullptr || d < 1) return COMPASS_ERR_INVALID_ARG;
  *out = decomp_time(t_comp, t_comm, alpha, beta, d);
  return COMPASS_OK;
}

extern "C" int compass_model_optimal_degree(double t_comp, double t_comm, double alpha, double beta, int d_max,
                                            int as_printed, int* d_final, double* d_cont) {
  if (d_final == nullptr || d_max < 1) return COMPASS_ERR_INVALID_ARG;
  *d_final = optimal_degree(t_comp, t_comm, alpha, beta, d_max, as_printed != 0, d_cont);
  return COMPASS_OK;
}

extern "C" int compass_model_fusion_time(double t_comp, double t_comm, int n_chunks, double alpha_f, double beta_f,
                                         double m_volume, double* out) {
  if (out == nullptr || n_chunks < 1) return COMPASS_ERR_INVALID_ARG;
  *out = fusion_time(t_comp, t_comm, n_chunks, alpha_f, beta_f, m_volume);
  return COMPASS_OK;
}

extern "C" int compass_calib_fit_decomp(const double* t_comp, const double* t_comm, const int* d, const double* t_meas,
                                        size_t n, double* alpha, double* beta) {
  if (!t_comp || !t_comm || !d || !t_meas || !alpha || !beta || n == 0) return COMPASS_ERR_INVALID_ARG;
  if (n > 4096) return COMPASS_ERR_UNSUPPORTED;
  double xs[4096], ys[4096];
  for (size_t i = 0; i < n; ++i) {
    if (d[i] < 2) return COMPASS_ERR_INVALID_ARG;
    const double dd = double(d[i]);
    const double t_stage = (t_comp[i] > t_comm[i] ? t_comp[i] : t_comm[i]) / dd;
    if (!(t_stage > 0.0)) return COMPASS_ERR_INVALID_ARG;
    xs[i] = dd;
    ys[i] = (t_meas[i] - (t_comp[i] + t_comm[i]) / dd) / ((dd - 1.0) * t_stage);   // Eq. 2 solved for eta
  }
  return ols(xs, ys, n, alpha, beta) ? COMPASS_OK : COMPASS_ERR_INVALID_ARG;
}

extern "C" int compass_calib_fit_line(const double* x, const double* y, size_t n, double* a, double* b) {
  if (!x || !y || !a || !b || n == 0) return COMPASS_ERR_INVALID_ARG;
  return ols(x, y, n, a, b) ? COMPASS_OK : COMPASS_ERR_INVALID_ARG;
}

extern "C" int compass_calib_fit_fusion(const double* t_comp, const double* t_comm, const int* n_chunks,
                                        const double* m_volume, const double* t_meas, size_t n, double* alpha_f,
                                        double* beta_f) {
  if (!t_comp || !t_comm || !n_chunks || !m_volume || !t_meas || !alpha_f || !beta_f || n == 0)
    return COMPASS_ERR_INVALID_ARG;
  if (n > 4096) return COMPASS_ERR_UNSUPPORTED;
  double xs[4096], ys[4096];
  size_t k = 0;
  for (size_t i = 0; i < n; ++i) {
    if (n_chunks[i] < 2) continue;
    xs[k] = m_volume[i];
    ys[k] = (t_meas[i] - fusion_time(t_comp[i], t_comm[i], n_chunks[i], 0.0, 0.0, m_volume[i])) / double(n_chunks[i] - 1);
    ++k;
  }
  return ols(xs, ys, k, alpha_f, beta_f) ? COMPASS_OK : COMPASS_ERR_INVALID_ARG;
}

namespace {

// What the calibrated linear models say about one workload (f and g of Algorithm 1).
struct BaseTimes {
  double t_comp, t_comm, volume;
};
BaseTimes base_times(const compass_problem* pr, const compass_calib* cal) {
  const double P = double(pr->P), M = double(pr->M);
  const double inner = double(pr->op == COMPASS_OP_AG_GEMM ? pr->K : pr->N);   // width of what the collective moves
  BaseTimes b;
  b.volume = M * inner;
  b.t_comp = cal->comp_a + cal->comp_b * (2.0 * P * M * double(pr->N) * double(pr->K));
  b.t_comm = cal->comm_a + cal->comm_b * (2.0 * P * b.volume);
  return b;
}

struct Prediction {
  int strategy;
  double time;
};

}  // namespace

// Algorithm 1 with Eq. 2-8: every strategy gets a predicted time, the fastest wins.
extern "C" int compass_select_ex(const compass_problem* pr, const compass_calib* cal, int eq5_as_printed,
                                 compass_choice* out) {
  if (!pr || !cal || !out) return COMPASS_ERR_INVALID_ARG;
  if (pr->op != COMPASS_OP_AG_GEMM && pr->op != COMPASS_OP_GEMM_RS) return COMPASS_ERR_INVALID_ARG;
  if (pr->P < 1) return COMPASS_ERR_INVALID_ARG;
  if (pr->M <= 0 || pr->N <= 0 || pr->K <= 0 || pr->M % pr->P != 0) return COMPASS_ERR_SHAPE;
  const BaseTimes w = base_times(pr, cal);
  const int degree = optimal_degree(w.t_comp, w.t_comm, cal->alpha_decomp, cal->beta_decomp, largest_degree(pr->M / pr->P),
                                    eq5_as_printed != 0, nullptr);
  // Listed in the order ties are resolved: a later entry replaces an earlier one only when strictly faster,
  // so equal predictions stay with InterDecom.
  const Prediction table[2] = {
      {COMPASS_STRATEGY_INTERDECOM, decomp_time(w.t_comp, w.t_comm, cal->alpha_decomp, cal->beta_decomp, degree)},
      {COMPASS_STRATEGY_INTRAFUSION,
       fusion_time(w.t_comp, w.t_comm, pr->P, cal->alpha_fusion, cal->beta_fusion, w.volume)},
  };
  int best = 0;
  for (int i = 1; i < 2; ++i)
    if (table[i].time < table[best].time) best = i;
  out->strategy = table[best].strategy;
  out->t_star = table[best].time;
  out->d_star = degree;
  out->t_decomp = table[0].time;
  out->t_fusion = table[1].time;
  out->t_comp = w.t_comp;
  out->t_comm = w.t_comm;
  out->lambda = w.t_comm > 0.0 ? w.t_comp / w.t_comm : INFINITY;
  return COMPASS_OK;
}

extern "C" int compass_select(const compass_problem* pr, const compass_calib* cal, compass_choice* out) {
  return compass_select_ex(pr, cal, 0, out);
}
