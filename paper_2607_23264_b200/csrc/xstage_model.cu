// Host-side X-Stage (Burst-Gap) calculator: include/xstage.h.  Pure double-precision arithmetic, no GPU work.
#include <algorithm>
#include <cmath>
#include <limits>
#include <vector>

#include "../../include/xstage.h"

namespace {
inline double pos(double z) { return z > 0.0 ? z : 0.0; }
inline bool ok(const xstage_params* m) { return m && m->rate > 0.0 && m->t_iss0 >= 0.0; }
const double kNaN = std::numeric_limits<double>::quiet_NaN();
double median_of(std::vector<double> v) {
  std::sort(v.begin(), v.end());
  const size_t n = v.size();
  return n % 2 ? v[n / 2] : 0.5 * (v[n / 2 - 1] + v[n / 2]);
}
}  // namespace

extern "C" {

int xstage_calibrate(int64_t n_periodic, const double* p_volume, const double* p_gap, const double* p_t_iss,
                     const double* p_t_period, int64_t n_isolated, const double* i_volume, const double* i_t_iss,
                     double knee_tolerance, xstage_calibration* out) {
  if (!out || n_periodic < 1 || !p_volume || !p_gap || !p_t_iss || !p_t_period || n_isolated < 0 ||
      (n_isolated > 0 && (!i_volume || !i_t_iss)) || !(knee_tolerance >= 0.0))
    return -1;
  *out = xstage_calibration{};
  // the plateau: rows whose gap is among the largest third of the distinct gaps
  std::vector<double> gaps(p_gap, p_gap + n_periodic);
  std::sort(gaps.begin(), gaps.end());
  gaps.erase(std::unique(gaps.begin(), gaps.end()), gaps.end());
  const size_t third = std::max<size_t>(1, gaps.size() / 3);
  const double threshold = gaps[gaps.size() - third];
  std::vector<double> plateau, rates;
  for (int64_t i = 0; i < n_periodic; ++i) {
    if (p_gap[i] >= threshold) plateau.push_back(p_t_iss[i]);
    if (p_gap[i] == 0.0) {
      if (!(p_t_period[i] > 0.0)) return -1;
      rates.push_back(p_volume[i] / p_t_period[i]);
    }
  }
  out->t_iss0 = median_of(plateau);
  out->rate = rates.empty() ? 0.0 : median_of(rates);
  if (n_isolated < 3 || rates.empty()) return 0;
  // least-squares line through the smallest third of the isolated volumes
  const int64_t n = std::max<int64_t>(3, n_isolated / 3);
  double mx = 0.0, my = 0.0;
  for (int64_t i = 0; i < n; ++i) {
    mx += i_volume[i];
    my += i_t_iss[i];
  }
  mx /= n;
  my /= n;
  double sxx = 0.0, sxy = 0.0;
  for (int64_t i = 0; i < n; ++i) {
    sxx += (i_volume[i] - mx) * (i_volume[i] - mx);
    sxy += (i_volume[i] - mx) * (i_t_iss[i] - my);
  }
  const double b = sxx > 0.0 ? sxy / sxx : 0.0;
  const double a = my - b * mx;
  out->floor_intercept = a;
  out->floor_per_byte = b;
  for (int64_t i = n; i < n_isolated; ++i) {
    if (i_t_iss[i] > (1.0 + knee_tolerance) * (a + b * i_volume[i])) {
      out->has_knee = 1;
      out->knee_volume = i_volume[i - 1];
      out->capacity = pos(i_volume[i - 1] - out->rate * i_t_iss[i - 1]);
      break;
    }
  }
  return 0;
}

int xstage_burst_gap(const xstage_params* m, double volume, double gap, double* t_period, double* t_iss) {
  if (!ok(m) || volume < 0.0 || gap < 0.0) return -1;
  const double drain = volume / m->rate;
  if (t_period) *t_period = std::fmax(m->t_iss0 + gap, drain);
  if (t_iss) *t_iss = std::fmax(m->t_iss0, drain - gap);
  return 0;
}

double xstage_recovery_gap(const xstage_params* m, double volume) {
  if (!ok(m) || volume < 0.0) return kNaN;
  return pos(volume / m->rate - m->t_iss0);
}

double xstage_isolated_occupancy(const xstage_params* m, double volume) {
  if (!ok(m) || volume < 0.0) return kNaN;
  return pos(volume - m->rate * m->t_iss0);
}

int64_t xstage_audit(const xstage_params* m, int64_t count, const double* volume, const double* floor,
                     const double* gap, double q_initial, double* rho, double* delta_b, double* backlog,
                     int32_t* guard_ok) {
  if (!ok(m) || count < 0 || (count > 0 && (!volume || !gap)) || q_initial < 0.0) return -1;
  double q = q_initial;
  int64_t first_fail = count;
  if (backlog) backlog[0] = q;
  for (int64_t n = 0; n < count; ++n) {
    const double f = floor ? floor[n] : m->t_iss0;
    const double period = f + gap[n];
    if (!(period > 0.0) || volume[n] < 0.0) return -1;
    const double drained = m->rate * period;
    const double db = volume[n] - drained;
    const bool guard = q + pos(volume[n] - m->rate * f) <= m->capacity;
    if (rho) rho[n] = volume[n] / drained;
    if (delta_b) delta_b[n] = db;
    if (guard_ok) guard_ok[n] = guard ? 1 : 0;
    if (!guard && first_fail == count) first_fail = n;
    q = pos(q + db);
    if (backlog) backlog[n + 1] = q;
  }
  return first_fail;
}

double xstage_interleaved_gap(double t_l2_mma, double t_l1_mma, double n1, double n2) {
  if (!(n2 > 0.0) || n1 < 0.0) return kNaN;
  return t_l2_mma + (n1 / n2) * t_l1_mma;
}

double xstage_interleaved_issue_overhead(double overhead_wave, double t_l1_mma, double n1, double n2) {
  if (!(n2 > 0.0) || n1 < 0.0) return kNaN;
  return pos(overhead_wave - (n1 / n2) * t_l1_mma);
}

int xstage_average_rate_feasible(const xstage_params* m, double volume, double t_l2_mma, double t_l1_mma,
                                 double n1, double n2) {
  if (!ok(m) || !(n2 > 0.0) || n1 < 0.0 || volume < 0.0) return -1;
  const double cycle = n2 * (m->t_iss0 + t_l2_mma) + n1 * t_l1_mma;
  if (!(cycle > 0.0)) return -1;
  return (n2 * volume / cycle <= m->rate) ? 1 : 0;
}

int64_t xstage_lead_knee(int64_t b_n, int64_t k_sm, int64_t h_inter) {
  if (b_n <= 0 || k_sm <= 0 || h_inter <= 0) return -1;
  const int64_t num = b_n * k_sm, den = 2 * h_inter;
  return (num + den - 1) / den;
}

double xstage_mma_stall(double t_remote_store_span, double t_cover_mma) {
  return pos(t_remote_store_span - t_cover_mma);
}

int64_t xstage_fa_recovery_length(int64_t b_n, double recovery_gap, double sigma) {
  if (b_n <= 0 || !(sigma > 0.0) || recovery_gap < 0.0) return -1;
  return b_n * static_cast<int64_t>(std::ceil(recovery_gap / sigma));
}

}  // extern "C"
