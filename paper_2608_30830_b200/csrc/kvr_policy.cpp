// Host-side arithmetic of the retention policy that drives the mover: break-evens, congestion price,
// load-indexed host timer, finite-capacity replay and branch selection.  No CUDA in this file.
#include <cmath>
#include <cstdint>
#include <functional>
#include <limits>
#include <queue>
#include <vector>

#include "../../include/kvr.h"

namespace {

constexpr double kInf = std::numeric_limits<double>::infinity();

bool valid(const kvr_prices *p) { return p && p->alpha1 > 0 && p->beta2 >= 0 && p->beta3 > p->beta2; }

// one pass over the arrivals with a min-heap of slot departure times
void replay(const double *arrive, const double *wait, int64_t n, int64_t c2, double ttl, const kvr_prices *p,
            double *mean_cost, double *from_host) {
  std::priority_queue<double, std::vector<double>, std::greater<double>> leaving;
  double total = 0;
  int64_t hits = 0;
  for (int64_t i = 0; i < n; ++i) {
    const double a = arrive[i], w = wait[i];
    while (!leaving.empty() && leaving.top() <= a) leaving.pop();
    if ((int64_t)leaving.size() < c2) {
      leaving.push(a + (w < ttl ? w : ttl));
      if (w <= ttl) { total += p->beta2; ++hits; } else total += p->beta3;
    } else {
      total += p->beta3;
    }
  }
  *mean_cost = n ? total / (double)n : 0.0;
  *from_host = n ? (double)hits / (double)n : 0.0;
}

}  // namespace

extern "C" {

kvr_status kvr_policy_break_evens(const kvr_prices *p, double *t1, double *t_star) {
  if (!valid(p) || !t1 || !t_star) return KVR_ERR_INVALID_ARG;
  *t1 = p->beta2 / p->alpha1;
  *t_star = p->beta3 / p->alpha1;
  return KVR_OK;
}

kvr_status kvr_policy_host_ttl(const kvr_prices *p, double lambda, double c2, double w_ref, double *alpha2, double *t2) {
  if (!valid(p) || !(c2 > 0) || !(w_ref > 0) || lambda < 0) return KVR_ERR_INVALID_ARG;
  const double lambda_crit = c2 / w_ref;
  const double excess = lambda - lambda_crit;
  const double a2 = (excess > 0 ? excess : 0.0) * p->beta3 / c2;
  if (alpha2) *alpha2 = a2;
  if (t2) *t2 = lambda <= lambda_crit ? kInf : (p->beta3 - p->beta2) / a2;
  return KVR_OK;
}

kvr_status kvr_policy_replay(const kvr_prices *p, const double *arrive, const double *wait, int64_t n, int64_t c2,
                             double ttl, double *mean_cost, double *from_host) {
  if (!valid(p) || n < 0 || (n > 0 && (!arrive || !wait)) || c2 < 0 || !(ttl >= 0) || !mean_cost || !from_host)
    return KVR_ERR_INVALID_ARG;
  for (int64_t i = 1; i < n; ++i) if (arrive[i] < arrive[i - 1]) return KVR_ERR_INVALID_ARG;
  replay(arrive, wait, n, c2, ttl, p, mean_cost, from_host);
  return KVR_OK;
}

kvr_status kvr_policy_select(const kvr_prices *p, const double *arrive, const double *wait, int64_t n, double lambda,
                             int64_t c2, double w_ref, int32_t *use_ttl, double *cost_retain, double *cost_ttl, double *t2) {
  double ttl = 0, a2 = 0;
  if (kvr_status s = kvr_policy_host_ttl(p, lambda, (double)c2, w_ref, &a2, &ttl)) return s;
  double cr = 0, ct = 0, f = 0;
  if (kvr_status s = kvr_policy_replay(p, arrive, wait, n, c2, kInf, &cr, &f)) return s;
  if (kvr_status s = kvr_policy_replay(p, arrive, wait, n, c2, ttl, &ct, &f)) return s;
  if (use_ttl) *use_ttl = ct < cr ? 1 : 0;
  if (cost_retain) *cost_retain = cr;
  if (cost_ttl) *cost_ttl = ct;
  if (t2) *t2 = ttl;
  return KVR_OK;
}

}  // extern "C"
