// Host-only timing model of Lookahead Reasoning cycles and the strategy search of Section 3.3.
// Nothing here touches a device; it lives in the same library so that a scheduler has one thing to load.
#include <cmath>
#include <cstring>
#include <vector>

#include "lr_common.cuh"
#include "lr_cycle.h"

namespace {

bool bad_args(int32_t gamma, int64_t num, int64_t den, const uint8_t *v, int64_t n, const lr_cycle_stats *out, const char *who) {
  if (gamma < 1 || num < 0 || den < 1 || n < 0 || (n > 0 && v == nullptr) || out == nullptr) {
    lr::set_error("%s: needs gamma >= 1, num >= 0, den >= 1, a verdict stream and an output", who);
    return true;
  }
  return false;
}

double f_sync(int k, double a, double c) { return (1.0 - std::pow(a, k)) / ((1.0 - a) * (1.0 - c + c * k)); }

double f_async(int k, double a, double c) {
  if (k >= (int)std::ceil(1.0 / c)) return 1.0 / (c + (1.0 - c) * (1.0 - a));  // the draft model is the limit
  const double ak = std::pow(a, k);
  return (1.0 - ak) / ((1.0 - a) + c * (a - ak * a - k * (1.0 - a) * ak));      // the depth is the limit
}

bool rate_ok(double x) { return x > 0.0 && x < 1.0; }

}  // namespace

extern "C" int lr_cycle_simulate_sync(int32_t gamma, int64_t num, int64_t den, const uint8_t *v, int64_t n, lr_cycle_stats *out) {
  if (bad_args(gamma, num, den, v, n, out, "lr_cycle_simulate_sync")) return LR_EINVAL;
  memset(out, 0, sizeof(*out));
  const int64_t per = gamma - 1, cycles = per > 0 ? n / per : n;
  for (int64_t cyc = 0; cyc < cycles; ++cyc) {
    int64_t accepted = 0;
    while (accepted < per && v[cyc * per + accepted]) ++accepted;
    out->steps += accepted + 1;
  }
  out->stages = cycles;
  out->time = cycles * (per * num + den);
  out->verdicts_used = cycles * per;
  out->peak_in_flight = cycles > 0 ? gamma : 0;
  return LR_OK;
}

extern "C" int lr_cycle_simulate_async(int32_t gamma, int64_t num, int64_t den, const uint8_t *v, int64_t n, lr_cycle_stats *out) {
  if (bad_args(gamma, num, den, v, n, out, "lr_cycle_simulate_async")) return LR_EINVAL;
  memset(out, 0, sizeof(*out));
  // start times of the last gamma positions of the current stage (a ring): position i may start once the
  // draft model is free (start[i-1] + num) and generation i - gamma is done (start[i-gamma] + den)
  std::vector<int64_t> ring((size_t)gamma, 0);
  int64_t pos = 0, prev = 0, used = 0, stage_peak = 0;  // stage_peak counts only once its stage is whole
  for (int64_t i = 0; i < n; ++i) {
    int64_t t = pos == 0 ? 0 : prev + num;
    if (pos >= gamma) t = std::max(t, ring[(size_t)(pos % gamma)] + den);
    ring[(size_t)(pos % gamma)] = t;
    prev = t;
    // generations in flight at t: the earlier positions of the ring that have not finished, and this one
    int64_t in_flight = 0;
    const int64_t lo = std::max<int64_t>(0, pos - gamma + 1);
    for (int64_t j = lo; j <= pos; ++j) in_flight += ring[(size_t)(j % gamma)] + den > t;
    stage_peak = std::max(stage_peak, in_flight);
    if (v[i]) {
      ++pos;
      continue;
    }
    out->time += t + den;   // the rejected draft is found when the target's step of this position is done
    out->steps += pos + 1;  // the accepted drafts and that step
    out->stages += 1;
    out->peak_in_flight = std::max(out->peak_in_flight, stage_peak);
    used = i + 1;
    pos = 0;
    stage_peak = 0;
  }
  out->verdicts_used = used;
  return LR_OK;
}

extern "C" double lr_cycle_speedup(int32_t mode, int32_t k, double alpha, double c) {
  if (k < 1 || !rate_ok(alpha) || !rate_ok(c) || mode < 0 || mode > 2) return NAN;
  return mode == 1 ? f_async(k, alpha, c) : f_sync(k, alpha, c);  // g(k2) has f_sync's form
}

extern "C" int lr_cycle_best_strategy(int32_t budget, double a1, double c1, double a2, double c2, int32_t asynchronous,
                                      int32_t *k1_out, int32_t *k2_out, double *h_out) {
  if (budget < 1 || !rate_ok(a1) || !rate_ok(c1) || !rate_ok(a2) || !rate_ok(c2) || !k1_out || !k2_out || !h_out) {
    lr::set_error("lr_cycle_best_strategy: needs budget >= 1, rates and costs in (0, 1) and three outputs");
    return LR_EINVAL;
  }
  const int cap = (int)std::ceil(1.0 / c1);
  double best = -1.0;
  int bk1 = 1, bk2 = 1;
  for (int k1 = 1; k1 <= budget; ++k1) {
    const int dim_f = asynchronous ? std::min(cap, k1) : k1;
    const double f = asynchronous ? f_async(k1, a1, c1) : f_sync(k1, a1, c1);
    for (int k2 = 1; k2 <= budget && dim_f * k2 <= budget; ++k2) {
      const double h = f * f_sync(k2, a2, c2);
      if (h > best) {
        best = h;
        bk1 = k1;
        bk2 = k2;
      }
    }
  }
  *k1_out = bk1;
  *k2_out = bk2;
  *h_out = best;
  return LR_OK;
}
