#include "hdet_scalars.h"

#include <algorithm>
#include <cmath>

namespace hdet {

void spread_multipliers(int n, double alpha, double* rho) {
  const double centre = 0.5 * (n - 1);
  const double delta = std::max(centre, 0.5);
  for (int r = 0; r < n; ++r) rho[r] = 1.0 + alpha * ((double)r - centre) / delta;
}

double base_rate(int kind, int64_t i, int64_t total_steps, double max_lr, double pct_start,
                 double div_factor, double final_div_factor) {
  if (kind == 0) return max_lr;
  // Two phases with real-valued boundaries: [0, p*S - 1] rising from max/div to max,
  // then [p*S - 1, S - 1] falling to max/(div*final_div).
  const double lo = max_lr / div_factor;
  const double floor_lr = lo / final_div_factor;
  const double knee = pct_start * (double)total_steps - 1.0;
  const double last = (double)total_steps - 1.0;
  const double x = std::min((double)i, last);  // past the last scheduled step the final rate is held
  double from, to, frac;
  if (x <= knee) {
    from = lo; to = max_lr; frac = x / knee;
  } else {
    from = max_lr; to = floor_lr; frac = (x - knee) / (last - knee);
  }
  if (kind == 1) return to + 0.5 * (from - to) * (1.0 + std::cos(M_PI * frac));
  return from + (to - from) * frac;
}

double decay_gamma(double f_div, double f_final, int64_t total_steps, int64_t warmup_steps, int64_t sync_interval) {
  const double intervals = (double)(total_steps - warmup_steps) / (double)sync_interval;
  if (!(intervals > 0.0)) return 0.0;
  return 1.0 - std::exp(-std::log(f_div / f_final) / intervals);
}

void softmax_weights(int n, const double* losses, double sigma, double* w) {
  double mean = 0.0;
  for (int r = 0; r < n; ++r) mean += losses[r];
  mean /= n;
  double top = -INFINITY;
  for (int r = 0; r < n; ++r) {
    w[r] = (mean - losses[r]) / sigma;
    top = std::max(top, w[r]);
  }
  double z = 0.0;
  for (int r = 0; r < n; ++r) {
    w[r] = std::exp(w[r] - top);
    z += w[r];
  }
  for (int r = 0; r < n; ++r) w[r] /= z;
}

uint64_t mix64(uint64_t x) {
  x = (x ^ (x >> 30)) * 0xBF58476D1CE4E5B9ull;
  x = (x ^ (x >> 27)) * 0x94D049BB133111EBull;
  return x ^ (x >> 31);
}

void draw_permutation(uint64_t seed, uint64_t sync_index, uint64_t channel, int n, int32_t* perm) {
  const uint64_t key = mix64(mix64(mix64(seed) + sync_index) + channel);
  for (int r = 0; r < n; ++r) perm[r] = r;
  for (int j = n - 1; j >= 1; --j) {
    const uint64_t u = mix64(key + (uint64_t)j * 0x9E3779B97F4A7C15ull);
    std::swap(perm[j], perm[(int)(u % (uint64_t)(j + 1))]);
  }
}

}  // namespace hdet
