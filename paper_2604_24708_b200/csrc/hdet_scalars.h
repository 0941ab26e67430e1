// Double-precision scalars of the HDET hot path: spread multipliers (Eq. 1), the one-cycle base
// schedule named in Algorithm 1's Require list, the controller (Eq. 4 - Eq. 8) and the permutation
// generator behind Eq. 9.  Written once for host and device: the host API evaluates them on the CPU,
// the device-resident stepping mode evaluates the same code in a one-warp kernel.
#pragma once
#include <cstdint>
#include <cmath>

#if defined(__CUDACC__)
#define HDET_HD __host__ __device__ inline
#else
#define HDET_HD inline
#endif

namespace hdet {

// rho_r of Eq. 1: 1 + alpha (r - (N-1)/2) / max((N-1)/2, 1/2).
HDET_HD double spread_multiplier(int n, double alpha, int r) {
  const double centre = 0.5 * (n - 1);
  const double delta = centre > 0.5 ? centre : 0.5;
  return 1.0 + alpha * ((double)r - centre) / delta;
}

HDET_HD void spread_multipliers(int n, double alpha, double* rho) {
  for (int r = 0; r < n; ++r) rho[r] = spread_multiplier(n, alpha, r);
}

// Base rate at 0-based step index i.  kind: 0 constant, 1 one-cycle cosine, 2 one-cycle linear.
// Two phases with real-valued boundaries: [0, p*S - 1] rising from max/div to max, then
// [p*S - 1, S - 1] falling to max/(div*final_div); past the last scheduled step the final rate is held.
HDET_HD double base_rate(int kind, int64_t i, int64_t total_steps, double max_lr, double pct_start,
                         double div_factor, double final_div_factor) {
  if (kind == 0) return max_lr;
  const double lo = max_lr / div_factor;
  const double floor_lr = lo / final_div_factor;
  const double knee = pct_start * (double)total_steps - 1.0;
  const double last = (double)total_steps - 1.0;
  const double x = (double)i < last ? (double)i : last;
  double from, to, frac;
  if (x <= knee) {
    from = lo; to = max_lr; frac = x / knee;
  } else {
    from = max_lr; to = floor_lr; frac = (x - knee) / (last - knee);
  }
  if (kind == 1) return to + 0.5 * (from - to) * (1.0 + cos(3.14159265358979323846 * frac));
  return from + (to - from) * frac;
}

// gamma of Eq. 8 with K = (S - S_warm) / T taken as a real number; K <= 0 gives 0.
HDET_HD double decay_gamma(double f_div, double f_final, int64_t total_steps, int64_t warmup_steps,
                           int64_t sync_interval) {
  const double intervals = (double)(total_steps - warmup_steps) / (double)sync_interval;
  if (!(intervals > 0.0)) return 0.0;
  return 1.0 - exp(-log(f_div / f_final) / intervals);
}

// w of Eq. 4 from the N round losses (the largest score is subtracted before exp).
HDET_HD void softmax_weights(int n, const double* losses, double sigma, double* w) {
  double mean = 0.0;
  for (int r = 0; r < n; ++r) mean += losses[r];
  mean /= n;
  double top = 0.0;
  for (int r = 0; r < n; ++r) {
    w[r] = (mean - losses[r]) / sigma;
    if (r == 0 || w[r] > top) top = w[r];
  }
  double z = 0.0;
  for (int r = 0; r < n; ++r) {
    w[r] = exp(w[r] - top);
    z += w[r];
  }
  for (int r = 0; r < n; ++r) w[r] /= z;
}

// 64-bit mixing function (finaliser of SplitMix64, Steele, Lea & Flood 2014).
HDET_HD uint64_t mix64(uint64_t x) {
  x = (x ^ (x >> 30)) * 0xBF58476D1CE4E5B9ull;
  x = (x ^ (x >> 27)) * 0x94D049BB133111EBull;
  return x ^ (x >> 31);
}

// pi of Eq. 9 for one channel at one sync: Fisher-Yates from the identity, j = n-1 .. 1,
// swap j with mix64(key + j * 0x9E3779B97F4A7C15) mod (j + 1),
// key = mix64(mix64(mix64(seed) + sync_index) + channel).
HDET_HD void draw_permutation(uint64_t seed, uint64_t sync_index, uint64_t channel, int n, int32_t* perm) {
  const uint64_t key = mix64(mix64(mix64(seed) + sync_index) + channel);
  for (int r = 0; r < n; ++r) perm[r] = r;
  for (int j = n - 1; j >= 1; --j) {
    const uint64_t u = mix64(key + (uint64_t)j * 0x9E3779B97F4A7C15ull);
    const int k = (int)(u % (uint64_t)(j + 1));
    const int32_t tmp = perm[j];
    perm[j] = perm[k];
    perm[k] = tmp;
  }
}

}  // namespace hdet
