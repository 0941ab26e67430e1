// Host-side double-precision scalars of the HDET hot path: spread multipliers (Eq. 1),
// the one-cycle base schedule named in Algorithm 1's Require list, the controller
// (Eq. 4 - Eq. 8) and the permutation generator behind Eq. 9.
#pragma once
#include <cstdint>

namespace hdet {

// rho_r of Eq. 1 for r = 0 .. n-1.
void spread_multipliers(int n, double alpha, double* rho);

// Base rate at 0-based step index i.  kind: 0 constant, 1 one-cycle cosine, 2 one-cycle linear.
double base_rate(int kind, int64_t i, int64_t total_steps, double max_lr, double pct_start,
                 double div_factor, double final_div_factor);

// gamma of Eq. 8 with K = (S - S_warm) / T taken as a real number; K <= 0 gives 0.
double decay_gamma(double f_div, double f_final, int64_t total_steps, int64_t warmup_steps, int64_t sync_interval);

// w of Eq. 4 from the N round losses.
void softmax_weights(int n, const double* losses, double sigma, double* w);

// 64-bit mixing function (finaliser of SplitMix64, Steele, Lea & Flood 2014).
uint64_t mix64(uint64_t x);

// pi of Eq. 9 for one channel at one sync: Fisher-Yates from the identity, j = n-1 .. 1,
// swap j with mix64(key + j * 0x9E3779B97F4A7C15) mod (j + 1),
// key = mix64(mix64(mix64(seed) + sync_index) + channel).
void draw_permutation(uint64_t seed, uint64_t sync_index, uint64_t channel, int n, int32_t* perm);

}  // namespace hdet
