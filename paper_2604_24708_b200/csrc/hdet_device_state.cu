#include "hdet_device_state.cuh"
#include "hdet_scalars.h"

namespace hdet {
namespace {

constexpr unsigned kFull = 0xffffffffu;

__device__ __forceinline__ double warp_sum(double x) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) x += __shfl_xor_sync(kFull, x, o);
  return x;
}
__device__ __forceinline__ double warp_max(double x) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) x = fmax(x, __shfl_xor_sync(kFull, x, o));
  return x;
}

// One warp; lane r holds replica r.
__global__ void __launch_bounds__(32) device_scalars_kernel(DevState* d, const DevConst c, const void* losses,
                                                            int loss_is_f64) {
  const int lane = threadIdx.x;
  hdet_state& st = d->st;
  StepScalars& sc = d->scal;
  const long long i = st.step;
  const long long t = i + 1;
  const bool fired = st.fired != 0;
  double bc1 = 1.0, bc2 = 1.0;
  if (c.adam) {
    bc1 = 1.0 - pow(c.beta1, (double)t);
    bc2 = 1.0 - pow(c.beta2, (double)t);
  }
  for (int g = 0; g < c.n_groups; ++g) {
    const double b = fired ? st.ctrl_base[g]
                           : base_rate(c.kind, i, c.total_steps, c.max_lr[g], c.pct_start, c.div_factor,
                                       c.final_div_factor);
    if (lane < c.n) {
      const double lr = b * spread_multiplier(c.n, c.alpha_lr, st.perm_lr[g][lane]);        // Eq. 1, Eq. 9
      const double wd = st.wd_base[g] * spread_multiplier(c.n, c.alpha_wd, st.perm_wd[g][lane]);
      st.lr[g][lane] = lr;
      st.wd[g][lane] = wd;
      sc.lr_wd[g][lane] = (float)(c.adam ? lr * wd : wd);
      sc.step[g][lane] = (float)(c.adam ? lr / bc1 : lr);
    }
    if (lane == 0) st.base[g] = b;
  }
  if (losses != nullptr && lane < c.n) {
    const double l = loss_is_f64 ? static_cast<const double*>(losses)[lane]
                                 : (double)static_cast<const float*>(losses)[lane];
    st.loss_acc[lane] += l;                                                                 // Algorithm 1: L_acc
  }
  __syncwarp();
  if (lane == 0) {
    sc.one_minus_beta1 = (float)(1.0 - c.beta1);
    sc.one_minus_beta2 = (float)(1.0 - c.beta2);
    sc.rsqrt_bc2 = (float)(1.0 / sqrt(bc2));
    sc.eps = (float)c.eps;
    sc.momentum = c.adam ? 0.0f : (float)c.momentum;
    sc.inv_n = 1.0 / (double)c.n;
    sc.n_replicas = c.n;
    st.n_acc += 1;
    st.step = t;
    st.round_ended = 0;
  }
}

__global__ void __launch_bounds__(32) device_round_end_kernel(DevState* d, const DevConst c) {
  const int lane = threadIdx.x;
  hdet_state& st = d->st;
  const bool active = lane < c.n;
  const long long t = st.step;
  const double L = active ? st.loss_acc[lane] / (double)st.n_acc : 0.0;   // mean loss of the round
  __syncwarp();
  if (active) {
    st.loss_round[lane] = L;
    st.loss_acc[lane] = 0.0;
  }
  if (lane == 0) st.n_acc = 0;
  if (!c.autolr || t < c.warmup_steps) return;

  // Eq. 4: softmax of (Lbar - L_r) / sigma over the replicas (lanes).
  const double mean = warp_sum(L) / (double)c.n;
  const double score = active ? (mean - L) / c.sigma : -INFINITY;
  const double top = warp_max(score);
  const double e = active ? exp(score - top) : 0.0;
  const double w = e / warp_sum(e);
  if (active) st.weights[lane] = w;
  const double gamma = decay_gamma(c.f_div, c.f_final, c.total_steps, c.warmup_steps, c.sync_interval);   // Eq. 8
  for (int g = 0; g < c.n_groups; ++g) {
    const double eta = active ? st.lr[g][lane] : 0.0;
    const double weighted = warp_sum(w * eta);                    // Eq. 5
    const double plain = warp_sum(eta) / (double)c.n;
    if (lane == 0) {
      const double delta = weighted - plain;                      // Eq. 6
      const double v = c.ctrl_beta * st.velocity[g] + (1.0 - c.ctrl_beta) * delta;   // Eq. 7
      st.delta[g] = delta;
      st.velocity[g] = v;
      st.ctrl_base[g] = plain * (1.0 - gamma) + v * c.lambda;
    }
    if (c.auto_wd) {   // Remark 1: the same update on the weight decays of the last step, without decay
      const double h = active ? st.wd[g][lane] : 0.0;
      const double w_wd = warp_sum(w * h);
      const double p_wd = warp_sum(h) / (double)c.n;
      if (lane == 0) {
        const double d_wd = w_wd - p_wd;
        const double v_wd = c.ctrl_beta * st.wd_velocity[g] + (1.0 - c.ctrl_beta) * d_wd;
        st.wd_delta[g] = d_wd;
        st.wd_velocity[g] = v_wd;
        st.wd_base[g] = p_wd + v_wd * c.lambda;
      }
    }
  }
  if (lane == 0) st.fired = 1;
  if (c.reshuffle && lane < 2 * c.n_groups) {                     // Eq. 9: one lane per channel
    const int g = lane >> 1;
    int32_t* perm = (lane & 1) ? st.perm_wd[g] : st.perm_lr[g];
    draw_permutation(c.seed, (unsigned long long)(t / c.sync_interval), (unsigned long long)lane, c.n, perm);
  }
}

}  // namespace

cudaError_t launch_device_scalars(DevState* d, const DevConst& c, const void* losses, int loss_is_f64,
                                  cudaStream_t stream) {
  device_scalars_kernel<<<1, 32, 0, stream>>>(d, c, losses, loss_is_f64);
  return cudaGetLastError();
}

cudaError_t launch_device_round_end(DevState* d, const DevConst& c, cudaStream_t stream) {
  device_round_end_kernel<<<1, 32, 0, stream>>>(d, c);
  return cudaGetLastError();
}

}  // namespace hdet
