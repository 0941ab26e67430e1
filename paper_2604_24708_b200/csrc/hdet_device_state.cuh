// Device-resident copy of Algorithm 1's scalar state and the one-warp kernels that advance it, so that
// a step needs no host arithmetic, no host-to-device copy and no read-back of the losses.
#pragma once
#include <cuda_runtime.h>

#include "hdet_kernels.cuh"

namespace hdet {

// Constants of a handle (configuration + schedule), passed by value to the scalar kernels.
struct DevConst {
  int n, n_groups, adam, kind, autolr, auto_wd, reshuffle;
  long long total_steps, warmup_steps, sync_interval;
  double beta1, beta2, eps, momentum, alpha_lr, alpha_wd;
  double pct_start, div_factor, final_div_factor;
  double ctrl_beta, sigma, lambda, f_div, f_final;
  double max_lr[HDET_MAX_GROUPS], weight_decay[HDET_MAX_GROUPS];
  unsigned long long seed;
};

// What lives on the device: the launch scalars the fan-out kernels read, and the state block
// (same layout as the public hdet_state, so get/set are plain copies).
struct DevState {
  StepScalars scal;
  hdet_state st;
};

// Before the fan-out kernel of a step: rates, decays and bias corrections for update t = st.step + 1
// (Eq. 1, schedule, Eq. 9 permutations) into `scal`; adds the step's losses (device array of N
// doubles or floats, may be NULL) to the round accumulator; advances the step counter.
cudaError_t launch_device_scalars(DevState* d, const DevConst& c, const void* losses, int loss_is_f64,
                                  cudaStream_t stream);

// After the fan-out kernel of a round's last step: latches the round's mean losses and, when auto-LR
// is on and t >= S_warm, runs the controller (Eq. 4 - Eq. 9).
cudaError_t launch_device_round_end(DevState* d, const DevConst& c, cudaStream_t stream);

}  // namespace hdet
