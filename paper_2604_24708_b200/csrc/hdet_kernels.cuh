// Device-side data structures and launchers of the fan-out / converge kernels.
#pragma once
#include <cuda_runtime.h>

#include <cstdint>

#include "../../include/hdet.h"

namespace hdet {

// One tile = kTileVecs float4 vectors per thread of a kThreads-wide CTA.
constexpr int kThreads = 256;
constexpr int kTileVecs = 2;
constexpr int kTileElems = kThreads * 4 * kTileVecs;  // 2048 elements

// Bits of TensorDesc::vec.
constexpr int kVecLoads = 1;
constexpr int kVecBulk = 2;

// Per-tensor descriptor, resident on the device (built once by hdet_create).
struct TensorDesc {
  float* param;
  const void* grad;
  float* exp_avg;
  float* exp_avg_sq;
  long long numel;
  long long param_stride;
  long long grad_stride;
  long long state_stride;  // 0: one pair of moments shared by all replicas
  int group;
  int vec;  // kVecLoads: pointers and strides allow 128-bit accesses; | kVecBulk: also 16-byte bulk copies of whole tiles
  long long partial_off;  // element offset of this tensor inside the partial-sum staging buffer (multiple of 4)
  float* partial;         // set per tile by the kernels (NULL in the table)
  unsigned short* param_bf16;  // optional bf16 copy of the averaged parameters (one copy), or NULL
};

// One unit of work: tile `tile` (kTileElems elements) of tensor `tensor`.
struct Tile {
  int tensor;
  int tile;
};

// Per-launch scalars, passed by value as kernel parameters (no device table to update).
struct StepScalars {
  float lr_wd[HDET_MAX_GROUPS][HDET_MAX_REPLICAS];  // AdamW: lr * wd (decoupled decay factor is 1 - lr_wd); SGD: wd
  float step[HDET_MAX_GROUPS][HDET_MAX_REPLICAS];   // AdamW: lr / (1 - beta1^t); SGD: lr
  float one_minus_beta1, one_minus_beta2;
  float rsqrt_bc2;  // 1 / sqrt(1 - beta2^t)
  float eps;
  float momentum;   // SGD momentum (0 = none)
  double inv_n;     // 1 / N
  int n_replicas;
};

// fp32 -> bfloat16 bit pattern, round to nearest even.
__device__ __forceinline__ unsigned short bf16_bits(float x) {
  const unsigned u = __float_as_uint(x);
  if ((u & 0x7FFFFFFFu) > 0x7F800000u) return (unsigned short)((u >> 16) | 0x40u);   // a NaN stays a NaN
  return (unsigned short)((u + 0x7FFFu + ((u >> 16) & 1u)) >> 16);
}
__device__ __forceinline__ uint2 bf16_bits4(const float4& x) {
  return make_uint2((unsigned)bf16_bits(x.x) | ((unsigned)bf16_bits(x.y) << 16),
                    (unsigned)bf16_bits(x.z) | ((unsigned)bf16_bits(x.w) << 16));
}

// Eq. 3 on one tile: every replica <- (1/N) sum over replicas, fp64 accumulation r = 0..N-1, one rounding.
// The one statement of the stand-alone mean; hdet_converge and hdet_converge_static both run it.
__device__ __forceinline__ void converge_tile(const TensorDesc& td, int tile_index, int n, double inv_n) {
  const long long off = (long long)tile_index * kTileElems;
  const long long rest = td.numel - off;
  const int len = rest < kTileElems ? (int)rest : kTileElems;
  const int nvec = td.vec ? (len >> 2) : 0;
  float* const P = td.param + off;
  for (int j = threadIdx.x; j < nvec; j += kThreads) {
    double s0 = 0.0, s1 = 0.0, s2 = 0.0, s3 = 0.0;
#pragma unroll 4
    for (int r = 0; r < n; ++r) {
      const float4 x = __ldcs(reinterpret_cast<const float4*>(P + r * td.param_stride + 4 * j));
      s0 += (double)x.x; s1 += (double)x.y; s2 += (double)x.z; s3 += (double)x.w;
    }
    const float4 mean = make_float4((float)(s0 * inv_n), (float)(s1 * inv_n), (float)(s2 * inv_n), (float)(s3 * inv_n));
    for (int r = 0; r < n; ++r) __stcs(reinterpret_cast<float4*>(P + r * td.param_stride + 4 * j), mean);
    if (td.param_bf16) __stcs(reinterpret_cast<uint2*>(td.param_bf16 + off + 4 * j), bf16_bits4(mean));
  }
  for (int e = 4 * nvec + threadIdx.x; e < len; e += kThreads) {
    double sum = 0.0;
    for (int r = 0; r < n; ++r) sum += (double)__ldcs(P + r * td.param_stride + e);
    const float mean = (float)(sum * inv_n);
    for (int r = 0; r < n; ++r) __stcs(P + r * td.param_stride + e, mean);
    if (td.param_bf16) td.param_bf16[off + e] = bf16_bits(mean);
  }
}

struct LaunchPlan {
  const TensorDesc* tensors;
  const Tile* tiles;
  int n_tiles;
  int grid;            // CTAs to launch; each takes tiles blockIdx.x, blockIdx.x + grid, ...
  unsigned* status;    // device status word; bit 0 = non-finite parameter seen
  const StepScalars* scal_dev;  // device-resident launch scalars; NULL = use the by-value kernel parameter
  float* partial;      // non-NULL: a fused converge writes local replica sums here instead of the mean
};

// Fan-out update of every replica of every tile (Eq. 2 or Adam); with `converge` the
// replica mean (Eq. 3) is formed from the updated values and written to all replicas.
// `grad_mean`: every replica steps with the replica mean of the gradients (Algorithm 1's gradient
// all-reduce).  `shared_state`: AdamW with one pair of moments for all replicas (state_stride 0).
// `sgd_momentum`: SGD keeps a momentum buffer in exp_avg.
cudaError_t launch_fanout(int optimizer, bool sgd_momentum, int grad_dtype, bool converge, bool grad_mean,
                          bool shared_state, const LaunchPlan& plan, const StepScalars& s, cudaStream_t stream);

// Per device, before the first launch: lets the bulk-copy kernels this handle will use take their shared-memory
// ring (an attribute of the kernel).  Called by hdet_create so that no attribute call falls into a stream capture.
cudaError_t prepare_fanout(int optimizer, int grad_dtype, bool grad_mean, bool shared_state);

// Eq. 10: every replica <- replica 0 + N(0, nu^2 ||replica 0||^2 / total_numel) noise.  `scratch` holds
// n_tiles + 1 doubles.  Three launches.
cudaError_t launch_warm_init(const LaunchPlan& plan, int n_replicas, int replica_offset, double nu, double total_numel,
                             unsigned long long seed, double* scratch, cudaStream_t stream);

// Every local replica <- plan.partial * inv_n_global (the all-reduced sums of a sharded converge).
cudaError_t launch_apply_mean(const LaunchPlan& plan, int n_local, double inv_n_global, cudaStream_t stream);

// The same with the exchange done by the kernel: every local replica <- (sum over the n_buffers staging buffers,
// in the given order) * inv_n_global.  The buffers may live on other GPUs (plain peer loads).
cudaError_t launch_apply_mean_peers(const LaunchPlan& plan, const float* const* buffers, int n_buffers, int n_local,
                                    double inv_n_global, cudaStream_t stream);

// Diagnostic: a one-CTA kernel whose bounded barrier wait runs out (about a second) and sets bit 1 of *status.
cudaError_t launch_bounded_wait_probe(unsigned* status, cudaStream_t stream);

// Stand-alone Eq. 3.
cudaError_t launch_converge(const LaunchPlan& plan, int n_replicas, cudaStream_t stream);

}  // namespace hdet
