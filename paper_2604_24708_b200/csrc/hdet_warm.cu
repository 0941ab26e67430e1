// Warm noisy initialisation (Section 3.5, Eq. 10): theta_r <- theta_bar_0 + eps_r with
// eps_r ~ N(0, nu^2 ||theta_bar_0||^2 / d), independent per replica and parameter.
//
// Three kernels: per-tile sums of squares of the checkpoint (replica 0) in fp64; one CTA that adds the
// partial sums in a fixed order and writes sigma = nu sqrt(||theta_bar_0||^2 / d); and the fan-out of the
// checkpoint plus noise to all N replicas, one CTA per tile streaming every replica of the tile.  The
// noise is counter-based (any element can be drawn on its own), so results do not depend on the launch
// shape: key = mix64(mix64(mix64(mix64(seed) + "WARM") + replica) + tensor); the element pair p = e / 2
// takes u = mix64(key + p * 0x9E3779B97F4A7C15), u1 = ((u >> 41) + 0.5) / 2^23,
// u2 = ((u >> 16) & 0xFFFFFF) / 2^24, and Box-Muller gives z_even = sqrt(-2 ln u1) cos(2 pi u2),
// z_odd = sqrt(-2 ln u1) sin(2 pi u2).
#include "hdet_kernels.cuh"
#include "hdet_scalars.h"

namespace hdet {
namespace {

constexpr unsigned long long kGolden = 0x9E3779B97F4A7C15ull;

__device__ __forceinline__ double block_sum(double x, double* smem) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) x += __shfl_xor_sync(0xffffffffu, x, o);
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  if (lane == 0) smem[warp] = x;
  __syncthreads();
  double total = 0.0;
  if (threadIdx.x == 0)
    for (int w = 0; w < (int)(blockDim.x >> 5); ++w) total += smem[w];
  __syncthreads();
  return total;  // valid on thread 0
}

__global__ void __launch_bounds__(kThreads, 4) warm_norm_kernel(const __grid_constant__ LaunchPlan plan, double* partial) {
  __shared__ double smem[kThreads / 32];
  for (int t = blockIdx.x; t < plan.n_tiles; t += gridDim.x) {
    const Tile tile = plan.tiles[t];
    const TensorDesc td = plan.tensors[tile.tensor];
    const long long off = (long long)tile.tile * kTileElems;
    const long long rest = td.numel - off;
    const int len = rest < kTileElems ? (int)rest : kTileElems;
    const int nvec = td.vec ? (len >> 2) : 0;
    const float* P = td.param + off;   // replica 0 holds the checkpoint
    double acc = 0.0;
    for (int j = threadIdx.x; j < nvec; j += kThreads) {
      const float4 x = __ldcs(reinterpret_cast<const float4*>(P + 4 * j));
      acc += (double)x.x * x.x + (double)x.y * x.y + (double)x.z * x.z + (double)x.w * x.w;
    }
    for (int e = 4 * nvec + threadIdx.x; e < len; e += kThreads) {
      const float x = __ldcs(P + e);
      acc += (double)x * x;
    }
    const double total = block_sum(acc, smem);
    if (threadIdx.x == 0) partial[t] = total;
  }
}

// One CTA: fixed assignment of partial sums to threads, fixed reduction order.
__global__ void __launch_bounds__(1024) warm_sigma_kernel(const double* partial, int n_tiles, double nu, double d,
                                                          double* sigma_out) {
  __shared__ double smem[32];
  double acc = 0.0;
  for (int i = threadIdx.x; i < n_tiles; i += blockDim.x) acc += partial[i];
  const double total = block_sum(acc, smem);
  if (threadIdx.x == 0) *sigma_out = nu * sqrt(total / d);
}

// Two standard normal draws for the element pair p of (replica, tensor) key `key`.
__device__ __forceinline__ void gaussian_pair(unsigned long long key, unsigned long long p, float& z_even, float& z_odd) {
  const unsigned long long u = mix64(key + p * kGolden);
  const float u1 = ((float)(unsigned)(u >> 41) + 0.5f) * (1.0f / 8388608.0f);
  const float u2 = (float)(unsigned)((u >> 16) & 0xFFFFFFull) * (1.0f / 16777216.0f);
  // logf stays exact-rounded (u1 can be within 2^-24 of 1, where a fast log would lose the radius);
  // sine and cosine use the fast intrinsics on an angle reduced to [-pi, pi): cos(a + pi) = -cos a.
  const float radius = sqrtf(-2.0f * logf(u1));
  float s, c;
  __sincosf(6.283185307179586f * (u2 - 0.5f), &s, &c);
  z_even = -radius * c;
  z_odd = -radius * s;
}

__global__ void __launch_bounds__(kThreads, 4)
warm_noise_kernel(const __grid_constant__ LaunchPlan plan, const double* sigma_ptr, int n, unsigned long long base_key) {
  const float sigma = (float)(*sigma_ptr);
  __shared__ unsigned long long keys[HDET_MAX_REPLICAS];   // one key per replica for the tile's tensor
  for (int t = blockIdx.x; t < plan.n_tiles; t += gridDim.x) {
    const Tile tile = plan.tiles[t];
    __syncthreads();
    if (threadIdx.x < n)
      keys[threadIdx.x] = mix64(mix64(base_key + (unsigned long long)threadIdx.x) + (unsigned long long)tile.tensor);
    __syncthreads();
    const TensorDesc td = plan.tensors[tile.tensor];
    const long long off = (long long)tile.tile * kTileElems;
    const long long rest = td.numel - off;
    const int len = rest < kTileElems ? (int)rest : kTileElems;
    const int nvec = td.vec ? (len >> 2) : 0;
    float* const P = td.param + off;
    for (int j = threadIdx.x; j < nvec; j += kThreads) {
      const float4 x0 = __ldcs(reinterpret_cast<const float4*>(P + 4 * j));       // checkpoint, read once
      const unsigned long long p = (unsigned long long)(off + 4 * j) >> 1;        // first of two element pairs
      for (int r = 0; r < n; ++r) {
        const unsigned long long key = keys[r];
        float z0, z1, z2, z3;
        gaussian_pair(key, p, z0, z1);
        gaussian_pair(key, p + 1, z2, z3);
        __stcs(reinterpret_cast<float4*>(P + r * td.param_stride + 4 * j),
               make_float4(fmaf(sigma, z0, x0.x), fmaf(sigma, z1, x0.y), fmaf(sigma, z2, x0.z), fmaf(sigma, z3, x0.w)));
      }
    }
    for (int e = 4 * nvec + threadIdx.x; e < len; e += kThreads) {
      const float x0 = __ldcs(P + e);
      const unsigned long long elem = (unsigned long long)(off + e);
      for (int r = 0; r < n; ++r) {
        const unsigned long long key = keys[r];
        float ze, zo;
        gaussian_pair(key, elem >> 1, ze, zo);
        __stcs(P + r * td.param_stride + e, fmaf(sigma, (elem & 1) ? zo : ze, x0));
      }
    }
  }
}

}  // namespace

cudaError_t launch_warm_init(const LaunchPlan& plan, int n_replicas, int replica_offset, double nu, double total_numel,
                             unsigned long long seed, double* scratch, cudaStream_t stream) {
  if (plan.n_tiles == 0) return cudaSuccess;
  double* partial = scratch;                 // n_tiles partial sums
  double* sigma = scratch + plan.n_tiles;    // then sigma
  warm_norm_kernel<<<plan.grid, kThreads, 0, stream>>>(plan, partial);
  cudaError_t e = cudaGetLastError();
  if (e != cudaSuccess) return e;
  warm_sigma_kernel<<<1, 1024, 0, stream>>>(partial, plan.n_tiles, nu, total_numel, sigma);
  e = cudaGetLastError();
  if (e != cudaSuccess) return e;
  // local replica r draws the noise of global replica replica_offset + r
  const unsigned long long base_key = mix64(mix64(seed) + 0x5741524Dull) + (unsigned long long)replica_offset;
  warm_noise_kernel<<<plan.grid, kThreads, 0, stream>>>(plan, sigma, n_replicas, base_key);
  return cudaGetLastError();
}

}  // namespace hdet
