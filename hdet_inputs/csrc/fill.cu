// CUDA side of the seeded input generator: fills device buffers with exactly the values
// hdet_inputs/generator.py produces on the CPU (integer arithmetic plus one IEEE fp32
// multiply; bf16 by round-to-nearest-even on the bit pattern).  It holds nothing of the
// HDET method; it exists so that full-size workloads can be generated on the device.
#include <cuda_runtime.h>

#include <cstdint>

namespace {

__device__ __forceinline__ uint64_t mix64(uint64_t x) {
  x = (x ^ (x >> 30)) * 0xBF58476D1CE4E5B9ull;
  x = (x ^ (x >> 27)) * 0x94D049BB133111EBull;
  return x ^ (x >> 31);
}

__device__ __forceinline__ float value_at(uint64_t key, uint64_t index, float scale) {
  const uint64_t u = mix64(key + index * 0x9E3779B97F4A7C15ull);
  const int z = (int)((u & 0xFFFF) + ((u >> 16) & 0xFFFF) + ((u >> 32) & 0xFFFF) + (u >> 48)) - 131070;
  return __fmul_rn((float)z, scale);
}

__device__ __forceinline__ unsigned short to_bf16_bits(float x) {
  const unsigned b = __float_as_uint(x);
  return (unsigned short)((b + 0x7FFFu + ((b >> 16) & 1u)) >> 16);
}

template <bool kBf16>
__global__ void fill_kernel(void* out, long long n, uint64_t key, uint64_t start, float scale) {
  const long long stride = (long long)gridDim.x * blockDim.x;
  for (long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x; i < n; i += stride) {
    const float v = value_at(key, start + (uint64_t)i, scale);
    if (kBf16) static_cast<unsigned short*>(out)[i] = to_bf16_bits(v);
    else static_cast<float*>(out)[i] = v;
  }
}

}  // namespace

// Fills out[0 .. n-1] (device memory) with the generator's values for indices start .. start+n-1.
// dtype: 0 = fp32, 1 = bf16.  Returns the cudaError_t of the launch.
extern "C" __attribute__((visibility("default")))
int hdet_inputs_fill(void* out, long long n, unsigned long long key, unsigned long long start, float scale,
                     int dtype, void* stream) {
  if (n <= 0) return 0;
  const int threads = 256;
  long long blocks = (n + threads - 1) / threads;
  if (blocks > 148 * 16) blocks = 148 * 16;
  if (dtype == 1)
    fill_kernel<true><<<(int)blocks, threads, 0, (cudaStream_t)stream>>>(out, n, key, start, scale);
  else
    fill_kernel<false><<<(int)blocks, threads, 0, (cudaStream_t)stream>>>(out, n, key, start, scale);
  return (int)cudaGetLastError();
}
