// hdet_converge_static: the replica mean (the arithmetic of converge_kernel) for callers that
// must not allocate device memory.  Its work tables live in one file-scope device array instead of
// buffers obtained from cudaMalloc.  See include/hdet.h for the contract.
#include <cstdio>
#include <mutex>
#include <vector>

#include "hdet_internal.h"
#include "hdet_kernels.cuh"

namespace {

using hdet::kThreads;
using hdet::kTileElems;
using hdet::TensorDesc;
using hdet::Tile;

constexpr int kMaxTensors = HDET_STATIC_MAX_TENSORS;
constexpr int kMaxTiles = HDET_STATIC_MAX_TILES;

// Layout of the scratch array: [status word, padded to 256 B][tensor descriptors][tiles].
constexpr size_t kStatusBytes = 256;
constexpr size_t kDescBytes = sizeof(TensorDesc) * kMaxTensors;
constexpr size_t kTileBytes = sizeof(Tile) * kMaxTiles;
constexpr size_t kScratchBytes = kStatusBytes + kDescBytes + kTileBytes;   // about 0.6 MB per GPU

// Every GPU that loads the library holds this array until the process exits.  In host code the
// name `g_scratch` is only a handle for the runtime, not a device address: the address a kernel
// can use comes from cudaGetSymbolAddress (see scratch_for_device below).
static __device__ __align__(256) unsigned char g_scratch[kScratchBytes];

__device__ __forceinline__ bool not_finite(float x) { return !(fabsf(x) <= 3.402823466e38f); }

__global__ void __launch_bounds__(kThreads, 4)
converge_static_kernel(const TensorDesc* __restrict__ tensors, const Tile* __restrict__ tiles, int n_tiles, int n,
                       double inv_n) {
  bool bad = false;
  for (int t = blockIdx.x; t < n_tiles; t += gridDim.x) {
    const Tile tile = tiles[t];
    const TensorDesc td = tensors[tile.tensor];
    const long long off = (long long)tile.tile * kTileElems;
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
      bad |= not_finite(mean.x) || not_finite(mean.y) || not_finite(mean.z) || not_finite(mean.w);
      for (int r = 0; r < n; ++r) __stcs(reinterpret_cast<float4*>(P + r * td.param_stride + 4 * j), mean);
    }
    for (int e = 4 * nvec + threadIdx.x; e < len; e += kThreads) {
      double sum = 0.0;
      for (int r = 0; r < n; ++r) sum += (double)__ldcs(P + r * td.param_stride + e);
      const float mean = (float)(sum * inv_n);
      bad |= not_finite(mean);
      for (int r = 0; r < n; ++r) __stcs(P + r * td.param_stride + e, mean);
    }
  }
  // Device code may name the array directly: word 0 is the status word (bit 0 = non-finite mean).
  if (bad) atomicOr(reinterpret_cast<unsigned*>(g_scratch), 1u);
}

struct DeviceSetup {
  bool ready = false;
  unsigned char* scratch = nullptr;   // device address of g_scratch on this device
  int grid_cap = 0;                   // SM count x resident CTAs per SM
};

constexpr int kMaxDevices = 64;
DeviceSetup g_setup[kMaxDevices];
std::mutex g_setup_mutex;

// Once per device, with that device current: resolve the device address of the scratch array.
cudaError_t scratch_for_device(int device, DeviceSetup** out) {
  std::lock_guard<std::mutex> lock(g_setup_mutex);
  DeviceSetup& s = g_setup[device];
  if (!s.ready) {
    void* ptr = nullptr;
    cudaError_t e = cudaGetSymbolAddress(&ptr, g_scratch);
    if (e != cudaSuccess) return e;
    int sms = 0, occ = 0;
    e = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, device);
    if (e != cudaSuccess) return e;
    e = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&occ, converge_static_kernel, kThreads, 0);
    if (e != cudaSuccess) return e;
    s.scratch = static_cast<unsigned char*>(ptr);
    s.grid_cap = sms * (occ < 1 ? 1 : occ);
    s.ready = true;
  }
  *out = &s;
  return cudaSuccess;
}

int fail(int code, const char* msg) {
  hdet::set_handleless_error(msg);
  return code;
}

}  // namespace

extern "C" HDET_API int hdet_converge_static(const hdet_tensor* tensors, int64_t n_tensors, int32_t n_replicas,
                                             int32_t device, void* stream) {
  if (n_tensors < 0 || (n_tensors > 0 && !tensors))
    return fail(HDET_ERR_INVALID_ARG, "hdet_converge_static: tensors is NULL or n_tensors < 0");
  if (n_replicas < 1 || n_replicas > HDET_MAX_REPLICAS)
    return fail(HDET_ERR_INVALID_ARG, "hdet_converge_static: n_replicas must be in 1..32");
  if (device < 0 || device >= kMaxDevices)
    return fail(HDET_ERR_INVALID_ARG, "hdet_converge_static: device ordinal out of range");
  if (n_tensors > kMaxTensors) {
    char msg[160];
    snprintf(msg, sizeof msg, "hdet_converge_static: %lld tensors exceed the static limit of %d (use hdet_converge)",
             (long long)n_tensors, kMaxTensors);
    return fail(HDET_ERR_UNSUPPORTED, msg);
  }
  if (n_tensors == 0) return HDET_OK;

  std::vector<TensorDesc> descs(n_tensors);
  std::vector<Tile> tiles;
  int64_t total_tiles = 0;
  for (int64_t k = 0; k < n_tensors; ++k) {
    const hdet_tensor& t = tensors[k];
    if (!t.param) return fail(HDET_ERR_INVALID_ARG, "hdet_converge_static: a param pointer is NULL");
    if (t.numel <= 0) return fail(HDET_ERR_INVALID_ARG, "hdet_converge_static: numel must be > 0");
    if (t.param_stride < 0 || (n_replicas > 1 && t.param_stride < t.numel))
      return fail(HDET_ERR_INVALID_ARG, "hdet_converge_static: param_stride is smaller than numel");
    if (reinterpret_cast<uintptr_t>(t.param) % 4 != 0)
      return fail(HDET_ERR_ALIGN, "hdet_converge_static: param is not 4-byte aligned");
    total_tiles += (t.numel + kTileElems - 1) / kTileElems;
    if (total_tiles > kMaxTiles) {
      char msg[220];
      snprintf(msg, sizeof msg,
               "hdet_converge_static: the list needs more than %d tiles of %d elements (static limit, "
               "134,217,728 elements per replica at most); use hdet_converge", kMaxTiles, kTileElems);
      return fail(HDET_ERR_UNSUPPORTED, msg);
    }
    TensorDesc d{};
    d.param = static_cast<float*>(t.param);
    d.numel = t.numel;
    d.param_stride = t.param_stride;
    d.vec = (reinterpret_cast<uintptr_t>(t.param) % 16 == 0 && t.param_stride % 4 == 0) ? 1 : 0;
    descs[k] = d;
  }
  tiles.reserve(total_tiles);
  for (int64_t k = 0; k < n_tensors; ++k)
    for (int64_t j = 0, nt = (tensors[k].numel + kTileElems - 1) / kTileElems; j < nt; ++j)
      tiles.push_back(Tile{(int)k, (int)j});

  int prev = -1;
  cudaError_t e = cudaGetDevice(&prev);
  if (e == cudaSuccess && prev != device) e = cudaSetDevice(device);
  DeviceSetup* setup = nullptr;
  if (e == cudaSuccess) e = scratch_for_device(device, &setup);
  if (e == cudaSuccess) {
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    unsigned char* base = setup->scratch;
    TensorDesc* d_desc = reinterpret_cast<TensorDesc*>(base + kStatusBytes);
    Tile* d_tiles = reinterpret_cast<Tile*>(base + kStatusBytes + kDescBytes);
    // The array keeps the previous call's contents: clear the status word, overwrite the tables in use.
    e = cudaMemsetAsync(base, 0, kStatusBytes, st);
    if (e == cudaSuccess)
      e = cudaMemcpyAsync(d_desc, descs.data(), descs.size() * sizeof(TensorDesc), cudaMemcpyHostToDevice, st);
    if (e == cudaSuccess)
      e = cudaMemcpyAsync(d_tiles, tiles.data(), tiles.size() * sizeof(Tile), cudaMemcpyHostToDevice, st);
    if (e == cudaSuccess) {
      const int n_tiles = (int)tiles.size();
      const int grid = n_tiles < setup->grid_cap ? n_tiles : setup->grid_cap;
      converge_static_kernel<<<grid, kThreads, 0, st>>>(d_desc, d_tiles, n_tiles, n_replicas, 1.0 / (double)n_replicas);
      e = cudaGetLastError();
    }
  }
  if (prev >= 0 && prev != device) cudaSetDevice(prev);
  if (e != cudaSuccess) {
    char msg[200];
    snprintf(msg, sizeof msg, "hdet_converge_static: %s", cudaGetErrorString(e));
    return fail(HDET_ERR_CUDA, msg);
  }
  return HDET_OK;
}
