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

// Layout of the scratch array: [tensor descriptors][tiles].  Nothing in it has to start at zero: a call
// overwrites every entry it is going to read.
constexpr size_t kDescBytes = sizeof(TensorDesc) * kMaxTensors;
constexpr size_t kTileBytes = sizeof(Tile) * kMaxTiles;
constexpr size_t kScratchBytes = kDescBytes + kTileBytes;   // about 0.6 MB per GPU

// Every GPU that loads the library holds this array until the process exits.  In host code the
// name `g_scratch` is only a handle for the runtime, not a device address: the address a kernel
// can use comes from cudaGetSymbolAddress (see scratch_for_device below).
static __device__ __align__(256) unsigned char g_scratch[kScratchBytes];

// The arithmetic is hdet::converge_tile, the same device function hdet_converge runs.
__global__ void __launch_bounds__(kThreads, 4)
converge_static_kernel(const TensorDesc* __restrict__ tensors, const Tile* __restrict__ tiles, int n_tiles, int n,
                       double inv_n) {
  for (int t = blockIdx.x; t < n_tiles; t += gridDim.x) {
    const Tile tile = tiles[t];
    const TensorDesc td = tensors[tile.tensor];
    hdet::converge_tile(td, tile.tile, n, inv_n);
  }
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
  hdet::TraceRange trace("hdet_converge_static");
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
    d.vec = (reinterpret_cast<uintptr_t>(t.param) % 16 == 0 && t.param_stride % 4 == 0) ? hdet::kVecLoads : 0;
    descs[k] = d;
  }
  tiles.reserve(total_tiles);
  for (int64_t k = 0; k < n_tensors; ++k)
    for (int64_t j = 0, nt = (tensors[k].numel + kTileElems - 1) / kTileElems; j < nt; ++j)
      tiles.push_back(Tile{(int)k, (int)j});

  int prev = -1;
  cudaError_t e = cudaGetDevice(&prev);
  if (e == cudaSuccess && prev != device) e = cudaSetDevice(device);
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  // The tables are copied from host buffers that die with this call, so the call cannot be recorded
  // into a stream capture: a replay would read freed host memory.  Refuse instead.
  bool capturing = false;
  if (e == cudaSuccess) {
    cudaStreamCaptureStatus cap = cudaStreamCaptureStatusNone;
    e = cudaStreamIsCapturing(st, &cap);
    capturing = e == cudaSuccess && cap != cudaStreamCaptureStatusNone;
  }
  DeviceSetup* setup = nullptr;
  if (e == cudaSuccess && !capturing) e = scratch_for_device(device, &setup);
  if (e == cudaSuccess && !capturing) {
    unsigned char* base = setup->scratch;
    TensorDesc* d_desc = reinterpret_cast<TensorDesc*>(base);
    Tile* d_tiles = reinterpret_cast<Tile*>(base + kDescBytes);
    // The array keeps the previous call's contents: overwrite the tables this call uses, in stream order.
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
  if (capturing)
    return fail(HDET_ERR_UNSUPPORTED, "hdet_converge_static: the stream is being captured; this call copies its tables "
                                      "from temporary host memory and refuses to be recorded");
  if (e != cudaSuccess) {
    char msg[200];
    snprintf(msg, sizeof msg, "hdet_converge_static: %s", cudaGetErrorString(e));
    return fail(HDET_ERR_CUDA, msg);
  }
  return HDET_OK;
}
