// Fan-out update and converge kernels for sm_100a.
//
// Work assignment: one CTA owns one tile (kTileElems consecutive elements of one tensor)
// and streams ALL N replicas of that tile, so the replica mean of Eq. 3 is a per-thread
// register accumulation: no inter-CTA dependence, no atomics on data.
// The path is HBM-bound (about 1.5 flop per byte).  Two ways of moving a tile:
//   - AdamW with per-replica moments, full 16-byte-aligned tiles: bulk asynchronous copies into a ring of
//     shared-memory stages, issued by a producer warp and tracked by shared-memory barriers (tile_bulk);
//     every wait on a barrier is bounded;
//   - everything else (SGD, shared moments, ragged or unaligned tiles): 128-bit warp-contiguous accesses,
//     read-once / write-once with streaming cache hints, replica r+1 loaded while replica r is being
//     computed and stored (explicit two-stage register pipeline); scalar accesses where alignment demands.
#include <cuda_bf16.h>

#include <type_traits>

#include "hdet_bulk.cuh"
#include "hdet_kernels.cuh"

namespace hdet {
namespace {

constexpr int kOptSgd = 0, kOptAdamW = 1, kOptSgdMomentum = 2;

struct AdamConsts {
  float one_minus_beta1, one_minus_beta2, rsqrt_bc2, eps, momentum;
};

// Adam with decoupled weight decay on one element (Section 4.1 names Adam; weight decay is a
// spreadable scalar per Remark 1):
//   theta *= 1 - lr*wd ; m = b1 m + (1-b1) g ; v = b2 v + (1-b2) g^2 ;
//   theta -= lr/(1-b1^t) * m / (sqrt(v)/sqrt(1-b2^t) + eps)
// The moving averages are evaluated as x + (1-b)(new - x) and the decay as theta - (lr*wd) theta:
// the fp32 images of b2 = 0.999 and of 1 - lr*wd are off by ~1e-8 relative, which the recurrences
// would amplify to ~1e-5 over a thousand updates; the small factors 1-b and lr*wd carry no such bias.
__device__ __forceinline__ void adam_element(float& th, float& m, float& v, float g, float lr_wd, float step,
                                             const AdamConsts& c) {
  m = fmaf(c.one_minus_beta1, g - m, m);
  v = fmaf(c.one_minus_beta2, fmaf(g, g, -v), v);
  const float denom = fmaf(sqrtf(v), c.rsqrt_bc2, c.eps);
  th = fmaf(-step, m / denom, fmaf(-lr_wd, th, th));
}

// Eq. 2: theta <- theta - eta_r * g.  With a weight decay the gradient is first extended by wd * theta
// (the coupled form of SGD; wd = 0 leaves g untouched bit for bit).
__device__ __forceinline__ void sgd_element(float& th, float g, float wd, float step) {
  th = fmaf(-step, fmaf(wd, th, g), th);
}

// SGD with a momentum buffer (not part of Eq. 2; the usual definition): g' = g + wd theta;
// buf = mu buf + g'; theta <- theta - eta_r buf.
__device__ __forceinline__ void sgd_momentum_element(float& th, float& buf, float g, float wd, float step, float mu) {
  buf = fmaf(mu, buf, fmaf(wd, th, g));
  th = fmaf(-step, buf, th);
}

__device__ __forceinline__ bool not_finite(float x) { return !(fabsf(x) <= 3.402823466e38f); }

// ---- gradient access: fp32 (float4 per 4 elements) or bf16 (uint2 per 4 elements) ----------
template <typename GradT> struct GradRaw;
template <> struct GradRaw<float> { using type = float4; };
template <> struct GradRaw<__nv_bfloat16> { using type = uint2; };

__device__ __forceinline__ float4 load_raw(const float* p) { return __ldcs(reinterpret_cast<const float4*>(p)); }
__device__ __forceinline__ uint2 load_raw(const __nv_bfloat16* p) { return __ldcs(reinterpret_cast<const uint2*>(p)); }
__device__ __forceinline__ void unpack(const float4& r, float (&g)[4]) { g[0] = r.x; g[1] = r.y; g[2] = r.z; g[3] = r.w; }
__device__ __forceinline__ void unpack(const uint2& r, float (&g)[4]) {
  g[0] = __uint_as_float(r.x << 16);
  g[1] = __uint_as_float(r.x & 0xffff0000u);
  g[2] = __uint_as_float(r.y << 16);
  g[3] = __uint_as_float(r.y & 0xffff0000u);
}
__device__ __forceinline__ float load_scalar(const float* p) { return __ldcs(p); }
__device__ __forceinline__ float load_scalar(const __nv_bfloat16* p) {
  return __uint_as_float(static_cast<unsigned>(__ldcs(reinterpret_cast<const unsigned short*>(p))) << 16);
}

// ---- scalar path: elements [begin, end) of one tensor, any alignment -----------------------
template <typename GradT, int kOpt, bool kConv, bool kMean>
__device__ void range_scalar(const TensorDesc& td, long long begin, long long end, const StepScalars& s,
                             const AdamConsts& c, bool& bad) {
  constexpr bool kAdam = kOpt == kOptAdamW, kMom = kOpt == kOptSgdMomentum;
  const int n = s.n_replicas;
  const GradT* grad = static_cast<const GradT*>(td.grad);
  for (long long e = begin + threadIdx.x; e < end; e += kThreads) {
    double sum = 0.0;
    float gbar = 0.f;
    if (kMean) {
      double acc = 0.0;
      for (int r = 0; r < n; ++r) acc += (double)load_scalar(grad + r * td.grad_stride + e);
      gbar = (float)(acc * s.inv_n);
    }
    for (int r = 0; r < n; ++r) {
      float th = __ldcs(td.param + r * td.param_stride + e);
      const float g = kMean ? gbar : load_scalar(grad + r * td.grad_stride + e);
      if (kAdam) {
        float m = __ldcs(td.exp_avg + r * td.state_stride + e);
        float v = __ldcs(td.exp_avg_sq + r * td.state_stride + e);
        adam_element(th, m, v, g, s.lr_wd[td.group][r], s.step[td.group][r], c);
        __stcs(td.exp_avg + r * td.state_stride + e, m);
        __stcs(td.exp_avg_sq + r * td.state_stride + e, v);
      } else if (kMom) {
        float buf = __ldcs(td.exp_avg + r * td.state_stride + e);
        sgd_momentum_element(th, buf, g, s.lr_wd[td.group][r], s.step[td.group][r], c.momentum);
        __stcs(td.exp_avg + r * td.state_stride + e, buf);
      } else {
        sgd_element(th, g, s.lr_wd[td.group][r], s.step[td.group][r]);
      }
      bad |= not_finite(th);
      if (kConv) sum += (double)th;
      else __stcs(td.param + r * td.param_stride + e, th);
    }
    if (kConv) {
      if (td.partial) {
        td.partial[e] = (float)sum;       // replica axis sharded over GPUs: hand out the local sum instead
      } else {
        const float mean = (float)(sum * s.inv_n);
        for (int r = 0; r < n; ++r) __stcs(td.param + r * td.param_stride + e, mean);
        if (td.param_bf16) td.param_bf16[e] = bf16_bits(mean);
      }
    }
  }
}

// ---- vector path ---------------------------------------------------------------------------
// gbar[k][q] = (1/N) sum_r g_r for the thread's vectors of one tile.  The sum is taken in fp64 (exact for
// bf16 gradients, correctly rounded for fp32 ones): where the g_r cancel, Adam's m / (sqrt(v) + eps) is
// sensitive to the low bits of the mean.
template <typename GradT, int kV>
__device__ __forceinline__ void mean_gradient(const GradT* Gp, long long gs, const int (&idx)[kV],
                                              const bool (&ok)[kV], int n, double inv_n,
                                              float (&gbar)[kV][4]) {
  double acc[kV][4];
#pragma unroll
  for (int k = 0; k < kV; ++k)
#pragma unroll
    for (int q = 0; q < 4; ++q) acc[k][q] = 0.0;
#pragma unroll 4
  for (int r = 0; r < n; ++r) {
#pragma unroll
    for (int k = 0; k < kV; ++k) {
      if (!ok[k]) continue;
      float g[4];
      unpack(load_raw(Gp + r * gs + idx[k]), g);
#pragma unroll
      for (int q = 0; q < 4; ++q) acc[k][q] += (double)g[q];
    }
  }
#pragma unroll
  for (int k = 0; k < kV; ++k)
#pragma unroll
    for (int q = 0; q < 4; ++q) gbar[k][q] = (float)(acc[k][q] * inv_n);
}

template <typename GradT, int kOpt, int kV>
struct ReplicaRegs {
  float4 th[kV];
  float4 m[kOpt != kOptSgd ? kV : 1];        // Adam first moment, or the SGD momentum buffer
  float4 v[kOpt == kOptAdamW ? kV : 1];
  typename GradRaw<GradT>::type g[kV];
};

// Processes float4 vectors j = (first + k) * kThreads + threadIdx.x, k = 0..kV-1, j < nvec, of the tile that
// starts at element `off` of the tensor.  kFull: every such j is below nvec.
template <typename GradT, int kOpt, bool kConv, bool kMean, bool kFull, int kV>
__device__ __forceinline__ void tile_vector_pass(const TensorDesc& td, long long off, int first, int nvec,
                                                 const StepScalars& s, const AdamConsts& c, bool& bad) {
  constexpr bool kAdam = kOpt == kOptAdamW, kMom = kOpt == kOptSgdMomentum;
  using Regs = ReplicaRegs<GradT, kOpt, kV>;
  const int n = s.n_replicas;
  const int grp = td.group;
  float* const P = td.param + off;
  float* const M = (kAdam || kMom) ? td.exp_avg + off : nullptr;
  float* const V = kAdam ? td.exp_avg_sq + off : nullptr;
  const GradT* const Gp = static_cast<const GradT*>(td.grad) + off;
  const long long ps = td.param_stride, gs = td.grad_stride, ss = td.state_stride;

  int idx[kV];
  bool ok[kV];
#pragma unroll
  for (int k = 0; k < kV; ++k) {
    const int j = (first + k) * kThreads + threadIdx.x;
    idx[k] = j * 4;
    ok[k] = kFull || j < nvec;
  }

  auto load = [&](Regs& b, int r) {
#pragma unroll
    for (int k = 0; k < kV; ++k) {
      if (ok[k]) {
        b.th[k] = __ldcs(reinterpret_cast<const float4*>(P + r * ps + idx[k]));
        if (kAdam || kMom) b.m[k] = __ldcs(reinterpret_cast<const float4*>(M + r * ss + idx[k]));
        if (kAdam) b.v[k] = __ldcs(reinterpret_cast<const float4*>(V + r * ss + idx[k]));
        if (!kMean) b.g[k] = load_raw(Gp + r * gs + idx[k]);
      } else {
        b.th[k] = make_float4(0.f, 0.f, 0.f, 0.f);
        if (kAdam || kMom) b.m[k] = b.th[k];
        if (kAdam) b.v[k] = b.th[k];
        b.g[k] = typename GradRaw<GradT>::type{};
      }
    }
  };

  // Replica 0 is requested first; then the gradient replica-mean (the all-reduced gradient of
  // Algorithm 1) is formed once per tile while those loads are in flight.
  Regs a, b;
  load(a, 0);
  float gbar[kV][4];
  if constexpr (kMean) mean_gradient<GradT, kV>(Gp, gs, idx, ok, n, s.inv_n, gbar);

  double sum[kConv ? kV : 1][4];
  if (kConv) {
#pragma unroll
    for (int k = 0; k < kV; ++k)
#pragma unroll
      for (int q = 0; q < 4; ++q) sum[k][q] = 0.0;
  }

  auto update_store = [&](Regs& b, int r) {
    const float lr_wd = s.lr_wd[grp][r];
    const float step = s.step[grp][r];
#pragma unroll
    for (int k = 0; k < kV; ++k) {
      float g[4];
      if constexpr (kMean) {
#pragma unroll
        for (int q = 0; q < 4; ++q) g[q] = gbar[k][q];
      } else {
        unpack(b.g[k], g);
      }
      float th[4] = {b.th[k].x, b.th[k].y, b.th[k].z, b.th[k].w};
      if (kAdam) {
        float m[4] = {b.m[k].x, b.m[k].y, b.m[k].z, b.m[k].w};
        float v[4] = {b.v[k].x, b.v[k].y, b.v[k].z, b.v[k].w};
#pragma unroll
        for (int q = 0; q < 4; ++q) adam_element(th[q], m[q], v[q], g[q], lr_wd, step, c);
        if (ok[k]) {
          __stcs(reinterpret_cast<float4*>(M + r * ss + idx[k]), make_float4(m[0], m[1], m[2], m[3]));
          __stcs(reinterpret_cast<float4*>(V + r * ss + idx[k]), make_float4(v[0], v[1], v[2], v[3]));
        }
      } else if (kMom) {
        float buf[4] = {b.m[k].x, b.m[k].y, b.m[k].z, b.m[k].w};
#pragma unroll
        for (int q = 0; q < 4; ++q) sgd_momentum_element(th[q], buf[q], g[q], lr_wd, step, c.momentum);
        if (ok[k]) __stcs(reinterpret_cast<float4*>(M + r * ss + idx[k]), make_float4(buf[0], buf[1], buf[2], buf[3]));
      } else {
#pragma unroll
        for (int q = 0; q < 4; ++q) sgd_element(th[q], g[q], lr_wd, step);
      }
      if (ok[k]) {   // idle lanes of a partial tile carry zeros, which eps = 0 turns into 0/0
#pragma unroll
        for (int q = 0; q < 4; ++q) bad |= not_finite(th[q]);
      }
      if (kConv) {
#pragma unroll
        for (int q = 0; q < 4; ++q) sum[k][q] += (double)th[q];
      } else if (ok[k]) {
        __stcs(reinterpret_cast<float4*>(P + r * ps + idx[k]), make_float4(th[0], th[1], th[2], th[3]));
      }
    }
  };

  // Two-stage register pipeline over the replica axis.
  int r = 0;
  for (; r + 1 < n; r += 2) {
    load(b, r + 1);
    update_store(a, r);
    if (r + 2 < n) load(a, r + 2);
    update_store(b, r + 1);
  }
  if (r < n) update_store(a, r);

  if (kConv) {
    // Eq. 3: the mean of the updated replicas goes to every replica.
#pragma unroll
    for (int k = 0; k < kV; ++k) {
      if (!ok[k]) continue;
      if (td.partial) {   // replica axis sharded over GPUs: the local sum goes to the staging buffer
        *reinterpret_cast<float4*>(td.partial + off + idx[k]) =
            make_float4((float)sum[k][0], (float)sum[k][1], (float)sum[k][2], (float)sum[k][3]);
        continue;
      }
      const float4 mean = make_float4((float)(sum[k][0] * s.inv_n), (float)(sum[k][1] * s.inv_n),
                                      (float)(sum[k][2] * s.inv_n), (float)(sum[k][3] * s.inv_n));
      for (int rr = 0; rr < n; ++rr) __stcs(reinterpret_cast<float4*>(P + rr * ps + idx[k]), mean);
      if (td.param_bf16) __stcs(reinterpret_cast<uint2*>(td.param_bf16 + off + idx[k]), bf16_bits4(mean));
    }
  }
}

// The whole tile in passes of kV vectors per thread.  Two vectors per pass keep more loads in flight; the
// kernels that also hold the bulk-copy path have fewer registers per thread and take one vector per pass.
template <typename GradT, int kOpt, bool kConv, bool kMean, bool kFull, int kV>
__device__ __forceinline__ void tile_vector(const TensorDesc& td, long long off, int nvec, const StepScalars& s,
                                            const AdamConsts& c, bool& bad) {
  static_assert(kTileVecs % kV == 0, "passes cover the tile");
#pragma unroll 1
  for (int first = 0; first < kTileVecs; first += kV) {
    if (!kFull && first * kThreads >= nvec) break;
    tile_vector_pass<GradT, kOpt, kConv, kMean, kFull, kV>(td, off, first, nvec, s, c, bad);
  }
}

// ---- bulk-copy path: a full tile of an AdamW tensor whose arrays are all 16-byte aligned ----------------
// One tile per CTA, CTAs dispatched in tile order: CTAs that run at the same time then stream neighbouring
// addresses, which the DRAM likes (giving a CTA several consecutive tiles measured 1.5 - 3 % slower).
// The CTA has one extra warp.  Its lane 0 (the producer) moves every byte of the tile with bulk copies:
// replica r's theta, m, v and gradient tiles land in one of kStages shared-memory stages; the 256
// consumer threads wait for the stage, update it in place and signal; the producer then writes m and v
// (and theta, when no mean is formed) back from the stage with bulk stores and refills the stage with
// replica r + kStages.  For Eq. 3 the consumers keep the fp64 sums in registers, put the mean into a
// shared tile once, and the producer sends that one tile to all N replicas.  Compared with the register
// pipeline below this takes the address arithmetic and the load/store instructions of 26 bytes per
// element off the consumer warps and keeps more bytes in flight per SM; the arithmetic per element, and
// so every result bit, is the same.
// With the gradient replica-mean the ring first carries the gradient tiles alone, several replicas per
// stage (the consumers form g_bar in fp64, r = 0..N-1), then the N (theta, m, v) stages.
constexpr int kProducerThreads = 32;
constexpr int kStages = 3;
constexpr int kMaxDevices = 64;

template <typename GradT>
struct BulkLayout {
  static constexpr uint32_t kF32Bytes = kTileElems * 4;
  static constexpr uint32_t kGradBytes = kTileElems * sizeof(GradT);
  static constexpr uint32_t kStageBytes = 3 * kF32Bytes + kGradBytes;     // theta | m | v | gradient
  static constexpr uint32_t kMeanOff = kStages * kStageBytes;             // one fp32 tile for the mean
  static constexpr uint32_t kBf16Off = kMeanOff + kF32Bytes;              // one bf16 tile: the mean's bf16 copy
  static constexpr uint32_t kBarrierOff = kBf16Off + kTileElems * 2;      // full[kStages], done[kStages], mean written
  static constexpr uint32_t kBytes = kBarrierOff + 8 * (2 * kStages + 1);
};

__device__ __forceinline__ void read_grad(const unsigned char* slot, int j, float (&g)[4], float) {
  unpack(reinterpret_cast<const float4*>(slot)[j], g);
}
__device__ __forceinline__ void read_grad(const unsigned char* slot, int j, float (&g)[4], __nv_bfloat16) {
  unpack(reinterpret_cast<const uint2*>(slot)[j], g);
}

// Called once per kernel by thread 0, before the CTA-wide barrier that follows the scalar staging.
template <typename GradT>
__device__ __forceinline__ void bulk_init_barriers(unsigned char* smem) {
  const uint32_t bars = bulk::smem_addr(smem + BulkLayout<GradT>::kBarrierOff);
  for (int i = 0; i < kStages; ++i) {
    bulk::barrier_init(bars + 8 * i, 1);                         // full: the producer's announcement
    bulk::barrier_init(bars + 8 * (kStages + i), kThreads);      // done: every consumer thread
  }
  bulk::barrier_init(bars + 8 * 2 * kStages, kThreads);          // mean tile written
  bulk::barrier_init_fence();
}

template <typename GradT, bool kConv, bool kMean>
__device__ __forceinline__ void tile_bulk(const TensorDesc& td, long long off, const StepScalars& s,
                                          const AdamConsts& c, bool& bad, unsigned char* smem, unsigned* status) {
  using L = BulkLayout<GradT>;
  const int n = s.n_replicas;
  // With the gradient mean the ring first carries the gradient tiles alone, as many replicas per stage as fit
  // (7 for bf16, 4 for fp32), then the N replicas.
  constexpr int kGradPerItem = L::kStageBytes / L::kGradBytes;
  const int n_grad_items = kMean ? (n + kGradPerItem - 1) / kGradPerItem : 0;
  const int n_items = n_grad_items + n;
  const uint32_t base = bulk::smem_addr(smem);
  const uint32_t full = base + L::kBarrierOff, done = full + 8 * kStages, mean_done = done + 8 * kStages;
  float* const P = td.param + off;
  float* const M = td.exp_avg + off;
  float* const V = td.exp_avg_sq + off;
  const GradT* const G = static_cast<const GradT*>(td.grad) + off;
  const long long ps = td.param_stride, gs = td.grad_stride, ss = td.state_stride;

  if (threadIdx.x >= kThreads) {
    // ---- producer: one lane issues every copy of the tile ------------------------------------------------
    if (threadIdx.x != kThreads) return;
    auto request = [&](int i) {
      const int st = i % kStages;
      const uint32_t slot = base + st * L::kStageBytes, bar = full + 8 * st;
      if (i < n_grad_items) {
        const int r0 = i * kGradPerItem, count = n - r0 < kGradPerItem ? n - r0 : kGradPerItem;
        bulk::barrier_expect(bar, count * L::kGradBytes);
        for (int q = 0; q < count; ++q) bulk::load(slot + q * L::kGradBytes, G + (r0 + q) * gs, L::kGradBytes, bar);
        return;
      }
      const int r = i - n_grad_items;
      bulk::barrier_expect(bar, kMean ? 3 * L::kF32Bytes : L::kStageBytes);
      bulk::load(slot, P + r * ps, L::kF32Bytes, bar);
      bulk::load(slot + L::kF32Bytes, M + r * ss, L::kF32Bytes, bar);
      bulk::load(slot + 2 * L::kF32Bytes, V + r * ss, L::kF32Bytes, bar);
      if (!kMean) bulk::load(slot + 3 * L::kF32Bytes, G + r * gs, L::kGradBytes, bar);
    };
    for (int i = 0; i < kStages && i < n_items; ++i) request(i);
    bool alive = true;
    for (int i = 0; i < n_items; ++i) {
      const int st = i % kStages;
      if (!bulk::barrier_wait(done + 8 * st, (i / kStages) & 1)) { alive = false; break; }
      if (i >= n_grad_items) {
        const int r = i - n_grad_items;
        const uint32_t slot = base + st * L::kStageBytes;
        if (!kConv) bulk::store(P + r * ps, slot, L::kF32Bytes);
        bulk::store(M + r * ss, slot + L::kF32Bytes, L::kF32Bytes);
        bulk::store(V + r * ss, slot + 2 * L::kF32Bytes, L::kF32Bytes);
        bulk::commit();
      }
      if (i + kStages < n_items) {
        bulk::wait_stores_read();          // the stage is refilled only after its stores have read it
        request(i + kStages);
      }
    }
    if (kConv && alive) {
      if (bulk::barrier_wait(mean_done, 0)) {
        const uint32_t mean_tile = base + L::kMeanOff;
        if (td.partial) {                  // replica axis sharded over GPUs: the local sums go to the staging buffer
          bulk::store(td.partial + off, mean_tile, L::kF32Bytes);
        } else {                           // Eq. 3: one shared tile goes to every replica
          for (int r = 0; r < n; ++r) bulk::store(P + r * ps, mean_tile, L::kF32Bytes);
          if (td.param_bf16) bulk::store(td.param_bf16 + off, base + L::kBf16Off, kTileElems * 2);
        }
        bulk::commit();
      } else {
        alive = false;
      }
    }
    bulk::wait_stores_read();              // shared memory must outlive the stores that read it
    if (!alive) {
      atomicOr(status, 2u);
      // Loads already requested may still be writing this CTA's shared memory: give each a bounded wait.
      for (int st = 0; st < kStages; ++st) { bulk::barrier_wait(full + 8 * st, 0); bulk::barrier_wait(full + 8 * st, 1); }
    }
    return;
  }

  // ---- consumers: thread i owns vectors i and i + 256 of the tile, as in the register path ---------------
  const int grp = td.group;
  const bool to_partial = td.partial != nullptr;
  const bool with_bf16 = !to_partial && td.param_bf16 != nullptr;
  float gbar[kMean ? kTileVecs : 1][4];
  int i = 0;
  if constexpr (kMean) {
    double acc[kTileVecs][4];
#pragma unroll
    for (int k = 0; k < kTileVecs; ++k)
#pragma unroll
      for (int q = 0; q < 4; ++q) acc[k][q] = 0.0;
    for (; i < n_grad_items; ++i) {
      const int st = i % kStages;
      if (!bulk::barrier_wait(full + 8 * st, (i / kStages) & 1)) { atomicOr(status, 2u); return; }
      const int r0 = i * kGradPerItem, count = n - r0 < kGradPerItem ? n - r0 : kGradPerItem;
      for (int r = 0; r < count; ++r) {        // replicas in order, so the sum is the one of the register path
        const unsigned char* slot = smem + st * L::kStageBytes + r * L::kGradBytes;
#pragma unroll
        for (int k = 0; k < kTileVecs; ++k) {
          float g[4];
          read_grad(slot, k * kThreads + threadIdx.x, g, GradT{});
#pragma unroll
          for (int q = 0; q < 4; ++q) acc[k][q] += (double)g[q];
        }
      }
      bulk::barrier_arrive(done + 8 * st);
    }
#pragma unroll
    for (int k = 0; k < kTileVecs; ++k)
#pragma unroll
      for (int q = 0; q < 4; ++q) gbar[k][q] = (float)(acc[k][q] * s.inv_n);
  }

  double sum[kConv ? kTileVecs : 1][4];
  if (kConv) {
#pragma unroll
    for (int k = 0; k < kTileVecs; ++k)
#pragma unroll
      for (int q = 0; q < 4; ++q) sum[k][q] = 0.0;
  }
  for (; i < n_items; ++i) {
    const int r = i - n_grad_items;
    const int st = i % kStages;
    if (!bulk::barrier_wait(full + 8 * st, (i / kStages) & 1)) { atomicOr(status, 2u); return; }
    unsigned char* const slot = smem + st * L::kStageBytes;
    float4* const TH = reinterpret_cast<float4*>(slot);
    float4* const MM = reinterpret_cast<float4*>(slot + L::kF32Bytes);
    float4* const VV = reinterpret_cast<float4*>(slot + 2 * L::kF32Bytes);
    const float lr_wd = s.lr_wd[grp][r];
    const float step = s.step[grp][r];
#pragma unroll
    for (int k = 0; k < kTileVecs; ++k) {
      const int j = k * kThreads + threadIdx.x;
      const float4 t4 = TH[j], m4 = MM[j], v4 = VV[j];
      float g[4];
      if constexpr (kMean) {
#pragma unroll
        for (int q = 0; q < 4; ++q) g[q] = gbar[k][q];
      } else {
        read_grad(slot + 3 * L::kF32Bytes, j, g, GradT{});
      }
      float th[4] = {t4.x, t4.y, t4.z, t4.w};
      float m[4] = {m4.x, m4.y, m4.z, m4.w};
      float v[4] = {v4.x, v4.y, v4.z, v4.w};
#pragma unroll
      for (int q = 0; q < 4; ++q) {
        adam_element(th[q], m[q], v[q], g[q], lr_wd, step, c);
        bad |= not_finite(th[q]);
      }
      MM[j] = make_float4(m[0], m[1], m[2], m[3]);
      VV[j] = make_float4(v[0], v[1], v[2], v[3]);
      if (kConv) {
#pragma unroll
        for (int q = 0; q < 4; ++q) sum[k][q] += (double)th[q];
      } else {
        TH[j] = make_float4(th[0], th[1], th[2], th[3]);
      }
    }
    bulk::publish_smem_writes();
    bulk::barrier_arrive(done + 8 * st);
  }
  if (kConv) {
    float4* const mean_tile = reinterpret_cast<float4*>(smem + L::kMeanOff);
#pragma unroll
    for (int k = 0; k < kTileVecs; ++k) {
      const int j = k * kThreads + threadIdx.x;
      mean_tile[j] = to_partial
                         ? make_float4((float)sum[k][0], (float)sum[k][1], (float)sum[k][2], (float)sum[k][3])
                         : make_float4((float)(sum[k][0] * s.inv_n), (float)(sum[k][1] * s.inv_n),
                                       (float)(sum[k][2] * s.inv_n), (float)(sum[k][3] * s.inv_n));
      if (with_bf16) reinterpret_cast<uint2*>(smem + L::kBf16Off)[j] = bf16_bits4(mean_tile[j]);
    }
    bulk::publish_smem_writes();
    bulk::barrier_arrive(mean_done);
  }
}

// The launch scalars are staged in shared memory once per CTA, from the kernel parameter (host stepping)
// or from the device-resident copy (device stepping); the update loops then read them with broadcast
// shared-memory loads.  Selecting between the two sources by pointer instead costs 7 % of the kernel's
// bandwidth: the by-value parameter is then no longer read through the constant bank.
__device__ __forceinline__ void stage_scalars(StepScalars& sh, const StepScalars& s_param, const StepScalars* s_dev) {
  static_assert(HDET_MAX_GROUPS * HDET_MAX_REPLICAS == kThreads, "one (group, replica) pair per thread");
  if (threadIdx.x < kThreads) {     // a CTA of the bulk-copy kernels has one more warp than there are pairs
    const int g = threadIdx.x / HDET_MAX_REPLICAS, r = threadIdx.x % HDET_MAX_REPLICAS;
    if (s_dev) {
      sh.lr_wd[g][r] = s_dev->lr_wd[g][r];
      sh.step[g][r] = s_dev->step[g][r];
      if (threadIdx.x == 0) {
        sh.one_minus_beta1 = s_dev->one_minus_beta1; sh.one_minus_beta2 = s_dev->one_minus_beta2;
        sh.rsqrt_bc2 = s_dev->rsqrt_bc2; sh.eps = s_dev->eps; sh.inv_n = s_dev->inv_n; sh.n_replicas = s_dev->n_replicas;
        sh.momentum = s_dev->momentum;
      }
    } else {
      sh.lr_wd[g][r] = s_param.lr_wd[g][r];
      sh.step[g][r] = s_param.step[g][r];
      if (threadIdx.x == 0) {
        sh.one_minus_beta1 = s_param.one_minus_beta1; sh.one_minus_beta2 = s_param.one_minus_beta2;
        sh.rsqrt_bc2 = s_param.rsqrt_bc2; sh.eps = s_param.eps; sh.inv_n = s_param.inv_n; sh.n_replicas = s_param.n_replicas;
        sh.momentum = s_param.momentum;
      }
    }
  }
  __syncthreads();
}

// One tile through the register path: 128-bit accesses where the tensor allows them, scalar accesses for the
// rest (a tail of 1-3 elements, or a tensor that is not 16-byte aligned).
template <typename GradT, int kOpt, bool kConv, bool kMean, int kV>
__device__ __forceinline__ void tile_registers(const TensorDesc& td, long long off, int len, const StepScalars& s,
                                               const AdamConsts& c, bool& bad) {
  if (td.vec) {
    if (len == kTileElems) {
      tile_vector<GradT, kOpt, kConv, kMean, true, kV>(td, off, kThreads * kTileVecs, s, c, bad);
    } else {
      const int nvec = len >> 2;
      if (nvec) tile_vector<GradT, kOpt, kConv, kMean, false, kV>(td, off, nvec, s, c, bad);
      if (len & 3) range_scalar<GradT, kOpt, kConv, kMean>(td, off + 4ll * nvec, off + len, s, c, bad);
    }
  } else {
    range_scalar<GradT, kOpt, kConv, kMean>(td, off, off + len, s, c, bad);
  }
}

// The same as a real function call, one vector per pass: in the kernels that also hold the bulk-copy path it
// serves the few tiles that path cannot take, and must not raise the register count of the common case.
// Everything is passed and returned BY VALUE: a reference would force the caller to keep the descriptor in
// its stack frame, and then every CTA of the common case would write it to local memory first.
template <typename GradT, int kOpt, bool kConv, bool kMean>
__device__ __noinline__ bool tile_registers_outlined(TensorDesc td, long long off, int len, const StepScalars* s,
                                                     AdamConsts c) {
  bool bad = false;
  tile_registers<GradT, kOpt, kConv, kMean, 1>(td, off, len, *s, c, bad);
  return bad;
}

// AdamW tensors with per-replica moments run in a CTA of 256 consumer threads plus one producer warp and
// take the bulk-copy path for every full tile of a 16-byte-aligned tensor; all other tiles, and SGD, take
// the register path with the 256 consumer threads.
template <int kOpt>
constexpr bool kHasBulkPath = kOpt == kOptAdamW;

template <typename GradT, int kOpt, bool kConv, bool kMean>
__global__ void __launch_bounds__(kHasBulkPath<kOpt> ? kThreads + kProducerThreads : kThreads, (kOpt == kOptSgd && !kMean) ? 3 : 2)
fanout_kernel(const __grid_constant__ LaunchPlan plan, const __grid_constant__ StepScalars s_param) {
  __shared__ StepScalars s;
  if constexpr (kHasBulkPath<kOpt>) {
    // One tile per CTA (the barriers are set up for one tile).
    extern __shared__ __align__(128) unsigned char stage_smem[];   // BulkLayout<GradT>::kBytes
    __shared__ unsigned abandoned;
    const Tile tile = plan.tiles[blockIdx.x];
    if (threadIdx.x == 0) {
      bulk_init_barriers<GradT>(stage_smem);
      // Once any CTA has given up on a copy the launch is lost; the CTAs still to come leave at once, so
      // that the launch ends after one bounded wait instead of one per tile.
      abandoned = *reinterpret_cast<volatile unsigned*>(plan.status) & 2u;
    }
    TensorDesc td = plan.tensors[tile.tensor];
    td.partial = plan.partial ? plan.partial + td.partial_off : nullptr;
    stage_scalars(s, s_param, plan.scal_dev);
    if (abandoned) return;
    const AdamConsts c{s.one_minus_beta1, s.one_minus_beta2, s.rsqrt_bc2, s.eps, s.momentum};
    bool bad = false;
    const long long off = (long long)tile.tile * kTileElems;
    const long long rest = td.numel - off;
    if ((td.vec & kVecBulk) && rest >= kTileElems) {
      tile_bulk<GradT, kConv, kMean>(td, off, s, c, bad, stage_smem, plan.status);
    } else {
      if (threadIdx.x >= kThreads) return;     // the producer warp has no part in the register path
      bad = tile_registers_outlined<GradT, kOpt, kConv, kMean>(td, off, rest < kTileElems ? (int)rest : kTileElems, &s, c);
    }
    if (bad) atomicOr(plan.status, 1u);
  } else {
    stage_scalars(s, s_param, plan.scal_dev);
    const AdamConsts c{s.one_minus_beta1, s.one_minus_beta2, s.rsqrt_bc2, s.eps, s.momentum};
    bool bad = false;
    for (int t = blockIdx.x; t < plan.n_tiles; t += gridDim.x) {
      const Tile tile = plan.tiles[t];
      TensorDesc td = plan.tensors[tile.tensor];
      td.partial = plan.partial ? plan.partial + td.partial_off : nullptr;
      const long long off = (long long)tile.tile * kTileElems;
      const long long rest = td.numel - off;
      tile_registers<GradT, kOpt, kConv, kMean, kTileVecs>(td, off, rest < kTileElems ? (int)rest : kTileElems, s, c, bad);
    }
    if (bad) atomicOr(plan.status, 1u);
  }
}

// ---- AdamW with ONE pair of moments for all replicas ------------------------------------------------
// When every replica sees the same gradient (a shared gradient as in Eq. 2, or the replica mean of
// Algorithm 1's gradient all-reduce) the Adam moments are identical on all replicas: they are stored
// once (state_stride = 0), updated once per tile, and the step direction u = m / (sqrt(v)/sqrt(bc2) + eps)
// is computed once; each replica then costs two fused multiply-adds per element:
//   theta_r <- theta_r - (lr_r wd_r) theta_r - (lr_r / bc1) u.
// Bytes per replica-element: 8 (theta) + (gradient + 16) / N, or 8 + gradient + 16 / N with the mean.
constexpr int kChunk = 8;      // replicas of one vector whose parameters are loaded together
constexpr int kGradChunk = 4;  // replicas whose bf16 gradients are loaded together for the mean (fp32: half)

template <typename GradT, bool kConv, bool kMean>
__device__ void range_scalar_shared(const TensorDesc& td, long long begin, long long end, const StepScalars& s,
                                    const AdamConsts& c, bool& bad) {
  const int n = s.n_replicas;
  const GradT* grad = static_cast<const GradT*>(td.grad);
  for (long long e = begin + threadIdx.x; e < end; e += kThreads) {
    float g;
    if (kMean) {
      double acc = 0.0;
      for (int r = 0; r < n; ++r) acc += (double)load_scalar(grad + r * td.grad_stride + e);
      g = (float)(acc * s.inv_n);
    } else {
      g = load_scalar(grad + e);
    }
    float m = __ldcs(td.exp_avg + e), v = __ldcs(td.exp_avg_sq + e);
    m = fmaf(c.one_minus_beta1, g - m, m);
    v = fmaf(c.one_minus_beta2, fmaf(g, g, -v), v);
    const float u = m / fmaf(sqrtf(v), c.rsqrt_bc2, c.eps);
    __stcs(td.exp_avg + e, m);
    __stcs(td.exp_avg_sq + e, v);
    double sum = 0.0;
    for (int r = 0; r < n; ++r) {
      float th = __ldcs(td.param + r * td.param_stride + e);
      th = fmaf(-s.step[td.group][r], u, fmaf(-s.lr_wd[td.group][r], th, th));
      bad |= not_finite(th);
      if (kConv) sum += (double)th;
      else __stcs(td.param + r * td.param_stride + e, th);
    }
    if (kConv) {
      if (td.partial) {
        td.partial[e] = (float)sum;       // replica axis sharded over GPUs: hand out the local sum instead
      } else {
        const float mean = (float)(sum * s.inv_n);
        for (int r = 0; r < n; ++r) __stcs(td.param + r * td.param_stride + e, mean);
        if (td.param_bf16) td.param_bf16[e] = bf16_bits(mean);
      }
    }
  }
}

template <typename GradT, bool kConv, bool kMean, bool kFull>
__device__ __forceinline__ void tile_vector_shared(const TensorDesc& td, long long off, int nvec,
                                                   const StepScalars& s, const AdamConsts& c, bool& bad) {
  const int n = s.n_replicas;
  const int grp = td.group;
  float* const P = td.param + off;
  float* const M = td.exp_avg + off;
  float* const V = td.exp_avg_sq + off;
  const GradT* const Gp = static_cast<const GradT*>(td.grad) + off;
  const long long ps = td.param_stride, gs = td.grad_stride;

  // One float4 vector at a time: all loads of the vector (up to kChunk replicas of theta, the gradient(s),
  // both moments) are issued together, so little register state is needed and three CTAs fit on an SM.
#pragma unroll
  for (int k = 0; k < kTileVecs; ++k) {
    const int j = k * kThreads + threadIdx.x;
    if (!kFull && j >= nvec) continue;
    const int at = j * 4;

    // All loads of the vector are requested before anything is consumed.  For the replica mean the N
    // gradient loads come in groups of kG replicas whose fp64 sum needs the previous group, so the
    // parameter loads are spread over the same groups: every wait covers a full wave of loads instead of
    // a thin one of gradients only.
    float4 th[kChunk];
    float4 m4, v4;
    float g[4];
    if constexpr (kMean) {
      double acc[4] = {0.0, 0.0, 0.0, 0.0};
      constexpr int kG = sizeof(typename GradRaw<GradT>::type) == 16 ? kGradChunk / 2 : kGradChunk;
      m4 = __ldcs(reinterpret_cast<const float4*>(M + at));
      v4 = __ldcs(reinterpret_cast<const float4*>(V + at));
#pragma unroll
      for (int r0 = 0; r0 < kChunk; r0 += kG) {                      // replicas 0 .. kChunk-1, unrolled
        typename GradRaw<GradT>::type raw[kG];
#pragma unroll
        for (int q = 0; q < kG; ++q) {
          if (r0 + q < n) {
            raw[q] = load_raw(Gp + (r0 + q) * gs + at);
            th[r0 + q] = __ldcs(reinterpret_cast<const float4*>(P + (r0 + q) * ps + at));
          } else {
            raw[q] = typename GradRaw<GradT>::type{};
            th[r0 + q] = make_float4(0.f, 0.f, 0.f, 0.f);
          }
        }
        asm volatile("" ::: "memory");                                // keep the next group's loads after this wait
#pragma unroll
        for (int q = 0; q < kG; ++q) {
          float gr[4];
          unpack(raw[q], gr);
#pragma unroll
          for (int e = 0; e < 4; ++e) acc[e] += (double)gr[e];
        }
      }
      for (int r0 = kChunk; r0 < n; r0 += kG) {                       // gradients of further replicas
        typename GradRaw<GradT>::type raw[kG];
#pragma unroll
        for (int q = 0; q < kG; ++q)
          raw[q] = r0 + q < n ? load_raw(Gp + (r0 + q) * gs + at) : typename GradRaw<GradT>::type{};
#pragma unroll
        for (int q = 0; q < kG; ++q) {
          float gr[4];
          unpack(raw[q], gr);
#pragma unroll
          for (int e = 0; e < 4; ++e) acc[e] += (double)gr[e];
        }
      }
#pragma unroll
      for (int q = 0; q < 4; ++q) g[q] = (float)(acc[q] * s.inv_n);
    } else {
#pragma unroll
      for (int q = 0; q < kChunk; ++q)
        th[q] = q < n ? __ldcs(reinterpret_cast<const float4*>(P + q * ps + at)) : make_float4(0.f, 0.f, 0.f, 0.f);
      m4 = __ldcs(reinterpret_cast<const float4*>(M + at));
      v4 = __ldcs(reinterpret_cast<const float4*>(V + at));
      unpack(load_raw(Gp + at), g);
    }

    // Step direction u = m' / (sqrt(v')/sqrt(bc2) + eps), once per element for all replicas.
    float m[4] = {m4.x, m4.y, m4.z, m4.w};
    float v[4] = {v4.x, v4.y, v4.z, v4.w};
    float u[4];
#pragma unroll
    for (int q = 0; q < 4; ++q) {
      m[q] = fmaf(c.one_minus_beta1, g[q] - m[q], m[q]);
      v[q] = fmaf(c.one_minus_beta2, fmaf(g[q], g[q], -v[q]), v[q]);
      u[q] = m[q] / fmaf(sqrtf(v[q]), c.rsqrt_bc2, c.eps);
    }
    __stcs(reinterpret_cast<float4*>(M + at), make_float4(m[0], m[1], m[2], m[3]));
    __stcs(reinterpret_cast<float4*>(V + at), make_float4(v[0], v[1], v[2], v[3]));

    double sum[4] = {0.0, 0.0, 0.0, 0.0};
    for (int r0 = 0; r0 < n; r0 += kChunk) {
      if (r0 > 0) {
#pragma unroll
        for (int q = 0; q < kChunk; ++q)
          th[q] = r0 + q < n ? __ldcs(reinterpret_cast<const float4*>(P + (r0 + q) * ps + at))
                             : make_float4(0.f, 0.f, 0.f, 0.f);
      }
#pragma unroll
      for (int q = 0; q < kChunk; ++q) {
        const int r = r0 + q;
        if (r < n) {
          const float lr_wd = s.lr_wd[grp][r];
          const float step = s.step[grp][r];
          float t4[4] = {th[q].x, th[q].y, th[q].z, th[q].w};
#pragma unroll
          for (int e = 0; e < 4; ++e) {
            t4[e] = fmaf(-step, u[e], fmaf(-lr_wd, t4[e], t4[e]));
            bad |= not_finite(t4[e]);
          }
          if (kConv) {
#pragma unroll
            for (int e = 0; e < 4; ++e) sum[e] += (double)t4[e];
          } else {
            __stcs(reinterpret_cast<float4*>(P + r * ps + at), make_float4(t4[0], t4[1], t4[2], t4[3]));
          }
        }
      }
    }
    if (kConv) {
      if (td.partial) {
        *reinterpret_cast<float4*>(td.partial + off + at) =
            make_float4((float)sum[0], (float)sum[1], (float)sum[2], (float)sum[3]);
      } else {
        const float4 mean = make_float4((float)(sum[0] * s.inv_n), (float)(sum[1] * s.inv_n),
                                        (float)(sum[2] * s.inv_n), (float)(sum[3] * s.inv_n));
        for (int rr = 0; rr < n; ++rr) __stcs(reinterpret_cast<float4*>(P + rr * ps + at), mean);
        if (td.param_bf16) __stcs(reinterpret_cast<uint2*>(td.param_bf16 + off + at), bf16_bits4(mean));
      }
    }
  }
}

// Three CTAs per SM (80 registers).  Six of the eight instantiations then spill 8 - 96 bytes per thread; giving
// those two CTAs and 128 registers instead removes the spills and measured 2 - 10 % SLOWER on the 1.3 B list
// (6.26 against 6.63 TB/s for the gradient mean with converge): the third CTA's loads in flight are worth more
// than the few spilled values, which stay in L1.
template <typename GradT, bool kConv, bool kMean>
__global__ void __launch_bounds__(kThreads, 3)
fanout_shared_kernel(const __grid_constant__ LaunchPlan plan, const __grid_constant__ StepScalars s_param) {
  __shared__ StepScalars s;
  stage_scalars(s, s_param, plan.scal_dev);
  const AdamConsts c{s.one_minus_beta1, s.one_minus_beta2, s.rsqrt_bc2, s.eps, s.momentum};
  bool bad = false;
  for (int t = blockIdx.x; t < plan.n_tiles; t += gridDim.x) {
    const Tile tile = plan.tiles[t];
    TensorDesc td = plan.tensors[tile.tensor];
    td.partial = plan.partial ? plan.partial + td.partial_off : nullptr;
    const long long off = (long long)tile.tile * kTileElems;
    const long long rest = td.numel - off;
    const int len = rest < kTileElems ? (int)rest : kTileElems;
    if (td.vec) {
      if (len == kTileElems) {
        tile_vector_shared<GradT, kConv, kMean, true>(td, off, kThreads * kTileVecs, s, c, bad);
      } else {
        const int nvec = len >> 2;
        if (nvec) tile_vector_shared<GradT, kConv, kMean, false>(td, off, nvec, s, c, bad);
        if (len & 3) range_scalar_shared<GradT, kConv, kMean>(td, off + 4ll * nvec, off + len, s, c, bad);
      }
    } else {
      range_scalar_shared<GradT, kConv, kMean>(td, off, off + len, s, c, bad);
    }
  }
  if (bad) atomicOr(plan.status, 1u);
}


// ---- stand-alone converge (Eq. 3) -------------------------------------------------------------
__global__ void __launch_bounds__(kThreads, 4)
converge_kernel(const __grid_constant__ LaunchPlan plan, int n, double inv_n) {
  for (int t = blockIdx.x; t < plan.n_tiles; t += gridDim.x) {
    const Tile tile = plan.tiles[t];
    const TensorDesc td = plan.tensors[tile.tensor];
    converge_tile(td, tile.tile, n, inv_n);
  }
}

// ---- second half of a converge whose replica axis is sharded over GPUs ----------------------------
// plan.partial holds, per element, the sum over ALL replicas of all GPUs (the local sums after an
// all-reduce); every local replica receives sum / N_global (Eq. 3).
__global__ void __launch_bounds__(kThreads, 4)
apply_mean_kernel(const __grid_constant__ LaunchPlan plan, int n_local, double inv_n_global) {
  for (int t = blockIdx.x; t < plan.n_tiles; t += gridDim.x) {
    const Tile tile = plan.tiles[t];
    const TensorDesc td = plan.tensors[tile.tensor];
    const long long off = (long long)tile.tile * kTileElems;
    const long long rest = td.numel - off;
    const int len = rest < kTileElems ? (int)rest : kTileElems;
    const int nvec = td.vec ? (len >> 2) : 0;
    float* const P = td.param + off;
    const float* const S = plan.partial + td.partial_off + off;
    for (int j = threadIdx.x; j < nvec; j += kThreads) {
      const float4 x = __ldcs(reinterpret_cast<const float4*>(S + 4 * j));
      const float4 mean = make_float4((float)(x.x * inv_n_global), (float)(x.y * inv_n_global),
                                      (float)(x.z * inv_n_global), (float)(x.w * inv_n_global));
      for (int r = 0; r < n_local; ++r) __stcs(reinterpret_cast<float4*>(P + r * td.param_stride + 4 * j), mean);
      if (td.param_bf16) __stcs(reinterpret_cast<uint2*>(td.param_bf16 + off + 4 * j), bf16_bits4(mean));
    }
    for (int e = 4 * nvec + threadIdx.x; e < len; e += kThreads) {
      const float mean = (float)(__ldcs(S + e) * inv_n_global);
      for (int r = 0; r < n_local; ++r) __stcs(P + r * td.param_stride + e, mean);
      if (td.param_bf16) td.param_bf16[off + e] = bf16_bits(mean);
    }
  }
}

// ---- the same with the exchange inside the kernel: plain loads from every rank's staging buffer ---------
// bufs.p[b] is rank b's staging buffer (this GPU's own, or a peer's mapped into this process and read over
// NVLink with ordinary loads).  The sums are added in rank order b = 0..B-1 in fp64, so every rank computes the
// same bits; the mean goes to the local replicas.  The kernel waits for nobody: the caller orders it after every
// rank's hdet_step_sharded (a barrier between the two launches) and keeps the buffers untouched until every
// rank's launch of this kernel has finished.
struct PeerBuffers {
  const float* p[HDET_MAX_REPLICAS];
  int count;
};

__global__ void __launch_bounds__(kThreads, 4)
apply_mean_peers_kernel(const __grid_constant__ LaunchPlan plan, const __grid_constant__ PeerBuffers bufs, int n_local,
                        double inv_n_global) {
  for (int t = blockIdx.x; t < plan.n_tiles; t += gridDim.x) {
    const Tile tile = plan.tiles[t];
    const TensorDesc td = plan.tensors[tile.tensor];
    const long long off = (long long)tile.tile * kTileElems;
    const long long rest = td.numel - off;
    const int len = rest < kTileElems ? (int)rest : kTileElems;
    const int nvec = td.vec ? (len >> 2) : 0;
    float* const P = td.param + off;
    const long long at = td.partial_off + off;
    for (int j = threadIdx.x; j < nvec; j += kThreads) {
      double s0 = 0.0, s1 = 0.0, s2 = 0.0, s3 = 0.0;
#pragma unroll 4
      for (int b = 0; b < bufs.count; ++b) {
        const float4 x = __ldcs(reinterpret_cast<const float4*>(bufs.p[b] + at + 4 * j));
        s0 += (double)x.x; s1 += (double)x.y; s2 += (double)x.z; s3 += (double)x.w;
      }
      const float4 mean = make_float4((float)(s0 * inv_n_global), (float)(s1 * inv_n_global),
                                      (float)(s2 * inv_n_global), (float)(s3 * inv_n_global));
      for (int r = 0; r < n_local; ++r) __stcs(reinterpret_cast<float4*>(P + r * td.param_stride + 4 * j), mean);
      if (td.param_bf16) __stcs(reinterpret_cast<uint2*>(td.param_bf16 + off + 4 * j), bf16_bits4(mean));
    }
    for (int e = 4 * nvec + threadIdx.x; e < len; e += kThreads) {
      double sum = 0.0;
      for (int b = 0; b < bufs.count; ++b) sum += (double)__ldcs(bufs.p[b] + at + e);
      const float mean = (float)(sum * inv_n_global);
      for (int r = 0; r < n_local; ++r) __stcs(P + r * td.param_stride + e, mean);
      if (td.param_bf16) td.param_bf16[off + e] = bf16_bits(mean);
    }
  }
}

// The stage ring needs more dynamic shared memory than the default limit: opt in once per device and kernel.
template <typename Kernel>
cudaError_t opt_in_shared_memory(Kernel kernel, int bytes, bool (&opted_in)[kMaxDevices]) {
  int dev = 0;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return e;
  if (dev < 0 || dev >= kMaxDevices) return cudaErrorInvalidDevice;
  if (!opted_in[dev]) {
    e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes);
    if (e != cudaSuccess) return e;
    opted_in[dev] = true;
  }
  return cudaSuccess;
}

template <typename GradT, int kOpt, bool kConv, bool kMean>
cudaError_t opt_in_one() {
  if constexpr (kHasBulkPath<kOpt>) {
    static bool opted_in[kMaxDevices] = {};
    return opt_in_shared_memory(fanout_kernel<GradT, kOpt, kConv, kMean>, (int)BulkLayout<GradT>::kBytes, opted_in);
  }
  return cudaSuccess;
}

template <typename GradT, int kOpt, bool kConv, bool kMean>
cudaError_t launch_one(const LaunchPlan& plan, const StepScalars& s, cudaStream_t stream) {
  if constexpr (kHasBulkPath<kOpt>) {
    const cudaError_t e = opt_in_one<GradT, kOpt, kConv, kMean>();   // a flag check after the first time
    if (e != cudaSuccess) return e;
    fanout_kernel<GradT, kOpt, kConv, kMean>
        <<<plan.n_tiles, kThreads + kProducerThreads, BulkLayout<GradT>::kBytes, stream>>>(plan, s);
  } else {
    fanout_kernel<GradT, kOpt, kConv, kMean><<<plan.grid, kThreads, 0, stream>>>(plan, s);
  }
  return cudaGetLastError();
}

template <typename GradT, bool kConv, bool kMean>
cudaError_t launch_shared(const LaunchPlan& plan, const StepScalars& s, cudaStream_t stream) {
  fanout_shared_kernel<GradT, kConv, kMean><<<plan.grid, kThreads, 0, stream>>>(plan, s);
  return cudaGetLastError();
}

template <typename GradT, bool kConv, bool kMean>
cudaError_t pick_state(int opt, bool shared_state, const LaunchPlan& plan, const StepScalars& s, cudaStream_t st) {
  if (opt == kOptAdamW && shared_state) return launch_shared<GradT, kConv, kMean>(plan, s, st);
  if (opt == kOptAdamW) return launch_one<GradT, kOptAdamW, kConv, kMean>(plan, s, st);
  if (opt == kOptSgdMomentum) return launch_one<GradT, kOptSgdMomentum, kConv, kMean>(plan, s, st);
  return launch_one<GradT, kOptSgd, kConv, kMean>(plan, s, st);
}

template <typename GradT>
cudaError_t pick_flags(int opt, bool converge, bool mean, bool shared_state, const LaunchPlan& plan,
                       const StepScalars& s, cudaStream_t st) {
  if (converge) return mean ? pick_state<GradT, true, true>(opt, shared_state, plan, s, st)
                            : pick_state<GradT, true, false>(opt, shared_state, plan, s, st);
  return mean ? pick_state<GradT, false, true>(opt, shared_state, plan, s, st)
              : pick_state<GradT, false, false>(opt, shared_state, plan, s, st);
}

}  // namespace

cudaError_t prepare_fanout(int optimizer, int grad_dtype, bool grad_mean, bool shared_state) {
  if (optimizer != HDET_OPT_ADAMW || shared_state) return cudaSuccess;     // only the bulk-copy kernels need it
  cudaError_t e;
  if (grad_dtype == HDET_DTYPE_BF16) {
    e = grad_mean ? opt_in_one<__nv_bfloat16, kOptAdamW, true, true>() : opt_in_one<__nv_bfloat16, kOptAdamW, true, false>();
    if (e == cudaSuccess)
      e = grad_mean ? opt_in_one<__nv_bfloat16, kOptAdamW, false, true>() : opt_in_one<__nv_bfloat16, kOptAdamW, false, false>();
  } else {
    e = grad_mean ? opt_in_one<float, kOptAdamW, true, true>() : opt_in_one<float, kOptAdamW, true, false>();
    if (e == cudaSuccess)
      e = grad_mean ? opt_in_one<float, kOptAdamW, false, true>() : opt_in_one<float, kOptAdamW, false, false>();
  }
  return e;
}

cudaError_t launch_fanout(int optimizer, bool sgd_momentum, int grad_dtype, bool converge, bool grad_mean,
                          bool shared_state, const LaunchPlan& plan, const StepScalars& s, cudaStream_t stream) {
  if (plan.n_tiles == 0) return cudaSuccess;
  const int opt = optimizer == HDET_OPT_ADAMW ? kOptAdamW : (sgd_momentum ? kOptSgdMomentum : kOptSgd);
  if (grad_dtype == HDET_DTYPE_BF16)
    return pick_flags<__nv_bfloat16>(opt, converge, grad_mean, shared_state, plan, s, stream);
  return pick_flags<float>(opt, converge, grad_mean, shared_state, plan, s, stream);
}

// One CTA waits, with the limit every bulk-copy wait has, on a barrier that nothing will complete, and records
// the outcome the way tile_bulk does.
__global__ void bounded_wait_probe_kernel(unsigned* status) {
  __shared__ __align__(8) unsigned long long barrier;
  const uint32_t bar = bulk::smem_addr(&barrier);
  if (threadIdx.x == 0) {
    bulk::barrier_init(bar, 1);
    bulk::barrier_init_fence();
  }
  __syncthreads();
  if (!bulk::barrier_wait(bar, 0) && threadIdx.x == 0) atomicOr(status, 2u);
}

cudaError_t launch_bounded_wait_probe(unsigned* status, cudaStream_t stream) {
  bounded_wait_probe_kernel<<<1, 32, 0, stream>>>(status);
  return cudaGetLastError();
}

cudaError_t launch_apply_mean(const LaunchPlan& plan, int n_local, double inv_n_global, cudaStream_t stream) {
  if (plan.n_tiles == 0) return cudaSuccess;
  apply_mean_kernel<<<plan.grid, kThreads, 0, stream>>>(plan, n_local, inv_n_global);
  return cudaGetLastError();
}

cudaError_t launch_apply_mean_peers(const LaunchPlan& plan, const float* const* buffers, int n_buffers, int n_local,
                                    double inv_n_global, cudaStream_t stream) {
  if (plan.n_tiles == 0) return cudaSuccess;
  PeerBuffers bufs{};
  for (int b = 0; b < n_buffers; ++b) bufs.p[b] = buffers[b];
  bufs.count = n_buffers;
  apply_mean_peers_kernel<<<plan.grid, kThreads, 0, stream>>>(plan, bufs, n_local, inv_n_global);
  return cudaGetLastError();
}

cudaError_t launch_converge(const LaunchPlan& plan, int n_replicas, cudaStream_t stream) {
  if (plan.n_tiles == 0) return cudaSuccess;
  converge_kernel<<<plan.grid, kThreads, 0, stream>>>(plan, n_replicas, 1.0 / (double)n_replicas);
  return cudaGetLastError();
}

}  // namespace hdet
