// C ABI of libhdet (see include/hdet.h): argument checks, the host-side scalar state of
// Algorithm 1 in double precision, and the kernel launches.
#include <cmath>
#include <cstdio>
#include <cstring>
#include <new>
#include <string>
#include <vector>

#include "hdet_device_state.cuh"
#include "hdet_internal.h"
#include "hdet_kernels.cuh"
#include "hdet_scalars.h"

using namespace hdet;

struct hdet_ctx {
  hdet_config cfg{};
  // schedule
  bool has_schedule = false;
  hdet_schedule sched{};
  double max_lr[HDET_MAX_GROUPS]{};
  double weight_decay[HDET_MAX_GROUPS]{};
  // Algorithm 1 state
  int64_t step = 0;
  int64_t n_acc = 0;
  bool fired = false;
  bool round_ended = false;
  double base[HDET_MAX_GROUPS]{};
  double ctrl_base[HDET_MAX_GROUPS]{};
  double velocity[HDET_MAX_GROUPS]{};
  double delta[HDET_MAX_GROUPS]{};
  double wd_base[HDET_MAX_GROUPS]{};       // base weight decay per group (Remark 1 channel)
  double wd_velocity[HDET_MAX_GROUPS]{};
  double wd_delta[HDET_MAX_GROUPS]{};
  double lr[HDET_MAX_GROUPS][HDET_MAX_REPLICAS]{};
  double wd[HDET_MAX_GROUPS][HDET_MAX_REPLICAS]{};
  int32_t perm_lr[HDET_MAX_GROUPS][HDET_MAX_REPLICAS]{};
  int32_t perm_wd[HDET_MAX_GROUPS][HDET_MAX_REPLICAS]{};
  double weights[HDET_MAX_REPLICAS]{};
  double loss_acc[HDET_MAX_REPLICAS]{};
  double loss_round[HDET_MAX_REPLICAS]{};
  double rho_lr[HDET_MAX_REPLICAS]{};
  double rho_wd[HDET_MAX_REPLICAS]{};
  // device side
  int64_t n_tensors = 0;
  TensorDesc* d_tensors = nullptr;
  Tile* d_tiles = nullptr;
  unsigned* d_status = nullptr;
  double* d_warm = nullptr;      // scratch of hdet_warm_init (n_tiles + 1 doubles), allocated on its first call
  double total_numel = 0.0;      // d of Eq. 10
  DevState* d_state = nullptr;   // device-resident scalar state (used by hdet_step_device)
  bool device_mode = false;      // the device copy of the state is the authoritative one
  int n_tiles = 0;
  int grid_fanout = 0;
  int grid_converge = 0;
  bool shared_state = false;   // AdamW with one pair of moments for all replicas
  int n_global = 0;            // N of Eq. 1 over all GPUs (= cfg.n_replicas unless the replica axis is sharded)
  int r_offset = 0;            // global index of local replica 0
  int64_t partial_numel = 0;   // elements of the partial-sum staging buffer
  std::vector<int64_t> partial_offsets;  // per tensor, inside that buffer
  std::vector<hdet_tensor> tensors;      // the caller's descriptors (for hdet_step_host_grads)
  // hdet_step_host_grads uploads the gradients in a few runs of consecutive tensors on a stream of its own and
  // updates each run's tiles as soon as its copies have landed, so that copies and updates overlap.
  struct UploadRun { int64_t first_tensor, n_tensors; int first_tile, n_tiles; };
  std::vector<UploadRun> upload_runs;
  cudaStream_t copy_stream = nullptr;    // created by the first hdet_step_host_grads call
  cudaEvent_t upload_begin = nullptr;
  std::vector<cudaEvent_t> upload_done;  // one per run
  int64_t launches = 0;
  std::string error;
};

namespace {

thread_local std::string g_create_error;

int fail(hdet_ctx* h, int code, const std::string& msg) {
  if (h) h->error = msg; else g_create_error = msg;
  return code;
}

int fail_cuda(hdet_ctx* h, const char* what, cudaError_t e) {
  return fail(h, HDET_ERR_CUDA, std::string(what) + ": " + cudaGetErrorString(e));
}

bool aligned(const void* p, size_t a) { return (reinterpret_cast<uintptr_t>(p) % a) == 0; }

// Sets the handle's device for the scope of one call and restores the caller's.
struct DeviceScope {
  int prev = -1;
  bool switched = false;
  cudaError_t err = cudaSuccess;
  explicit DeviceScope(int dev) {
    err = cudaGetDevice(&prev);
    if (err == cudaSuccess && prev != dev) {
      err = cudaSetDevice(dev);
      switched = err == cudaSuccess;
    }
  }
  ~DeviceScope() { if (switched) cudaSetDevice(prev); }
};

void free_device(hdet_ctx* h) {
  if (h->d_tensors) cudaFree(h->d_tensors);
  if (h->d_tiles) cudaFree(h->d_tiles);
  if (h->d_status) cudaFree(h->d_status);
  if (h->d_state) cudaFree(h->d_state);
  if (h->d_warm) cudaFree(h->d_warm);
  if (h->copy_stream) cudaStreamDestroy(h->copy_stream);
  if (h->upload_begin) cudaEventDestroy(h->upload_begin);
  for (cudaEvent_t ev : h->upload_done) cudaEventDestroy(ev);
  h->copy_stream = nullptr; h->upload_begin = nullptr; h->upload_done.clear();
  h->d_warm = nullptr;
  h->d_tensors = nullptr; h->d_tiles = nullptr; h->d_status = nullptr; h->d_state = nullptr;
}

// Rates and weight decays for the update at 0-based index h->step.
void compute_tables(hdet_ctx* h) {
  const int n = h->n_global, G = h->cfg.n_groups;
  for (int g = 0; g < G; ++g) {
    const double b = h->fired ? h->ctrl_base[g]
                              : base_rate(h->sched.kind, h->step, h->sched.total_steps, h->max_lr[g],
                                          h->sched.pct_start, h->sched.div_factor, h->sched.final_div_factor);
    h->base[g] = b;
    for (int r = 0; r < n; ++r) {
      h->lr[g][r] = b * h->rho_lr[h->perm_lr[g][r]];
      h->wd[g][r] = h->wd_base[g] * h->rho_wd[h->perm_wd[g][r]];
    }
  }
}

bool is_permutation(const int32_t* p, int n) {
  bool seen[HDET_MAX_REPLICAS] = {};
  for (int r = 0; r < n; ++r) {
    if (p[r] < 0 || p[r] >= n || seen[p[r]]) return false;
    seen[p[r]] = true;
  }
  return true;
}

// Host fields -> public state block (no device access).
void export_state(const hdet_ctx* h, hdet_state* out) {
  std::memset(out, 0, sizeof *out);
  out->step = h->step;
  out->n_acc = h->n_acc;
  out->fired = h->fired;
  out->round_ended = h->round_ended;
  std::memcpy(out->base, h->base, sizeof h->base);
  std::memcpy(out->ctrl_base, h->ctrl_base, sizeof h->ctrl_base);
  std::memcpy(out->velocity, h->velocity, sizeof h->velocity);
  std::memcpy(out->delta, h->delta, sizeof h->delta);
  std::memcpy(out->lr, h->lr, sizeof h->lr);
  std::memcpy(out->wd, h->wd, sizeof h->wd);
  std::memcpy(out->perm_lr, h->perm_lr, sizeof h->perm_lr);
  std::memcpy(out->perm_wd, h->perm_wd, sizeof h->perm_wd);
  std::memcpy(out->weights, h->weights, sizeof h->weights);
  std::memcpy(out->loss_acc, h->loss_acc, sizeof h->loss_acc);
  std::memcpy(out->loss_round, h->loss_round, sizeof h->loss_round);
  std::memcpy(out->wd_base, h->wd_base, sizeof h->wd_base);
  std::memcpy(out->wd_velocity, h->wd_velocity, sizeof h->wd_velocity);
  std::memcpy(out->wd_delta, h->wd_delta, sizeof h->wd_delta);
  out->gamma = h->has_schedule ? decay_gamma(h->sched.f_div, h->sched.f_final, h->sched.total_steps,
                                             h->sched.warmup_steps, h->cfg.sync_interval)
                               : 0.0;
}

// Public state block -> host fields (everything, including the tables of the last update).
void import_state(hdet_ctx* h, const hdet_state* in) {
  h->step = in->step;
  h->n_acc = in->n_acc;
  h->fired = in->fired != 0;
  h->round_ended = in->round_ended != 0;
  std::memcpy(h->base, in->base, sizeof h->base);
  std::memcpy(h->ctrl_base, in->ctrl_base, sizeof h->ctrl_base);
  std::memcpy(h->velocity, in->velocity, sizeof h->velocity);
  std::memcpy(h->delta, in->delta, sizeof h->delta);
  std::memcpy(h->lr, in->lr, sizeof h->lr);
  std::memcpy(h->wd, in->wd, sizeof h->wd);
  std::memcpy(h->perm_lr, in->perm_lr, sizeof h->perm_lr);
  std::memcpy(h->perm_wd, in->perm_wd, sizeof h->perm_wd);
  std::memcpy(h->weights, in->weights, sizeof h->weights);
  std::memcpy(h->loss_acc, in->loss_acc, sizeof h->loss_acc);
  std::memcpy(h->loss_round, in->loss_round, sizeof h->loss_round);
  std::memcpy(h->wd_base, in->wd_base, sizeof h->wd_base);
  std::memcpy(h->wd_velocity, in->wd_velocity, sizeof h->wd_velocity);
  std::memcpy(h->wd_delta, in->wd_delta, sizeof h->wd_delta);
}

DevConst device_constants(const hdet_ctx* h) {
  DevConst c{};
  c.n = h->n_global;
  c.n_groups = h->cfg.n_groups;
  c.adam = h->cfg.optimizer == HDET_OPT_ADAMW;
  c.kind = h->sched.kind;
  c.autolr = h->sched.autolr;
  c.auto_wd = h->sched.auto_wd;
  c.reshuffle = h->cfg.reshuffle;
  c.total_steps = h->sched.total_steps;
  c.warmup_steps = h->sched.warmup_steps;
  c.sync_interval = h->cfg.sync_interval;
  c.beta1 = h->cfg.beta1; c.beta2 = h->cfg.beta2; c.eps = h->cfg.eps; c.momentum = h->cfg.momentum;
  c.alpha_lr = h->cfg.alpha_lr; c.alpha_wd = h->cfg.alpha_wd;
  c.pct_start = h->sched.pct_start; c.div_factor = h->sched.div_factor; c.final_div_factor = h->sched.final_div_factor;
  c.ctrl_beta = h->sched.beta; c.sigma = h->sched.sigma; c.lambda = h->sched.lambda;
  c.f_div = h->sched.f_div; c.f_final = h->sched.f_final;
  for (int g = 0; g < HDET_MAX_GROUPS; ++g) { c.max_lr[g] = h->max_lr[g]; c.weight_decay[g] = h->weight_decay[g]; }
  c.seed = h->cfg.seed;
  return c;
}

// What hdet_create derives from the descriptors before it touches a device: per-tensor device descriptors
// (access path chosen from the alignment), the tile table and the layout of the partial-sum staging buffer.
struct WorkPlan {
  std::vector<TensorDesc> descs;
  std::vector<Tile> tiles;
  int64_t n_shared_state = 0;
  int64_t partial_numel = 0;
};

// Checks cfg and the descriptors and fills `out`.  Host arithmetic only.
int plan_work(const hdet_config* cfg, const hdet_tensor* tensors, int64_t n_tensors, WorkPlan& out) {
  if (n_tensors < 0 || (n_tensors > 0 && !tensors))
    return fail(nullptr, HDET_ERR_INVALID_ARG, "hdet_create: tensors is NULL or n_tensors < 0");
  if (cfg->n_replicas < 1 || cfg->n_replicas > HDET_MAX_REPLICAS)
    return fail(nullptr, HDET_ERR_INVALID_ARG, "hdet_create: n_replicas must be in 1..32");
  if (cfg->n_groups < 1 || cfg->n_groups > HDET_MAX_GROUPS)
    return fail(nullptr, HDET_ERR_INVALID_ARG, "hdet_create: n_groups must be in 1..8");
  if (cfg->optimizer != HDET_OPT_SGD && cfg->optimizer != HDET_OPT_ADAMW)
    return fail(nullptr, HDET_ERR_INVALID_ARG, "hdet_create: unknown optimizer");
  if (cfg->grad_dtype != HDET_DTYPE_F32 && cfg->grad_dtype != HDET_DTYPE_BF16)
    return fail(nullptr, HDET_ERR_INVALID_ARG, "hdet_create: unknown grad_dtype");
  if (!(cfg->alpha_lr >= 0.0 && cfg->alpha_lr < 1.0) || !(cfg->alpha_wd >= 0.0 && cfg->alpha_wd < 1.0))
    return fail(nullptr, HDET_ERR_INVALID_ARG, "hdet_create: spread ratios must satisfy 0 <= alpha < 1");
  if (cfg->sync_interval < 1) return fail(nullptr, HDET_ERR_INVALID_ARG, "hdet_create: sync_interval must be >= 1");
  if (cfg->optimizer == HDET_OPT_ADAMW) {
    if (!(cfg->beta1 >= 0.0 && cfg->beta1 < 1.0) || !(cfg->beta2 >= 0.0 && cfg->beta2 < 1.0) || !(cfg->eps >= 0.0))
      return fail(nullptr, HDET_ERR_INVALID_ARG, "hdet_create: need 0 <= beta1, beta2 < 1 and eps >= 0");
  }
  if (!(cfg->momentum >= 0.0 && cfg->momentum < 1.0))
    return fail(nullptr, HDET_ERR_INVALID_ARG, "hdet_create: need 0 <= momentum < 1");
  if (cfg->momentum != 0.0 && cfg->optimizer != HDET_OPT_SGD)
    return fail(nullptr, HDET_ERR_INVALID_ARG, "hdet_create: momentum applies to HDET_OPT_SGD only");
  if (cfg->grad_mode != HDET_GRAD_AS_GIVEN && cfg->grad_mode != HDET_GRAD_REPLICA_MEAN)
    return fail(nullptr, HDET_ERR_INVALID_ARG, "hdet_create: unknown grad_mode");

  const int n = cfg->n_replicas;
  const bool sharded = cfg->n_replicas_global != 0;
  const int n_global = sharded ? cfg->n_replicas_global : n;
  if (sharded && (cfg->replica_offset < 0 || n_global > HDET_MAX_REPLICAS || cfg->replica_offset + n > n_global))
    return fail(nullptr, HDET_ERR_INVALID_ARG,
                "hdet_create: need 0 <= replica_offset and replica_offset + n_replicas <= n_replicas_global <= 32");
  if (sharded && cfg->grad_mode == HDET_GRAD_REPLICA_MEAN)
    return fail(nullptr, HDET_ERR_UNSUPPORTED,
                "hdet_create: with a sharded replica axis the gradient mean spans GPUs; all-reduce it and pass a shared gradient");
  const size_t gsz = cfg->grad_dtype == HDET_DTYPE_BF16 ? 2 : 4;
  std::vector<TensorDesc>& descs = out.descs;
  std::vector<Tile>& tiles = out.tiles;
  int64_t& n_shared_state = out.n_shared_state;
  int64_t& partial_numel = out.partial_numel;
  const bool adamw = cfg->optimizer == HDET_OPT_ADAMW;
  const bool sgd_momentum = cfg->optimizer == HDET_OPT_SGD && cfg->momentum != 0.0;
  for (int64_t k = 0; k < n_tensors; ++k) {
    const hdet_tensor& t = tensors[k];
    char where[64];
    snprintf(where, sizeof where, "hdet_create: tensor %lld: ", (long long)k);
    if (!t.param || !t.grad) return fail(nullptr, HDET_ERR_INVALID_ARG, std::string(where) + "param or grad is NULL");
    if (cfg->optimizer == HDET_OPT_ADAMW && (!t.exp_avg || !t.exp_avg_sq))
      return fail(nullptr, HDET_ERR_INVALID_ARG, std::string(where) + "AdamW needs exp_avg and exp_avg_sq");
    if (sgd_momentum && (!t.exp_avg || (n > 1 && t.state_stride < t.numel)))
      return fail(nullptr, HDET_ERR_INVALID_ARG, std::string(where) +
                  "SGD with momentum needs exp_avg (the momentum buffer) with one copy per replica");
    if (t.numel <= 0) return fail(nullptr, HDET_ERR_INVALID_ARG, std::string(where) + "numel must be > 0");
    if (t.group < 0 || t.group >= cfg->n_groups)
      return fail(nullptr, HDET_ERR_INVALID_ARG, std::string(where) + "group out of range");
    if (n > 1 && (t.param_stride < t.numel || (t.grad_stride != 0 && t.grad_stride < t.numel) ||
                  (adamw && t.state_stride != 0 && t.state_stride < t.numel)))
      return fail(nullptr, HDET_ERR_INVALID_ARG, std::string(where) + "a replica stride is smaller than numel");
    if (n > 1 && adamw && t.state_stride == 0) {
      if (t.grad_stride != 0 && cfg->grad_mode != HDET_GRAD_REPLICA_MEAN)
        return fail(nullptr, HDET_ERR_INVALID_ARG, std::string(where) +
                    "state_stride 0 (shared moments) needs a gradient common to all replicas");
      ++n_shared_state;
    }
    if (t.param_stride < 0 || t.grad_stride < 0 || t.state_stride < 0)
      return fail(nullptr, HDET_ERR_INVALID_ARG, std::string(where) + "negative stride");
    if (!aligned(t.param, 4) || !aligned(t.grad, gsz) || (t.exp_avg && !aligned(t.exp_avg, 4)) ||
        (t.exp_avg_sq && !aligned(t.exp_avg_sq, 4)) || (t.param_bf16 && !aligned(t.param_bf16, 2)))
      return fail(nullptr, HDET_ERR_ALIGN, std::string(where) + "pointer not aligned to its element type");
    const int64_t n_tiles_t = (t.numel + kTileElems - 1) / kTileElems;
    if (n_tiles_t > INT32_MAX || (int64_t)tiles.size() + n_tiles_t > INT32_MAX)
      return fail(nullptr, HDET_ERR_UNSUPPORTED, std::string(where) + "too many tiles");
    TensorDesc d{};
    d.param = static_cast<float*>(t.param);
    d.grad = t.grad;
    d.exp_avg = static_cast<float*>(t.exp_avg);
    d.exp_avg_sq = static_cast<float*>(t.exp_avg_sq);
    d.numel = t.numel;
    d.param_stride = t.param_stride;
    d.grad_stride = t.grad_stride;
    d.state_stride = t.state_stride;
    d.group = t.group;
    bool vec = aligned(t.param, 16) && aligned(t.grad, 4 * gsz) && t.param_stride % 4 == 0 && t.grad_stride % 4 == 0;
    if (cfg->optimizer == HDET_OPT_ADAMW)
      vec = vec && aligned(t.exp_avg, 16) && aligned(t.exp_avg_sq, 16) && t.state_stride % 4 == 0;
    if (sgd_momentum) vec = vec && aligned(t.exp_avg, 16) && t.state_stride % 4 == 0;
    if (t.param_bf16) vec = vec && aligned(t.param_bf16, 8);          // four bf16 values per store
    d.param_bf16 = static_cast<unsigned short*>(t.param_bf16);
    d.vec = vec ? kVecLoads : 0;
    // Bulk copies move whole tiles and need every array, the gradient included, on 16-byte boundaries.
    if (vec && adamw && aligned(t.grad, 16) && (t.grad_stride * (int64_t)gsz) % 16 == 0 &&
        (!t.param_bf16 || aligned(t.param_bf16, 16)))
      d.vec |= kVecBulk;
    d.partial_off = partial_numel;
    d.partial = nullptr;
    partial_numel += (t.numel + 3) / 4 * 4;
    descs.push_back(d);
    for (int64_t j = 0; j < n_tiles_t; ++j) tiles.push_back(Tile{(int)k, (int)j});
  }

  if (n_shared_state != 0 && n_shared_state != n_tensors)
    return fail(nullptr, HDET_ERR_UNSUPPORTED, "hdet_create: state_stride 0 must be used by all tensors or by none");

  return HDET_OK;
}

}  // namespace

namespace hdet {
void set_handleless_error(const char* msg) { g_create_error = msg ? msg : ""; }
}  // namespace hdet

extern "C" {

int hdet_create(const hdet_config* cfg, const hdet_tensor* tensors, int64_t n_tensors, hdet_handle* out) {
  TraceRange trace("hdet_create");
  if (out) *out = nullptr;
  if (!cfg || !out) return fail(nullptr, HDET_ERR_INVALID_ARG, "hdet_create: cfg and out must not be NULL");
  WorkPlan work;
  if (const int rc = plan_work(cfg, tensors, n_tensors, work)) return rc;
  const std::vector<TensorDesc>& descs = work.descs;
  const std::vector<Tile>& tiles = work.tiles;
  const int64_t n_shared_state = work.n_shared_state, partial_numel = work.partial_numel;
  const int n = cfg->n_replicas;
  const bool sharded = cfg->n_replicas_global != 0;
  const int n_global = sharded ? cfg->n_replicas_global : n;

  hdet_ctx* h = new (std::nothrow) hdet_ctx();
  if (!h) return fail(nullptr, HDET_ERR_INVALID_ARG, "hdet_create: out of host memory");
  h->cfg = *cfg;
  h->n_tensors = n_tensors;
  h->n_tiles = (int)tiles.size();
  h->shared_state = n_shared_state != 0;
  for (int64_t k = 0; k < n_tensors; ++k) h->total_numel += (double)tensors[k].numel;
  h->n_global = n_global;
  h->r_offset = sharded ? cfg->replica_offset : 0;
  h->partial_numel = partial_numel;
  h->tensors.assign(tensors, tensors + n_tensors);
  {   // upload runs: at most kUploadRuns runs of consecutive tensors holding about the same number of elements each
    constexpr int kUploadRuns = 8;
    const double per_run = h->total_numel / kUploadRuns;
    hdet_ctx::UploadRun run{0, 0, 0, 0};
    double in_run = 0.0;
    int tile_cursor = 0;
    for (int64_t k = 0; k < n_tensors; ++k) {
      const int n_tiles_k = (int)((tensors[k].numel + kTileElems - 1) / kTileElems);
      run.n_tensors += 1;
      run.n_tiles += n_tiles_k;
      in_run += (double)tensors[k].numel;
      tile_cursor += n_tiles_k;
      if ((in_run >= per_run && (int)h->upload_runs.size() < kUploadRuns - 1) || k == n_tensors - 1) {
        h->upload_runs.push_back(run);
        run = hdet_ctx::UploadRun{k + 1, 0, tile_cursor, 0};
        in_run = 0.0;
      }
    }
  }
  for (const TensorDesc& d : descs) h->partial_offsets.push_back(d.partial_off);
  spread_multipliers(n_global, cfg->alpha_lr, h->rho_lr);
  spread_multipliers(n_global, cfg->alpha_wd, h->rho_wd);
  for (int g = 0; g < HDET_MAX_GROUPS; ++g)
    for (int r = 0; r < HDET_MAX_REPLICAS; ++r) h->perm_lr[g][r] = h->perm_wd[g][r] = r;

  if (n_tensors > 0) {
    DeviceScope scope(cfg->device);
    cudaError_t e = scope.err;
    if (e == cudaSuccess) e = cudaMalloc(&h->d_tensors, descs.size() * sizeof(TensorDesc));
    if (e == cudaSuccess) e = cudaMalloc(&h->d_tiles, tiles.size() * sizeof(Tile));
    if (e == cudaSuccess) e = cudaMalloc(&h->d_status, sizeof(unsigned));
    if (e == cudaSuccess) e = cudaMalloc(&h->d_state, sizeof(DevState));
    if (e == cudaSuccess) e = cudaMemcpy(h->d_tensors, descs.data(), descs.size() * sizeof(TensorDesc), cudaMemcpyHostToDevice);
    if (e == cudaSuccess) e = cudaMemcpy(h->d_tiles, tiles.data(), tiles.size() * sizeof(Tile), cudaMemcpyHostToDevice);
    if (e == cudaSuccess) e = cudaMemset(h->d_status, 0, sizeof(unsigned));
    if (e == cudaSuccess)
      e = prepare_fanout(cfg->optimizer, cfg->grad_dtype, cfg->grad_mode == HDET_GRAD_REPLICA_MEAN, h->shared_state);
    if (e != cudaSuccess) {
      free_device(h);
      delete h;
      return fail_cuda(nullptr, "hdet_create", e);
    }
    // One CTA per tile, handed out by the hardware scheduler as SMs free up.  Measured on B200: a
    // persistent grid with a static tile stride runs ~10 % slower, because every SM then gets the same
    // number of tiles although the SMs do not all see the same memory bandwidth.
    h->grid_fanout = h->n_tiles;
    h->grid_converge = h->n_tiles;
  }
  *out = h;
  return HDET_OK;
}

int hdet_plan_tiles(const hdet_config* cfg, const hdet_tensor* tensors, int64_t n_tensors, int32_t* tile_tensor,
                    int32_t* tile_index, int64_t capacity, int64_t* n_tiles, int32_t* tensor_access,
                    int64_t* partial_offsets) {
  if (!cfg || !n_tiles) return fail(nullptr, HDET_ERR_INVALID_ARG, "hdet_plan_tiles: cfg and n_tiles must not be NULL");
  WorkPlan work;
  if (const int rc = plan_work(cfg, tensors, n_tensors, work)) return rc;
  *n_tiles = (int64_t)work.tiles.size();
  if (tile_tensor && tile_index) {
    if (capacity < *n_tiles) return fail(nullptr, HDET_ERR_INVALID_ARG, "hdet_plan_tiles: capacity is smaller than the tile count");
    for (size_t i = 0; i < work.tiles.size(); ++i) {
      tile_tensor[i] = work.tiles[i].tensor;
      tile_index[i] = work.tiles[i].tile;
    }
  }
  for (int64_t k = 0; k < n_tensors; ++k) {
    if (tensor_access) tensor_access[k] = work.descs[k].vec;
    if (partial_offsets) partial_offsets[k] = work.descs[k].partial_off;
  }
  return HDET_OK;
}

int hdet_set_schedule(hdet_handle h, const hdet_schedule* s) {
  TraceRange trace("hdet_set_schedule");
  if (!h) return HDET_ERR_INVALID_ARG;
  if (!s || !s->max_lr) return fail(h, HDET_ERR_INVALID_ARG, "hdet_set_schedule: sched and max_lr must not be NULL");
  if (h->device_mode)
    return fail(h, HDET_ERR_STATE, "hdet_set_schedule: the scalar state lives on the device; hdet_get_state then "
                                   "hdet_set_state returns the handle to host stepping, where the schedule can be replaced");
  if (s->kind < HDET_SCHED_CONSTANT || s->kind > HDET_SCHED_ONECYCLE_LINEAR)
    return fail(h, HDET_ERR_INVALID_ARG, "hdet_set_schedule: unknown kind");
  if (s->total_steps < 1) return fail(h, HDET_ERR_INVALID_ARG, "hdet_set_schedule: total_steps must be >= 1");
  if (s->kind != HDET_SCHED_CONSTANT) {
    const double knee = s->pct_start * (double)s->total_steps;
    if (!(knee > 1.0) || !(s->pct_start < 1.0))
      return fail(h, HDET_ERR_INVALID_ARG, "hdet_set_schedule: need 1 < pct_start*total_steps and pct_start < 1");
    if (!(s->div_factor > 0.0) || !(s->final_div_factor > 0.0))
      return fail(h, HDET_ERR_INVALID_ARG, "hdet_set_schedule: div_factor and final_div_factor must be > 0");
  }
  if (s->autolr) {
    if (!(s->sigma > 0.0)) return fail(h, HDET_ERR_INVALID_ARG, "hdet_set_schedule: sigma must be > 0");
    if (!(s->f_div > 0.0) || !(s->f_final > 0.0))
      return fail(h, HDET_ERR_INVALID_ARG, "hdet_set_schedule: f_div and f_final must be > 0");
    if (s->warmup_steps < 0) return fail(h, HDET_ERR_INVALID_ARG, "hdet_set_schedule: warmup_steps must be >= 0");
  }
  for (int g = 0; g < h->cfg.n_groups; ++g) {
    if (!std::isfinite(s->max_lr[g])) return fail(h, HDET_ERR_INVALID_ARG, "hdet_set_schedule: max_lr is not finite");
    if (s->weight_decay && !std::isfinite(s->weight_decay[g]))
      return fail(h, HDET_ERR_INVALID_ARG, "hdet_set_schedule: weight_decay is not finite");
  }
  h->sched = *s;
  for (int g = 0; g < h->cfg.n_groups; ++g) {
    h->max_lr[g] = s->max_lr[g];
    h->weight_decay[g] = s->weight_decay ? s->weight_decay[g] : 0.0;
    h->wd_base[g] = h->weight_decay[g];
  }
  h->sched.max_lr = nullptr;
  h->sched.weight_decay = nullptr;
  h->has_schedule = true;
  return HDET_OK;
}

// One loop body of Algorithm 1 with host scalars.  `partial` != NULL: a round's last update writes the
// sums over the local replicas to `partial` instead of the mean (replica axis sharded over GPUs).
// Enqueues the host-to-device copies of tensors [first, first + count) on `st` (one strided copy per tensor).
static cudaError_t upload_gradients(hdet_ctx* h, const void* const* host_grads, int64_t first, int64_t count, cudaStream_t st) {
  const size_t gsz = h->cfg.grad_dtype == HDET_DTYPE_BF16 ? 2 : 4;
  for (int64_t k = first; k < first + count; ++k) {
    const hdet_tensor& t = h->tensors[k];
    const size_t row = (size_t)t.numel * gsz;
    cudaError_t e;
    if (t.grad_stride == 0 || h->cfg.n_replicas == 1) {
      e = cudaMemcpyAsync(t.grad, host_grads[k], row, cudaMemcpyHostToDevice, st);
    } else {   // N rows of one tensor, replica stride as pitch on both sides
      const size_t pitch = (size_t)t.grad_stride * gsz;
      e = cudaMemcpy2DAsync(t.grad, pitch, host_grads[k], pitch, row, (size_t)h->cfg.n_replicas, cudaMemcpyHostToDevice, st);
    }
    if (e != cudaSuccess) return e;
  }
  return cudaSuccess;
}

// `host_grads` != NULL: the gradients are uploaded from host memory first, run by run, each run's tiles updated as
// soon as its copies have landed (hdet_step_host_grads).
static int step_impl(hdet_handle h, const double* step_losses, bool sharded_call, float* partial, void* stream,
                     int32_t* did_converge, const void* const* host_grads = nullptr) {
  if (!h) return HDET_ERR_INVALID_ARG;
  if (did_converge) *did_converge = 0;
  if (!h->has_schedule) return fail(h, HDET_ERR_STATE, "hdet_step: call hdet_set_schedule first");
  if (h->device_mode)
    return fail(h, HDET_ERR_STATE, "hdet_step: the handle steps on the device (hdet_step_device); hdet_set_state returns it to host stepping");
  if (!sharded_call && h->n_global != h->cfg.n_replicas)
    return fail(h, HDET_ERR_STATE, "hdet_step: this handle holds a shard of the replica axis; use hdet_step_sharded and hdet_apply_mean");
  const int n = h->cfg.n_replicas, n_all = h->n_global, off = h->r_offset, G = h->cfg.n_groups;
  compute_tables(h);
  const int64_t t = h->step + 1;
  const bool ends_round = (t % h->cfg.sync_interval) == 0;

  if (h->n_tiles > 0) {
    StepScalars s{};
    const bool adam = h->cfg.optimizer == HDET_OPT_ADAMW;
    double bc1 = 1.0, bc2 = 1.0;
    if (adam) {
      bc1 = 1.0 - std::pow(h->cfg.beta1, (double)t);
      bc2 = 1.0 - std::pow(h->cfg.beta2, (double)t);
    }
    for (int g = 0; g < G; ++g)
      for (int r = 0; r < n; ++r) {
        const double lr = h->lr[g][off + r], wd = h->wd[g][off + r];   // local replica r is global replica off + r
        s.lr_wd[g][r] = (float)(adam ? lr * wd : wd);
        s.step[g][r] = (float)(adam ? lr / bc1 : lr);
      }
    s.one_minus_beta1 = (float)(1.0 - h->cfg.beta1);
    s.one_minus_beta2 = (float)(1.0 - h->cfg.beta2);
    s.rsqrt_bc2 = (float)(1.0 / std::sqrt(bc2));
    s.eps = (float)h->cfg.eps;
    s.momentum = adam ? 0.0f : (float)h->cfg.momentum;
    s.inv_n = 1.0 / (double)n;
    s.n_replicas = n;

    DeviceScope scope(h->cfg.device);
    if (scope.err != cudaSuccess) return fail_cuda(h, "hdet_step", scope.err);
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const bool fuse = ends_round && (h->cfg.fuse_converge || partial);
    LaunchPlan plan{h->d_tensors, h->d_tiles, h->n_tiles, h->grid_fanout, h->d_status, nullptr,
                    ends_round ? partial : nullptr};
    const bool sgd_momentum = h->cfg.optimizer == HDET_OPT_SGD && h->cfg.momentum != 0.0;
    const bool grad_mean = h->cfg.grad_mode == HDET_GRAD_REPLICA_MEAN;
    cudaError_t e = cudaSuccess;
    if (!host_grads) {
      e = launch_fanout(h->cfg.optimizer, sgd_momentum, h->cfg.grad_dtype, fuse, grad_mean, h->shared_state, plan, s, st);
      if (e != cudaSuccess) return fail_cuda(h, "hdet_step: fan-out launch", e);
      ++h->launches;
    } else {
      // Copies run on the handle's own stream, ordered after everything already enqueued on the caller's stream;
      // the caller's stream waits for each run's copies and then updates that run's tiles.
      if (!h->copy_stream) {
        e = cudaStreamCreateWithFlags(&h->copy_stream, cudaStreamNonBlocking);
        if (e == cudaSuccess) e = cudaEventCreateWithFlags(&h->upload_begin, cudaEventDisableTiming);
        for (size_t c = 0; e == cudaSuccess && c < h->upload_runs.size(); ++c) {
          cudaEvent_t ev = nullptr;
          e = cudaEventCreateWithFlags(&ev, cudaEventDisableTiming);
          if (e == cudaSuccess) h->upload_done.push_back(ev);
        }
        if (e != cudaSuccess) return fail_cuda(h, "hdet_step_host_grads: stream and events", e);
      }
      e = cudaEventRecord(h->upload_begin, st);
      if (e == cudaSuccess) e = cudaStreamWaitEvent(h->copy_stream, h->upload_begin, 0);
      for (size_t c = 0; e == cudaSuccess && c < h->upload_runs.size(); ++c) {
        const hdet_ctx::UploadRun& run = h->upload_runs[c];
        e = upload_gradients(h, host_grads, run.first_tensor, run.n_tensors, h->copy_stream);
        if (e == cudaSuccess) e = cudaEventRecord(h->upload_done[c], h->copy_stream);
        if (e == cudaSuccess) e = cudaStreamWaitEvent(st, h->upload_done[c], 0);
        if (e != cudaSuccess) break;
        LaunchPlan part = plan;
        part.tiles = h->d_tiles + run.first_tile;
        part.n_tiles = run.n_tiles;
        part.grid = run.n_tiles;
        e = launch_fanout(h->cfg.optimizer, sgd_momentum, h->cfg.grad_dtype, fuse, grad_mean, h->shared_state, part, s, st);
        if (e == cudaSuccess) ++h->launches;
      }
      if (e != cudaSuccess) return fail_cuda(h, "hdet_step_host_grads: upload and update", e);
    }
    if (ends_round && !fuse) {
      plan.grid = h->grid_converge;
      e = launch_converge(plan, n, st);
      if (e != cudaSuccess) return fail_cuda(h, "hdet_step: converge launch", e);
      ++h->launches;
    }
  }

  if (step_losses)
    for (int r = 0; r < n_all; ++r) h->loss_acc[r] += step_losses[r];
  ++h->n_acc;
  h->step = t;
  h->round_ended = false;
  if (ends_round) {
    for (int r = 0; r < n_all; ++r) {
      h->loss_round[r] = h->loss_acc[r] / (double)h->n_acc;
      h->loss_acc[r] = 0.0;
    }
    h->n_acc = 0;
    h->round_ended = true;
    if (did_converge) *did_converge = 1;
  }
  return HDET_OK;
}

int hdet_step(hdet_handle h, const double* step_losses, void* stream, int32_t* did_converge) {
  TraceRange trace("hdet_step");
  return step_impl(h, step_losses, false, nullptr, stream, did_converge);
}

int hdet_step_host_grads(hdet_handle h, const void* const* host_grads, const double* step_losses, void* stream,
                         int32_t* did_converge) {
  TraceRange trace("hdet_step_host_grads");
  if (!h) return HDET_ERR_INVALID_ARG;
  if (did_converge) *did_converge = 0;
  if (h->n_tensors > 0 && !host_grads) return fail(h, HDET_ERR_INVALID_ARG, "hdet_step_host_grads: host_grads is NULL");
  for (int64_t k = 0; k < h->n_tensors; ++k)
    if (!host_grads[k]) return fail(h, HDET_ERR_INVALID_ARG, "hdet_step_host_grads: a host gradient pointer is NULL");
  return step_impl(h, step_losses, false, nullptr, stream, did_converge, h->n_tensors > 0 ? host_grads : nullptr);
}

int hdet_step_sharded(hdet_handle h, const double* step_losses, void* d_partial, void* stream, int32_t* did_converge) {
  TraceRange trace("hdet_step_sharded");
  if (!h) return HDET_ERR_INVALID_ARG;
  if (h->n_tiles > 0 && !d_partial) return fail(h, HDET_ERR_INVALID_ARG, "hdet_step_sharded: d_partial is NULL");
  if (d_partial && !aligned(d_partial, 16))
    return fail(h, HDET_ERR_ALIGN, "hdet_step_sharded: d_partial must be 16-byte aligned");
  return step_impl(h, step_losses, true, static_cast<float*>(d_partial), stream, did_converge);
}

int hdet_apply_mean(hdet_handle h, const void* d_sum, void* stream) {
  TraceRange trace("hdet_apply_mean");
  if (!h) return HDET_ERR_INVALID_ARG;
  if (h->n_tiles == 0) return HDET_OK;
  if (!d_sum || !aligned(d_sum, 16)) return fail(h, HDET_ERR_INVALID_ARG, "hdet_apply_mean: d_sum is NULL or not 16-byte aligned");
  DeviceScope scope(h->cfg.device);
  if (scope.err != cudaSuccess) return fail_cuda(h, "hdet_apply_mean", scope.err);
  LaunchPlan plan{h->d_tensors, h->d_tiles, h->n_tiles, h->grid_converge, h->d_status, nullptr,
                  const_cast<float*>(static_cast<const float*>(d_sum))};
  cudaError_t e = launch_apply_mean(plan, h->cfg.n_replicas, 1.0 / (double)h->n_global, static_cast<cudaStream_t>(stream));
  if (e != cudaSuccess) return fail_cuda(h, "hdet_apply_mean: launch", e);
  ++h->launches;
  return HDET_OK;
}

int hdet_apply_mean_peers(hdet_handle h, const void* const* d_partials, int32_t n_buffers, void* stream) {
  if (!h) return HDET_ERR_INVALID_ARG;
  TraceRange trace("hdet_apply_mean_peers");
  if (h->n_tiles == 0) return HDET_OK;
  if (!d_partials || n_buffers < 1 || n_buffers > HDET_MAX_REPLICAS)
    return fail(h, HDET_ERR_INVALID_ARG, "hdet_apply_mean_peers: need 1 .. 32 staging buffers");
  const float* bufs[HDET_MAX_REPLICAS];
  for (int b = 0; b < n_buffers; ++b) {
    if (!d_partials[b] || !aligned(d_partials[b], 16))
      return fail(h, HDET_ERR_INVALID_ARG, "hdet_apply_mean_peers: a staging buffer is NULL or not 16-byte aligned");
    bufs[b] = static_cast<const float*>(d_partials[b]);
  }
  DeviceScope scope(h->cfg.device);
  if (scope.err != cudaSuccess) return fail_cuda(h, "hdet_apply_mean_peers", scope.err);
  LaunchPlan plan{h->d_tensors, h->d_tiles, h->n_tiles, h->grid_converge, h->d_status, nullptr, nullptr};
  cudaError_t e = launch_apply_mean_peers(plan, bufs, n_buffers, h->cfg.n_replicas, 1.0 / (double)h->n_global,
                                          static_cast<cudaStream_t>(stream));
  if (e != cudaSuccess) return fail_cuda(h, "hdet_apply_mean_peers: launch", e);
  ++h->launches;
  return HDET_OK;
}

int hdet_partial_layout(hdet_handle h, int64_t* offsets, int64_t n_offsets, int64_t* total_numel) {
  if (!h) return HDET_ERR_INVALID_ARG;
  if (offsets && n_offsets != h->n_tensors)
    return fail(h, HDET_ERR_INVALID_ARG, "hdet_partial_layout: n_offsets must equal the number of tensors");
  if (offsets)
    for (int64_t k = 0; k < h->n_tensors; ++k) offsets[k] = h->partial_offsets[k];
  if (total_numel) *total_numel = h->partial_numel;
  return HDET_OK;
}

int hdet_step_device(hdet_handle h, const void* d_step_losses, int32_t loss_dtype, void* stream, int32_t* did_converge) {
  TraceRange trace("hdet_step_device");
  if (!h) return HDET_ERR_INVALID_ARG;
  if (did_converge) *did_converge = 0;
  if (!h->has_schedule) return fail(h, HDET_ERR_STATE, "hdet_step_device: call hdet_set_schedule first");
  if (h->n_global != h->cfg.n_replicas)
    return fail(h, HDET_ERR_UNSUPPORTED, "hdet_step_device: not available when the replica axis is sharded over GPUs");
  if (h->n_tiles == 0 || !h->d_state)
    return fail(h, HDET_ERR_UNSUPPORTED, "hdet_step_device: the handle has no tensors, hence no device state");
  if (d_step_losses && loss_dtype != HDET_DTYPE_F32 && loss_dtype != HDET_DTYPE_F64)
    return fail(h, HDET_ERR_INVALID_ARG, "hdet_step_device: losses must be fp32 or fp64");
  DeviceScope scope(h->cfg.device);
  if (scope.err != cudaSuccess) return fail_cuda(h, "hdet_step_device", scope.err);
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  if (!h->device_mode) {
    // First device-resident step: the host state becomes the device state (one blocking copy).
    hdet_state snapshot;
    export_state(h, &snapshot);
    cudaError_t e = cudaMemcpy(&h->d_state->st, &snapshot, sizeof snapshot, cudaMemcpyHostToDevice);
    if (e != cudaSuccess) return fail_cuda(h, "hdet_step_device: state upload", e);
    h->device_mode = true;
  }
  const int n = h->cfg.n_replicas;
  const int64_t t = h->step + 1;
  const bool ends_round = (t % h->cfg.sync_interval) == 0;
  const DevConst c = device_constants(h);
  cudaError_t e = launch_device_scalars(h->d_state, c, d_step_losses, loss_dtype == HDET_DTYPE_F64, st);
  if (e != cudaSuccess) return fail_cuda(h, "hdet_step_device: scalar kernel launch", e);
  ++h->launches;
  const bool fuse = ends_round && h->cfg.fuse_converge;
  LaunchPlan plan{h->d_tensors, h->d_tiles, h->n_tiles, h->grid_fanout, h->d_status, &h->d_state->scal, nullptr};
  const StepScalars unused{};
  e = launch_fanout(h->cfg.optimizer, h->cfg.optimizer == HDET_OPT_SGD && h->cfg.momentum != 0.0, h->cfg.grad_dtype, fuse,
                                  h->cfg.grad_mode == HDET_GRAD_REPLICA_MEAN,
                    h->shared_state, plan, unused, st);
  if (e != cudaSuccess) return fail_cuda(h, "hdet_step_device: fan-out launch", e);
  ++h->launches;
  if (ends_round && !fuse) {
    plan.grid = h->grid_converge;
    e = launch_converge(plan, n, st);
    if (e != cudaSuccess) return fail_cuda(h, "hdet_step_device: converge launch", e);
    ++h->launches;
  }
  // Host shadow of what is known without reading the device: the step count and the round position.
  h->step = t;
  ++h->n_acc;
  h->round_ended = false;
  if (ends_round) {
    e = launch_device_round_end(h->d_state, c, st);
    if (e != cudaSuccess) return fail_cuda(h, "hdet_step_device: controller launch", e);
    ++h->launches;
    h->n_acc = 0;
    if (h->sched.autolr && t >= h->sched.warmup_steps) h->fired = true;
    if (did_converge) *did_converge = 1;
  }
  return HDET_OK;
}

int hdet_warm_init(hdet_handle h, double nu, uint64_t seed, void* stream) {
  TraceRange trace("hdet_warm_init");
  if (!h) return HDET_ERR_INVALID_ARG;
  if (!(nu >= 0.0) || !std::isfinite(nu)) return fail(h, HDET_ERR_INVALID_ARG, "hdet_warm_init: nu must be finite and >= 0");
  if (h->n_tiles == 0) return HDET_OK;
  DeviceScope scope(h->cfg.device);
  if (scope.err != cudaSuccess) return fail_cuda(h, "hdet_warm_init", scope.err);
  if (!h->d_warm) {
    cudaError_t e = cudaMalloc(&h->d_warm, sizeof(double) * ((size_t)h->n_tiles + 1));
    if (e != cudaSuccess) return fail_cuda(h, "hdet_warm_init: scratch allocation", e);
  }
  LaunchPlan plan{h->d_tensors, h->d_tiles, h->n_tiles, h->grid_converge, h->d_status, nullptr};
  cudaError_t e = launch_warm_init(plan, h->cfg.n_replicas, h->r_offset, nu, h->total_numel, seed, h->d_warm,
                                   static_cast<cudaStream_t>(stream));
  if (e != cudaSuccess) return fail_cuda(h, "hdet_warm_init: launch", e);
  h->launches += 3;
  return HDET_OK;
}

int hdet_converge(hdet_handle h, void* stream) {
  TraceRange trace("hdet_converge");
  if (!h) return HDET_ERR_INVALID_ARG;
  if (h->n_global != h->cfg.n_replicas)
    return fail(h, HDET_ERR_UNSUPPORTED, "hdet_converge: this handle holds a shard of the replica axis; use hdet_step_sharded and hdet_apply_mean");
  if (h->n_tiles == 0) return HDET_OK;
  DeviceScope scope(h->cfg.device);
  if (scope.err != cudaSuccess) return fail_cuda(h, "hdet_converge", scope.err);
  LaunchPlan plan{h->d_tensors, h->d_tiles, h->n_tiles, h->grid_converge, h->d_status, nullptr};
  cudaError_t e = launch_converge(plan, h->cfg.n_replicas, static_cast<cudaStream_t>(stream));
  if (e != cudaSuccess) return fail_cuda(h, "hdet_converge: launch", e);
  ++h->launches;
  return HDET_OK;
}

int hdet_autolr_update(hdet_handle h, const double* round_losses, void* /*stream*/) {
  TraceRange trace("hdet_autolr_update");
  if (!h) return HDET_ERR_INVALID_ARG;
  if (!h->has_schedule) return fail(h, HDET_ERR_STATE, "hdet_autolr_update: call hdet_set_schedule first");
  if (h->device_mode)
    return fail(h, HDET_ERR_STATE, "hdet_autolr_update: with hdet_step_device the controller already runs on the device");
  if (!h->round_ended)
    return fail(h, HDET_ERR_STATE, "hdet_autolr_update: the last hdet_step did not end a round (or the update already ran)");
  h->round_ended = false;
  if (!h->sched.autolr || h->step < h->sched.warmup_steps) return HDET_OK;
  const int n = h->n_global, G = h->cfg.n_groups;
  const double* L = round_losses ? round_losses : h->loss_round;
  for (int r = 0; r < n; ++r)
    if (!std::isfinite(L[r])) {
      h->round_ended = true;
      return fail(h, HDET_ERR_INVALID_ARG, "hdet_autolr_update: a round loss is not finite");
    }
  if (round_losses)
    for (int r = 0; r < n; ++r) h->loss_round[r] = round_losses[r];
  const double gamma = decay_gamma(h->sched.f_div, h->sched.f_final, h->sched.total_steps, h->sched.warmup_steps,
                                   h->cfg.sync_interval);
  softmax_weights(n, L, h->sched.sigma, h->weights);                       // Eq. 4
  for (int g = 0; g < G; ++g) {
    double weighted = 0.0, plain = 0.0;
    for (int r = 0; r < n; ++r) {
      weighted += h->weights[r] * h->lr[g][r];                             // Eq. 5
      plain += h->lr[g][r];
    }
    plain /= n;
    h->delta[g] = weighted - plain;                                        // Eq. 6
    h->velocity[g] = h->sched.beta * h->velocity[g] + (1.0 - h->sched.beta) * h->delta[g];   // Eq. 7
    h->ctrl_base[g] = plain * (1.0 - gamma) + h->velocity[g] * h->sched.lambda;
    if (h->sched.auto_wd) {   // Remark 1: the same update on the weight decays of the last step, without decay
      double w_wd = 0.0, p_wd = 0.0;
      for (int r = 0; r < n; ++r) {
        w_wd += h->weights[r] * h->wd[g][r];
        p_wd += h->wd[g][r];
      }
      p_wd /= n;
      h->wd_delta[g] = w_wd - p_wd;
      h->wd_velocity[g] = h->sched.beta * h->wd_velocity[g] + (1.0 - h->sched.beta) * h->wd_delta[g];
      h->wd_base[g] = p_wd + h->wd_velocity[g] * h->sched.lambda;
    }
  }
  h->fired = true;
  if (h->cfg.reshuffle) {                                                   // Eq. 9
    const uint64_t sync_index = (uint64_t)(h->step / h->cfg.sync_interval);
    for (int g = 0; g < G; ++g) {
      draw_permutation(h->cfg.seed, sync_index, 2ull * g, n, h->perm_lr[g]);
      draw_permutation(h->cfg.seed, sync_index, 2ull * g + 1, n, h->perm_wd[g]);
    }
  }
  return HDET_OK;
}

int hdet_get_state(hdet_handle h, hdet_state* out) {
  TraceRange trace("hdet_get_state");
  if (!h) return HDET_ERR_INVALID_ARG;
  if (!out) return fail(h, HDET_ERR_INVALID_ARG, "hdet_get_state: out is NULL");
  if (h->device_mode) {
    // The device copy is authoritative: read it back (blocking) and refresh the host fields from it.
    DeviceScope scope(h->cfg.device);
    cudaError_t e = scope.err;
    hdet_state dev;
    if (e == cudaSuccess) e = cudaMemcpy(&dev, &h->d_state->st, sizeof dev, cudaMemcpyDeviceToHost);
    if (e != cudaSuccess) return fail_cuda(h, "hdet_get_state: state read-back", e);
    import_state(h, &dev);
  }
  export_state(h, out);
  if (h->d_status) {
    DeviceScope scope(h->cfg.device);
    cudaError_t e = scope.err;
    unsigned word = 0;
    if (e == cudaSuccess) e = cudaMemcpy(&word, h->d_status, sizeof word, cudaMemcpyDeviceToHost);
    if (e != cudaSuccess) return fail_cuda(h, "hdet_get_state", e);
    out->device_status = word;
    if (word & 2u) return fail(h, HDET_ERR_TIMEOUT, "a kernel's bounded wait for its own bulk copies ran out; a tile was left unfinished");
    if (word & 1u) return fail(h, HDET_ERR_NONFINITE, "a kernel produced a non-finite parameter");
  }
  return HDET_OK;
}

int hdet_set_state(hdet_handle h, const hdet_state* in) {
  TraceRange trace("hdet_set_state");
  if (!h) return HDET_ERR_INVALID_ARG;
  if (!in) return fail(h, HDET_ERR_INVALID_ARG, "hdet_set_state: in is NULL");
  if (in->step < 0 || in->n_acc < 0) return fail(h, HDET_ERR_INVALID_ARG, "hdet_set_state: negative step or n_acc");
  const int n = h->n_global, G = h->cfg.n_groups;
  for (int g = 0; g < G; ++g)
    if (!is_permutation(in->perm_lr[g], n) || !is_permutation(in->perm_wd[g], n))
      return fail(h, HDET_ERR_INVALID_ARG, "hdet_set_state: a permutation array is not a permutation of 0..N-1");
  h->step = in->step;
  h->n_acc = in->n_acc;
  h->fired = in->fired != 0;
  h->round_ended = in->round_ended != 0;
  std::memcpy(h->ctrl_base, in->ctrl_base, sizeof h->ctrl_base);
  std::memcpy(h->velocity, in->velocity, sizeof h->velocity);
  std::memcpy(h->lr, in->lr, sizeof h->lr);  // rates of the last update: Eq. 5 needs them if a round just ended
  for (int g = 0; g < G; ++g) {
    std::memcpy(h->perm_lr[g], in->perm_lr[g], sizeof(int32_t) * n);
    std::memcpy(h->perm_wd[g], in->perm_wd[g], sizeof(int32_t) * n);
  }
  std::memcpy(h->loss_acc, in->loss_acc, sizeof h->loss_acc);
  std::memcpy(h->loss_round, in->loss_round, sizeof h->loss_round);
  std::memcpy(h->wd_base, in->wd_base, sizeof h->wd_base);
  std::memcpy(h->wd_velocity, in->wd_velocity, sizeof h->wd_velocity);
  std::memcpy(h->wd[0], in->wd[0], sizeof h->wd);  // decays of the last update: the Remark 1 channel needs them at a round end
  h->device_mode = false;   // the host copy is authoritative again; hdet_step_device uploads it anew
  if (h->d_status) {
    DeviceScope scope(h->cfg.device);
    cudaError_t e = scope.err;
    if (e == cudaSuccess) e = cudaDeviceSynchronize();   // earlier device-resident steps must not outlive the state they use
    if (e == cudaSuccess) e = cudaMemset(h->d_status, 0, sizeof(unsigned));
    if (e != cudaSuccess) return fail_cuda(h, "hdet_set_state", e);
  }
  return HDET_OK;
}

int hdet_selftest_bounded_wait(hdet_handle h, void* stream) {
  if (!h) return HDET_ERR_INVALID_ARG;
  TraceRange trace("hdet_selftest_bounded_wait");
  if (!h->d_status) return fail(h, HDET_ERR_UNSUPPORTED, "hdet_selftest_bounded_wait: the handle has no tensors, hence no device");
  DeviceScope scope(h->cfg.device);
  if (scope.err != cudaSuccess) return fail_cuda(h, "hdet_selftest_bounded_wait", scope.err);
  const cudaError_t e = launch_bounded_wait_probe(h->d_status, static_cast<cudaStream_t>(stream));
  if (e != cudaSuccess) return fail_cuda(h, "hdet_selftest_bounded_wait: launch", e);
  ++h->launches;
  return HDET_OK;
}

int hdet_destroy(hdet_handle h) {
  TraceRange trace("hdet_destroy");
  if (!h) return HDET_OK;
  if (h->d_tensors || h->d_tiles || h->d_status || h->d_state || h->d_warm || h->copy_stream) {
    DeviceScope scope(h->cfg.device);
    free_device(h);
  }
  delete h;
  return HDET_OK;
}

const char* hdet_last_error(hdet_handle h) { return h ? h->error.c_str() : g_create_error.c_str(); }

int64_t hdet_kernel_launches(hdet_handle h) { return h ? h->launches : 0; }

}  // extern "C"
