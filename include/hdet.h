/*
 * hdet.h -- C ABI of libhdet: the per-step hot path of Hyperparameter-Divergent
 * Ensemble Training (HDET, arXiv 2604.24708) with the N replicas stacked on one GPU.
 *
 * One handle drives Algorithm 1's loop body for a list of parameter tensors:
 *
 *   hdet_create        validate the tensor list, build the device work table
 *   hdet_set_schedule  base schedule (Algorithm 1, Require) and controller constants
 *   hdet_step          spread (Eq. 1) x base rate -> fused fan-out update (Eq. 2 /
 *                      Adam, Section 4.1); on the last update of a round the converge
 *                      mean (Eq. 3) is formed in the same kernel
 *   hdet_converge      stand-alone converge (Eq. 3)
 *   hdet_autolr_update controller (Eq. 4 - Eq. 9) after a converge
 *   hdet_get_state / hdet_set_state   scalars for logging and resume
 *   hdet_destroy
 * and, around that core:
 *   hdet_step_device       the same step with the scalar state and the controller on the device
 *   hdet_step_host_grads   the same step with the gradients uploaded from host memory first
 *   hdet_step_sharded / hdet_apply_mean / hdet_apply_mean_peers / hdet_partial_layout   replica axis split over GPUs
 *   hdet_warm_init         warm noisy initialisation (Eq. 10)
 *   hdet_converge_static   allocation-free variant of hdet_converge
 *   hdet_plan_tiles        host-only view of the work plan (tests, tools)
 *   hdet_selftest_bounded_wait   makes a kernel's bounded wait run out, to show the timeout status
 *
 * Conventions
 *   - Every tensor pointer is a DEVICE pointer owned by the caller; it must stay
 *     valid until hdet_destroy.  Scalar arrays (losses, max_lr, ...) are HOST pointers
 *     read during the call only.
 *   - Layout: replica r of a tensor starts at base + r * stride (strides in elements).
 *     Parameters and Adam moments are fp32.  Gradients are fp32 or bf16.
 *   - All kernels are launched on the caller's stream (a cudaStream_t passed as
 *     void*; NULL = the legacy default stream) and the calls return without
 *     synchronising unless stated otherwise.  Launches of one handle must be ordered
 *     on the device by the caller (same stream, or events).
 *   - No function throws or aborts; each returns an hdet_status.  hdet_last_error
 *     gives a text for the last failure on a handle.
 *   - The library owns only its work table, a status word and a small state block on the
 *     device, and the host controller state.  hdet_step / hdet_step_device / hdet_converge /
 *     hdet_autolr_update allocate nothing.
 *   - There is no CPU fallback: a handle with tensors needs a CUDA device.  A handle
 *     created with n_tensors == 0 touches no device and runs only the scalar part
 *     (schedule, spread, controller), which is what host-side tests use.
 */
#ifndef HDET_H_
#define HDET_H_

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#if defined(__GNUC__)
#define HDET_API __attribute__((visibility("default")))
#else
#define HDET_API
#endif

#define HDET_MAX_REPLICAS 32
#define HDET_MAX_GROUPS 8

typedef enum {
  HDET_OK = 0,
  HDET_ERR_INVALID_ARG = 1, /* NULL pointer, value out of range                          */
  HDET_ERR_STATE = 2,       /* call out of order (no schedule set, no round just ended)  */
  HDET_ERR_ALIGN = 3,       /* a pointer is not aligned to its element type              */
  HDET_ERR_UNSUPPORTED = 4, /* a valid request this build does not implement             */
  HDET_ERR_CUDA = 5,        /* a CUDA runtime call failed; see hdet_last_error           */
  HDET_ERR_NONFINITE = 6,   /* a kernel produced a non-finite parameter (sticky)         */
  HDET_ERR_TIMEOUT = 7      /* a kernel gave up waiting for one of its own bulk copies and
                               left a tile unfinished (sticky; parameters are then undefined) */
} hdet_status;

enum { HDET_OPT_SGD = 0, HDET_OPT_ADAMW = 1 };
enum { HDET_DTYPE_F32 = 0, HDET_DTYPE_BF16 = 1, HDET_DTYPE_F64 = 2 /* losses only */ };
enum { HDET_GRAD_AS_GIVEN = 0, HDET_GRAD_REPLICA_MEAN = 1 };
enum { HDET_SCHED_CONSTANT = 0, HDET_SCHED_ONECYCLE_COS = 1, HDET_SCHED_ONECYCLE_LINEAR = 2 };

typedef struct hdet_ctx* hdet_handle;

/* One parameter tensor with its N replicas.  Device pointers, caller-owned. */
typedef struct {
  void* param;          /* fp32 [N] x numel, replica stride param_stride                  */
  void* grad;           /* fp32 or bf16 (hdet_config.grad_dtype), replica stride grad_stride */
  void* exp_avg;        /* fp32 Adam first moment (SGD with momentum: the momentum buffer),
                           replica stride state_stride; NULL for plain SGD               */
  void* exp_avg_sq;     /* fp32 Adam second moment, replica stride state_stride; NULL for SGD */
  int64_t numel;        /* elements per replica, > 0                                      */
  int64_t param_stride; /* elements between replicas of param (>= numel when N > 1)       */
  int64_t grad_stride;  /* elements between replicas of grad; 0 = one gradient shared by
                           every replica (the all-reduced gradient of Eq. 2)              */
  int64_t state_stride; /* elements between replicas of both moments; 0 = ONE pair of moments
                           for all replicas, allowed only when every replica sees the same
                           gradient (grad_stride 0, or grad_mode HDET_GRAD_REPLICA_MEAN), and
                           then required of every tensor of the handle                    */
  int32_t group;        /* optimizer group, 0 .. n_groups-1                               */
  int32_t reserved;     /* set to 0                                                       */
  void* param_bf16;     /* optional bf16 [numel] (ONE copy, not one per replica), or NULL: every
                           converge (fused into a step, hdet_converge, hdet_apply_mean) also
                           writes the averaged parameters of Eq. 3 here, each the stored fp32
                           mean rounded to nearest even -- the weights the next forward pass of
                           Algorithm 1 reads in mixed precision; costs 2 bytes per parameter.
                           Updates that do not converge leave it untouched.                */
} hdet_tensor;
/* Alignment: pointers must be aligned to their element type (4 bytes fp32, 2 bytes
 * bf16) or hdet_create returns HDET_ERR_ALIGN.  A tensor whose pointers are 16-byte
 * aligned (gradients: 8 bytes for bf16, 16 for fp32) and whose strides are multiples of
 * 4 elements takes the vectorised path; any other tensor is processed correctly by
 * scalar loads.  param_bf16, when given, must be 2-byte aligned; it joins the vectorised path
 * when 8-byte aligned and the bulk-copy path (AdamW) when 16-byte aligned. */

typedef struct {
  int32_t n_replicas;    /* N of Eq. 1, 1 .. HDET_MAX_REPLICAS                            */
  int32_t n_groups;      /* optimizer parameter groups (Section 3.4), 1 .. HDET_MAX_GROUPS */
  int32_t optimizer;     /* HDET_OPT_SGD (Eq. 2) or HDET_OPT_ADAMW (Section 4.1)          */
  int32_t grad_dtype;    /* HDET_DTYPE_F32 or HDET_DTYPE_BF16                             */
  double beta1, beta2, eps; /* Adam constants (ignored by SGD)                            */
  double momentum;       /* SGD momentum mu, 0 <= mu < 1.  0 is Eq. 2.  mu > 0 (an extension, Eq. 2
                            has none): g' = g + wd theta, buf = mu buf + g', theta -= lr buf, with
                            buf in exp_avg (one copy per replica, starting at 0)             */
  double alpha_lr;       /* spread ratio alpha of Eq. 1 for the learning rate, 0 <= a < 1 */
  double alpha_wd;       /* spread ratio for the weight decay (Remark 1), 0 <= a < 1; 0 = none */
  int64_t sync_interval; /* T of Section 3.3, >= 1                                        */
  int32_t reshuffle;     /* 1: draw new permutations when the controller fires (Eq. 9)    */
  int32_t fuse_converge; /* 1: the round's last update also forms the mean (one pass over
                            the parameters); 0: update kernel then converge kernel        */
  uint64_t seed;         /* seed of the permutation generator                             */
  int32_t device;        /* CUDA device ordinal; ignored when n_tensors == 0              */
  int32_t grad_mode;     /* HDET_GRAD_AS_GIVEN: replica r steps with its own gradient (or the
                            shared one when grad_stride is 0).  HDET_GRAD_REPLICA_MEAN: the
                            kernel first averages the N per-replica gradients of a tile and
                            every replica steps with that mean -- the single-GPU form of the
                            gradient all-reduce in Algorithm 1's loop                      */
  int32_t n_replicas_global; /* 0: this handle holds all replicas.  > 0: the replica axis is sharded
                            over GPUs; this handle holds n_replicas of n_replicas_global replicas
                            (Eq. 1, Eq. 9 and the controller run over n_replicas_global <= 32)    */
  int32_t replica_offset;    /* global index of this handle's replica 0 (sharded handles only)     */
} hdet_config;

/* Base schedule and controller constants (Algorithm 1, Require).  Host arrays with
 * n_groups entries, copied during the call. */
typedef struct {
  int32_t kind;            /* HDET_SCHED_*                                                 */
  int32_t autolr;          /* 1: run the auto-LR controller (Section 3.4)                  */
  int64_t total_steps;     /* S                                                            */
  const double* max_lr;    /* eta_max per group (the constant rate for HDET_SCHED_CONSTANT) */
  const double* weight_decay; /* decoupled weight decay per group; NULL = all zero         */
  double pct_start;        /* p: fraction of S spent rising; needs 1 < p*S < S             */
  double div_factor;       /* initial rate = max_lr / div_factor                           */
  double final_div_factor; /* final rate = initial rate / final_div_factor                 */
  int64_t warmup_steps;    /* S_warm: the controller runs at syncs with t >= S_warm        */
  double beta;             /* velocity momentum of Eq. 7                                   */
  double sigma;            /* softmax temperature of Eq. 4, > 0                            */
  double lambda;           /* velocity gain of Eq. 7                                       */
  double f_div, f_final;   /* the two factors of Eq. 8, both > 0                           */
  int32_t auto_wd;         /* 1 (with autolr): the controller also adapts each group's weight-decay
                              base (Remark 1): Delta from the weight decays of the last update,
                              the same beta and lambda, no decay term                       */
  int32_t reserved;        /* set to 0                                                     */
} hdet_schedule;

/* Scalar state for logging and resume.  Tables are [group][replica]. */
typedef struct {
  int64_t step;                       /* completed updates t                               */
  int64_t n_acc;                      /* updates accumulated in loss_acc                   */
  int32_t fired;                      /* the controller has taken over the base rate       */
  int32_t round_ended;                /* the last hdet_step ended a round and
                                         hdet_autolr_update has not run since             */
  uint32_t device_status;             /* bit 0: a non-finite parameter was produced;
                                         bit 1: a bounded wait inside a kernel ran out     */
  int32_t reserved;
  double base[HDET_MAX_GROUPS];       /* base rate used by the last update                 */
  double ctrl_base[HDET_MAX_GROUPS];  /* eta_bar held by the controller (Eq. 7)            */
  double velocity[HDET_MAX_GROUPS];   /* v of Eq. 7                                        */
  double delta[HDET_MAX_GROUPS];      /* Delta of Eq. 6 at the last firing                 */
  double lr[HDET_MAX_GROUPS][HDET_MAX_REPLICAS]; /* rates used by the last update          */
  double wd[HDET_MAX_GROUPS][HDET_MAX_REPLICAS]; /* weight decays used by the last update  */
  int32_t perm_lr[HDET_MAX_GROUPS][HDET_MAX_REPLICAS]; /* pi of Eq. 9, learning rate       */
  int32_t perm_wd[HDET_MAX_GROUPS][HDET_MAX_REPLICAS]; /* pi of Eq. 9, weight decay        */
  double weights[HDET_MAX_REPLICAS];   /* w of Eq. 4 at the last firing                    */
  double loss_acc[HDET_MAX_REPLICAS];  /* running sum of losses in the current round       */
  double loss_round[HDET_MAX_REPLICAS];/* mean loss per replica over the last full round   */
  double gamma;                        /* decay of Eq. 8                                   */
  double wd_base[HDET_MAX_GROUPS];     /* base weight decay per group (adapted with auto_wd)   */
  double wd_velocity[HDET_MAX_GROUPS]; /* velocity of the weight-decay channel (Remark 1)      */
  double wd_delta[HDET_MAX_GROUPS];    /* its Delta at the last firing                         */
} hdet_state;

/*
 * hdet_create -- Algorithm 1, Init.  Checks cfg and the n_tensors descriptors, builds
 * the device work table (one entry per tile of a tensor) and a device status word on
 * cfg->device, and sets velocity 0, loss accumulator 0, identity permutations.
 * tensors may be NULL only when n_tensors == 0.  On success *out receives the handle;
 * on failure *out is NULL and nothing is left allocated.
 * Errors: INVALID_ARG (NULL, N/G/T/alpha out of range, numel <= 0, group out of range,
 * stride < numel with N > 1, missing moments for AdamW or missing buffer for SGD momentum,
 * momentum out of range or given with AdamW, state_stride 0 without a common gradient),
 * ALIGN, UNSUPPORTED (some but not all tensors with state_stride 0), CUDA.
 */
HDET_API int hdet_create(const hdet_config* cfg, const hdet_tensor* tensors, int64_t n_tensors, hdet_handle* out);

/*
 * hdet_set_schedule -- stores the base schedule eta(t) named in Algorithm 1's Require
 * list (one-cycle policy with cosine or linear annealing, or a constant) and the
 * controller constants (beta, sigma, lambda of Eq. 4 / Eq. 7; f_div, f_final of Eq. 8;
 * S_warm).  May be called again while the handle steps on the host; it does not reset the step
 * count, but it resets the base weight decays to sched->weight_decay.  While the scalar state
 * lives on the device (after hdet_step_device) the call returns HDET_ERR_STATE and changes
 * nothing: a schedule change would reach only part of the device state.  hdet_get_state followed
 * by hdet_set_state returns the handle to host stepping, where the schedule can be replaced.
 * Updates past step S keep the rate of step S - 1.
 * Errors: INVALID_ARG (NULL, S < 1, max_lr NULL, p*S <= 1 or p >= 1 for a one-cycle
 * kind, factors <= 0, sigma <= 0 with autolr, f_div or f_final <= 0), STATE (device-resident stepping).
 */
HDET_API int hdet_set_schedule(hdet_handle h, const hdet_schedule* sched);

/*
 * hdet_step -- one pass of Algorithm 1's loop body for update t = step + 1:
 *   base_g   = controller's eta_bar_g once it has fired, else schedule_g(t - 1)
 *   lr[g][r] = base_g * rho_{pi_g(r)}                 (Eq. 1, Section 3.2, Eq. 9)
 *   wd[g][r] = wd_g * rho'_{pi'_g(r)}                 (Remark 1; rho' uses alpha_wd)
 *   every replica of every tensor is updated in one kernel (Eq. 2 -- with a weight decay
 *   the SGD gradient is g + wd*theta --, or Adam with decoupled weight decay: theta *= 1 - lr*wd; m, v moving averages; theta -=
 *   lr * (m/(1-beta1^t)) / (sqrt(v/(1-beta2^t)) + eps))
 *   step_losses (HOST, N doubles, or NULL) are added to the round's accumulator
 *   if t mod T == 0 the replicas are averaged (Eq. 3) -- inside the same kernel when
 *   fuse_converge is set -- and *did_converge is set to 1 (else 0; may be NULL).
 * Asynchronous on `stream`.  Scalars are computed in double on the host and handed to
 * the kernel as fp32 launch parameters, so no host-to-device copy is issued.
 * Errors: INVALID_ARG, STATE (no schedule), CUDA (launch failure).
 */
HDET_API int hdet_step(hdet_handle h, const double* step_losses, void* stream, int32_t* did_converge);

/*
 * hdet_step_host_grads -- hdet_step for gradients that live in HOST memory: host_grads[k] points to
 * the gradients of tensor k laid out like its device gradient (replica r at host_grads[k] +
 * r * grad_stride elements; one copy when grad_stride is 0).  The call uploads them into the tensors' device
 * gradient arrays (one strided copy per tensor) and updates, so the copies are inside the call.  Copies and
 * updates overlap: the tensor list is cut into up to eight runs of consecutive tensors; the copies go to a
 * stream the handle creates on its first call here (ordered after everything already enqueued on `stream`),
 * and `stream` updates each run's tiles as soon as that run's copies have landed -- one kernel launch per run,
 * same arithmetic and same results as hdet_step on gradients already on the device.  When the call returns
 * everything is enqueued and later work on `stream` is ordered after all of it.  The host buffers must stay valid
 * until `stream` has passed the call's work; they should be pinned, otherwise every copy stages through the
 * driver and blocks.  The first call creates the stream and its events (no device memory).
 * Errors: as hdet_step, plus INVALID_ARG for NULL pointers and CUDA for a failed copy; nothing is enqueued when
 * an argument or the handle's state is rejected.
 */
HDET_API int hdet_step_host_grads(hdet_handle h, const void* const* host_grads, const double* step_losses,
                                  void* stream, int32_t* did_converge);

/*
 * Replica axis sharded over GPUs (the paper's own arrangement, one or more replicas per GPU).
 * Every rank creates a handle with n_replicas = its local replicas, n_replicas_global = N and its
 * replica_offset, and per step:
 *   hdet_step_sharded(h, losses of ALL N replicas (host, all-gathered by the caller), d_partial, ...)
 *     -- like hdet_step; on the last update of a round the kernel does not write a mean but the
 *        fp32 sums over the local replicas into d_partial (DEVICE, hdet_partial_layout elements,
 *        16-byte aligned, caller-owned), and sets *did_converge;
 *   the caller all-reduces d_partial (sum) over the ranks -- the one exchange of Eq. 3, P floats
 *   per round, e.g. ncclAllReduce / torch.distributed.all_reduce on the same stream;
 *   hdet_apply_mean(h, d_partial, stream) -- every local replica <- sum / N  (Eq. 3);
 *   hdet_autolr_update(h, ...) as usual (every rank computes the same scalars from the same losses).
 * The library itself calls no collective, so it has no dependency on a communication library and
 * remote data is only ever read from local memory.  With a sharded handle hdet_step, hdet_converge
 * and hdet_step_device return HDET_ERR_STATE / HDET_ERR_UNSUPPORTED, and grad_mode REPLICA_MEAN is
 * refused (all-reduce the gradients and pass a shared gradient instead).  hdet_step_sharded also works
 * on an unsharded handle (then hdet_apply_mean completes the converge locally).
 * hdet_partial_layout: offsets[k] = element offset of tensor k in the staging buffer (multiples of 4;
 * offsets may be NULL), *total_numel = its length.
 * Errors: INVALID_ARG, ALIGN, STATE, CUDA.
 */
HDET_API int hdet_step_sharded(hdet_handle h, const double* step_losses, void* d_partial, void* stream,
                               int32_t* did_converge);
HDET_API int hdet_apply_mean(hdet_handle h, const void* d_sum, void* stream);
HDET_API int hdet_partial_layout(hdet_handle h, int64_t* offsets, int64_t n_offsets, int64_t* total_numel);

/*
 * hdet_apply_mean_peers -- Eq. 3 across GPUs with the exchange inside the kernel instead of a collective call:
 * the second half of a sharded converge reads EVERY rank's staging buffer itself.  d_partials is a HOST array of
 * n_buffers DEVICE pointers, one per rank and in rank order (the same order on every rank, so that every rank
 * adds the same numbers in the same order and obtains the same bits): this GPU's own d_partial and its peers',
 * mapped into this process (peer access enabled, CUDA IPC, or symmetric memory) and read with ordinary loads
 * over NVLink.  Every local replica <- (sum over the buffers, fp64) / N; param_bf16 is refreshed.
 * The kernel waits for nobody.  The CALLER orders it: (1) every rank's hdet_step_sharded of the round; (2) a
 * barrier across the ranks that follows those kernels in stream order; (3) this call on every rank; (4) a second
 * barrier (or a second set of staging buffers used in alternation) before any rank's next round overwrites its
 * buffer.  Each rank reads (n_buffers - 1) x P floats from its peers, where a ring or in-switch all-reduce moves
 * 2 (W - 1) / W x P: the same at two ranks, four times as much at eight, so this form suits few ranks or small
 * models; hdet_apply_mean after an all-reduce is the general one.
 * Errors: INVALID_ARG (NULL or misaligned buffer, n_buffers outside 1 .. 32), CUDA.
 */
HDET_API int hdet_apply_mean_peers(hdet_handle h, const void* const* d_partials, int32_t n_buffers, void* stream);

/*
 * hdet_step_device -- hdet_step and, at the end of a round, hdet_autolr_update, with Algorithm 1's
 * scalar state kept on the device: nothing is computed on the host, nothing is copied, and the
 * losses are read from DEVICE memory (d_step_losses: N values of loss_dtype HDET_DTYPE_F32 or
 * HDET_DTYPE_F64, or NULL), so a training loop never has to wait for a loss to reach the host.
 * Per call: a one-warp fp64 kernel evaluates the schedule, Eq. 1 and the permutations of Eq. 9 into
 * the launch scalars and accumulates the losses; the fan-out kernel (fused with Eq. 3 on the last
 * update of a round) reads those scalars from device memory; after a round's last update a second
 * one-warp kernel latches the mean losses and, if auto-LR is on and t >= S_warm, runs Eq. 4 - Eq. 9
 * (softmax and sums by warp shuffles, one lane per replica).  The same double-precision code as the
 * host path is compiled for the device, so scalars agree with it to rounding of the math library.
 * Which kernels a call launches depends only on the step count, so a whole round of T calls can be
 * recorded once and replayed.  *did_converge as for hdet_step (may be NULL).
 * The first call after hdet_create / hdet_set_state copies the host state to the device with a
 * blocking copy; from then on the device copy is authoritative: hdet_get_state reads it back
 * (blocking) and refreshes the host copy, hdet_set_state returns the handle to host stepping, and
 * hdet_step / hdet_autolr_update return HDET_ERR_STATE in between.  If steps were replayed without
 * calling this function, call hdet_get_state before the next direct call so that the host knows the
 * step count again.
 * Errors: INVALID_ARG, STATE (no schedule), UNSUPPORTED (handle without tensors), CUDA.
 */
HDET_API int hdet_step_device(hdet_handle h, const void* d_step_losses, int32_t loss_dtype, void* stream,
                              int32_t* did_converge);

/*
 * hdet_warm_init -- warm noisy initialisation (Section 3.5, Eq. 10), to be called before the first
 * update when training starts from a checkpoint.  Replica 0 of every tensor must hold the checkpoint
 * theta_bar_0; on return (stream order) every replica r, replica 0 included, holds
 * theta_bar_0 + eps_r with eps_r ~ N(0, nu^2 ||theta_bar_0||^2 / d), where the norm and d (the number
 * of parameters) run over ALL tensors of the handle.  The noise is a counter-based Box-Muller draw
 * keyed by (seed, replica, tensor index, element index), so it does not depend on layout or launch
 * shape; nu = 0 copies the checkpoint to all replicas.  The paper uses nu = 0.01.
 * Moments and the step count are not touched.  The first call allocates a scratch buffer of one
 * double per 2048-element tile (freed by hdet_destroy); later calls allocate nothing.
 * Errors: INVALID_ARG (nu negative or not finite), CUDA.
 */
HDET_API int hdet_warm_init(hdet_handle h, double nu, uint64_t seed, void* stream);

/*
 * hdet_converge -- Eq. 3 on its own: theta_r <- (1/N) sum_r' theta_r' for every tensor.
 * Does not touch the step count, the moments or the loss accumulator.
 * Errors: INVALID_ARG, CUDA.
 */
HDET_API int hdet_converge(hdet_handle h, void* stream);

/*
 * hdet_autolr_update -- the auto-LR branch of Algorithm 1, to be called after the
 * hdet_step that set *did_converge.  With the round's mean losses L_r (round_losses,
 * HOST, N doubles; NULL = the accumulated mean) it computes w (Eq. 4), per group
 * Delta (Eq. 5 - 6) from the rates of the last update, the velocity and the new base
 * eta_bar (Eq. 7, gamma from Eq. 8), and draws new permutations (Eq. 9) when
 * reshuffle is set.  From then on hdet_step uses eta_bar as the group's base rate.
 * It is a no-op returning HDET_OK when autolr is off or t < S_warm.  It runs on the
 * host; `stream` is unused and may be NULL.
 * Errors: INVALID_ARG, STATE (the last hdet_step did not end a round, or the update
 * already ran for this round).
 */
HDET_API int hdet_autolr_update(hdet_handle h, const double* round_losses, void* stream);

/*
 * hdet_get_state -- copies the scalar state into *out.  Reads the device status word,
 * which synchronises with the device (cudaMemcpy) when the handle has tensors.
 * Returns HDET_ERR_NONFINITE (with *out filled) if a kernel flagged a non-finite value, and
 * HDET_ERR_TIMEOUT (with *out filled) if a kernel's bounded wait for its own copies ran out: the
 * kernels never spin without a limit, so a copy that does not complete ends as this status instead
 * of a hang.
 */
HDET_API int hdet_get_state(hdet_handle h, hdet_state* out);

/*
 * hdet_set_state -- restores step, n_acc, fired, round_ended, ctrl_base, velocity, the
 * permutations, loss_acc and loss_round from *in (resume); the other fields are
 * recomputed.  Clears the device status word.  Waits for the device to become idle (earlier
 * device-resident steps must not outlive the state they read) and returns the handle to host
 * stepping.
 * Errors: INVALID_ARG (NULL, negative step, an array that is not a permutation).
 */
HDET_API int hdet_set_state(hdet_handle h, const hdet_state* in);

/*
 * hdet_selftest_bounded_wait -- (no counterpart in the paper: a diagnostic of the library's failure handling.)
 * The bulk-copy kernels wait for their own copies with a limit of about a second; a copy that never completes
 * ends as HDET_ERR_TIMEOUT instead of a hung GPU.  This call exercises that path on purpose and without any
 * fault: it launches a one-CTA kernel that waits, with the same limit, on a barrier that nothing completes.
 * About a second later (stream order) bit 1 of the device status word is set; hdet_get_state then returns
 * HDET_ERR_TIMEOUT, update kernels launched while the bit is set leave their tiles untouched, and
 * hdet_set_state clears the bit, after which the handle steps normally.  The CUDA context stays usable.
 * Errors: INVALID_ARG, UNSUPPORTED (handle without tensors), CUDA.
 */
HDET_API int hdet_selftest_bounded_wait(hdet_handle h, void* stream);

/* hdet_destroy -- frees the work table and the handle.  NULL is accepted. */
HDET_API int hdet_destroy(hdet_handle h);

/*
 * hdet_converge_static -- (the paper has no counterpart: this is a packaging variant of
 * hdet_converge.)  Averages the N replicas of every listed tensor like hdet_converge, but needs
 * no handle and never allocates device memory.  It is meant for callers that cannot call
 * cudaMalloc at the point where they need the mean: code running under a framework that has
 * handed all device memory to its own pool, or a latency-critical loop where an allocation
 * (which may synchronise the device) is not acceptable.
 *
 * The caller passes the same hdet_tensor descriptors as to hdet_create; only param, numel and
 * param_stride are read (grad and the moments may be NULL; param_bf16 is ignored).  The work tables that hdet_create
 * would put in allocated memory are written, on every call, into one static device array of
 * about 0.6 MB that each GPU loading the library holds until the process exits.  Limits, checked
 * before anything is launched: at most HDET_STATIC_MAX_TENSORS tensors and HDET_STATIC_MAX_TILES
 * tiles of 2048 elements in total (each tensor occupies ceil(numel / 2048) tiles, so at most
 * 134,217,728 elements per replica); larger lists return HDET_ERR_UNSUPPORTED with a message and
 * should use hdet_converge.
 *
 * The first call on a device resolves the array's device address (cudaGetSymbolAddress) and
 * queries the launch shape; make that first call before any stream capture begins.  All calls share
 * the array, which keeps the previous call's contents: nothing in it has to start at zero, and each
 * call rewrites the tables it is going to read, in stream order.  Two calls whose work overlaps on the
 * GPU (different streams without an event between them, or different host threads) race on the array
 * and must be serialised by the caller.  The tables are copied from temporary pageable host memory
 * on every call, so the call may wait for earlier work on `stream`, and a call on a stream that is
 * being captured is refused with HDET_ERR_UNSUPPORTED (a recorded copy would outlive its source).
 * A non-finite mean is not reported by this entry point (it has no handle to hold a status).
 * Errors: INVALID_ARG, ALIGN, UNSUPPORTED (limits, capturing stream), CUDA; text via hdet_last_error(NULL).
 */
#define HDET_STATIC_MAX_TENSORS 1024
#define HDET_STATIC_MAX_TILES 65536
HDET_API int hdet_converge_static(const hdet_tensor* tensors, int64_t n_tensors, int32_t n_replicas,
                                  int32_t device, void* stream);

/* hdet_last_error -- text of the last failure on h (when h is NULL: of the last failed call
 * that has no handle, hdet_create or hdet_converge_static, on this thread).  The pointer stays valid until the next call on that handle. */
HDET_API const char* hdet_last_error(hdet_handle h);

/*
 * hdet_plan_tiles -- (no counterpart in the paper: a host-only view of the work plan, for tests and tools.)
 * Runs the checks of hdet_create on cfg and the descriptors and reports the plan hdet_create would build,
 * without touching a device (the pointers are only inspected for alignment, never dereferenced):
 *   *n_tiles              number of tiles; tile i covers elements [2048 * tile_index[i],
 *                         min(numel, 2048 * (tile_index[i] + 1))) of tensor tile_tensor[i]
 *   tile_tensor, tile_index   HOST arrays of `capacity` entries, or both NULL to query the count
 *   tensor_access[k]      HOST, n_tensors entries or NULL: 0 = scalar accesses, 1 = 128-bit accesses,
 *                         3 = 128-bit accesses and bulk copies of whole tiles (AdamW)
 *   partial_offsets[k]    HOST, n_tensors entries or NULL: as hdet_partial_layout
 * Errors: those of hdet_create's checks; INVALID_ARG when capacity is too small.
 */
HDET_API int hdet_plan_tiles(const hdet_config* cfg, const hdet_tensor* tensors, int64_t n_tensors, int32_t* tile_tensor,
                             int32_t* tile_index, int64_t capacity, int64_t* n_tiles, int32_t* tensor_access,
                             int64_t* partial_offsets);

/* hdet_kernel_launches -- number of kernels this handle has launched so far. */
HDET_API int64_t hdet_kernel_launches(hdet_handle h);

#ifdef __cplusplus
}
#endif
#endif /* HDET_H_ */
