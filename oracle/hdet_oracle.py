"""CPU oracle for the HDET fan-out / converge / auto-LR hot path, in double precision.

THIS IS TEST INFRASTRUCTURE.  It is a plain, slow, step-by-step statement of
what the paper's method computes, used only to check the CUDA library and to
serve as the timed CPU baseline of the benchmark.  The product never imports
it, and it imports nothing from the product: the two share no code.  Its only
dependency is numpy.

Every function names the passage of the paper (arXiv 2604.24708, "HDET:
Hyperparameter-Divergent Ensemble Training") it follows.  Where the paper is
silent the reading taken is stated in the function's docstring.

Parity pins: every function below is pinned by the CPU tests (worked example of
the experimental setup, closed forms, invariants, library special cases, brute
force).  Two things are pinned only by this repository's own written
definitions and are therefore "parity unpinned" by the paper:

* the exact sequence of permutations drawn by ``permutation`` (the paper says
  only "a fresh random permutation"); its building block, the SplitMix64
  finaliser, is pinned by that generator's published test vector;
* full-run trajectories of the synthetic workloads (no published values exist);
  they are covered by the invariants plus agreement of the two implementations.
"""
from __future__ import annotations

import math
from typing import List, Optional, Sequence

import numpy as np

SGD = 0
ADAMW = 1
SCHED_CONSTANT = 0
SCHED_ONECYCLE_COS = 1
SCHED_ONECYCLE_LINEAR = 2


# --------------------------------------------------------------------------- #
# Section 3.2, Eq. 1: spread multipliers
# --------------------------------------------------------------------------- #
def spread_multipliers(n: int, alpha: float) -> np.ndarray:
    """rho_r = 1 + alpha * (r - (N-1)/2) / delta with delta = max((N-1)/2, 0.5)  (Eq. 1).

    For N = 1 the numerator is zero, so rho_0 = 1.
    """
    delta = max((n - 1) / 2.0, 0.5)
    rho = np.empty(n, dtype=np.float64)
    for r in range(n):
        rho[r] = 1.0 + alpha * (r - (n - 1) / 2.0) / delta
    return rho


# --------------------------------------------------------------------------- #
# Base schedule named by Algorithm 1's Require list: OneCycleLR
# --------------------------------------------------------------------------- #
def onecycle_lr(i: int, total_steps: int, max_lr: float, pct_start: float = 0.3,
                div_factor: float = 25.0, final_div_factor: float = 1e4,
                kind: int = SCHED_ONECYCLE_COS) -> float:
    """Learning rate of the one-cycle policy at 0-based step i.

    The paper only names the scheduler (Section 2; Algorithm 1, Require); this is
    the publicly documented two-phase policy of the PyTorch scheduler it names,
    without momentum cycling: the rate climbs from max_lr/div_factor to max_lr
    over steps 0 .. p*S - 1, then falls to max_lr/(div_factor*final_div_factor)
    at step S - 1.  Phase boundaries are real numbers (p*S - 1 is not rounded).
    """
    initial = max_lr / div_factor
    floor = initial / final_div_factor
    end_up = float(pct_start * total_steps) - 1.0
    end_down = float(total_steps) - 1.0
    if i <= end_up:
        start, end = initial, max_lr
        q = i / end_up
    else:
        start, end = max_lr, floor
        q = (i - end_up) / (end_down - end_up)
    if kind == SCHED_ONECYCLE_COS:
        return end + (start - end) / 2.0 * (1.0 + math.cos(math.pi * q))
    if kind == SCHED_ONECYCLE_LINEAR:
        return start + (end - start) * q
    raise ValueError("kind")


def base_lr(kind: int, i: int, total_steps: int, max_lr: float, pct_start: float,
            div_factor: float, final_div_factor: float) -> float:
    """Shared base rate eta(t) of Section 3.2 for update number t = i + 1."""
    if kind == SCHED_CONSTANT:
        return max_lr
    return onecycle_lr(i, total_steps, max_lr, pct_start, div_factor, final_div_factor, kind)


# --------------------------------------------------------------------------- #
# Section 3.4, Eq. 4 - Eq. 8: auto-LR controller
# --------------------------------------------------------------------------- #
def decay_gamma(f_div: float, f_final: float, total_steps: int, warmup_steps: int, sync_interval: int) -> float:
    """gamma = 1 - exp(-log(f_div/f_final) / K), K = (S - S_warm) / T as a real number  (Eq. 8).

    The formula is taken literally; K <= 0 (no interval left) gives gamma = 0.
    """
    k = (total_steps - warmup_steps) / float(sync_interval)
    if k <= 0.0:
        return 0.0
    return 1.0 - math.exp(-math.log(f_div / f_final) / k)


def softmax_weights(losses: Sequence[float], sigma: float) -> np.ndarray:
    """s_r = (Lbar - L_r) / sigma, w = softmax(s)  (Eq. 4).  The maximum is subtracted before exp."""
    L = np.asarray(losses, dtype=np.float64)
    s = (L.mean() - L) / sigma
    e = np.exp(s - s.max())
    return e / e.sum()


def hypergradient(w: np.ndarray, eta: np.ndarray):
    """eta_tilde = sum_r w_r eta_r, eta_bar = (1/N) sum_r eta_r, Delta = eta_tilde - eta_bar  (Eq. 5, Eq. 6)."""
    tilde = float(np.sum(w * eta))
    bar = float(np.sum(eta) / len(eta))
    return tilde, bar, tilde - bar


def meta_update(v: float, bar: float, delta: float, beta: float, gamma: float, lam: float):
    """v' = beta v + (1 - beta) Delta;  eta_bar' = eta_bar (1 - gamma) + v' lambda  (Eq. 7)."""
    v_new = beta * v + (1.0 - beta) * delta
    return v_new, bar * (1.0 - gamma) + v_new * lam


# --------------------------------------------------------------------------- #
# Section 3.4, Eq. 9: random reassignment
# --------------------------------------------------------------------------- #
_U64 = (1 << 64) - 1


def mix64(x: int) -> int:
    """Finaliser of SplitMix64 (Steele, Lea & Flood 2014) on a Python int modulo 2**64."""
    x &= _U64
    x = ((x ^ (x >> 30)) * 0xBF58476D1CE4E5B9) & _U64
    x = ((x ^ (x >> 27)) * 0x94D049BB133111EB) & _U64
    return x ^ (x >> 31)


def permutation(seed: int, sync_index: int, channel: int, n: int) -> List[int]:
    """The permutation pi of Eq. 9 for one hyperparameter channel at one sync.

    The paper asks for a fresh, independent random permutation per hyperparameter;
    the generator is this repository's written definition: a key
    mix64(mix64(mix64(seed) + sync_index) + channel), then a Fisher-Yates pass
    from the identity, j = N-1 .. 1, swapping positions j and
    mix64(key + j * 0x9E3779B97F4A7C15) mod (j + 1).
    """
    key = mix64(mix64(mix64(seed) + sync_index) + channel)
    perm = list(range(n))
    for j in range(n - 1, 0, -1):
        u = mix64(key + j * 0x9E3779B97F4A7C15)
        k = u % (j + 1)
        perm[j], perm[k] = perm[k], perm[j]
    return perm


# --------------------------------------------------------------------------- #
# Eq. 2 and the Adam-family update named in Section 4.1
# --------------------------------------------------------------------------- #
def sgd_update(theta: np.ndarray, g: np.ndarray, lr: float) -> None:
    """theta <- theta - eta_r * g  (Eq. 2), in place."""
    theta -= lr * g


def sgd_momentum_update(theta: np.ndarray, buf: np.ndarray, g: np.ndarray, lr: float, wd: float, mu: float) -> None:
    """SGD with weight decay and a momentum buffer, in place (an extension: Eq. 2 has neither).

    The usual definition (as in torch.optim.SGD without dampening or Nesterov): g' = g + wd * theta,
    buf <- mu * buf + g' (buf starts at zero), theta <- theta - eta_r * buf.  With wd = mu = 0 this is Eq. 2.
    """
    g_eff = g + wd * theta
    buf[...] = mu * buf + g_eff
    theta -= lr * buf


def adamw_update(theta: np.ndarray, m: np.ndarray, v: np.ndarray, g: np.ndarray, lr: float, wd: float,
                 beta1: float, beta2: float, eps: float, t: int) -> None:
    """One Adam step with decoupled weight decay, in place; t is the 1-based update number.

    The paper says only that the optimizer is Adam and that weight decay is a
    scalar that may be explored (Section 4.1; Remark 1).  Reading taken: the
    decay multiplies the pre-update parameter, eps is added outside the square
    root of the bias-corrected second moment.
    """
    bc1 = 1.0 - beta1 ** t
    bc2 = 1.0 - beta2 ** t
    theta *= 1.0 - lr * wd
    m[...] = beta1 * m + (1.0 - beta1) * g
    v[...] = beta2 * v + (1.0 - beta2) * g * g
    theta -= lr * (m / bc1) / (np.sqrt(v / bc2) + eps)


# --------------------------------------------------------------------------- #
# Section 3.3, Eq. 3: converge
# --------------------------------------------------------------------------- #
def converge(theta: np.ndarray) -> None:
    """theta_r <- (1/N) sum_r' theta_r' for every r  (Eq. 3); theta has shape [N, numel], in place."""
    n = theta.shape[0]
    mean = np.zeros(theta.shape[1], dtype=np.float64)
    for r in range(n):
        mean += theta[r]
    mean /= n
    for r in range(n):
        theta[r] = mean


def bf16_bits(x: np.ndarray) -> np.ndarray:
    """The bfloat16 image of single-precision values, as 16-bit patterns, rounding to nearest, ties to even.

    Section 3.3's averaged parameters (Eq. 3) are what the next forward pass of Algorithm 1 reads; a
    mixed-precision model reads them as bfloat16.  The paper does not say how that copy is made.  Reading
    taken: it is the stored single-precision parameter rounded once to bfloat16, which keeps the upper 16 bits
    of the fp32 pattern: add 0x7FFF plus the lowest kept bit to the pattern, then drop the lower 16 bits.
    (Finite inputs only; the path never stores a NaN here without flagging it.)
    """
    u = np.ascontiguousarray(x, dtype=np.float32).view(np.uint32).astype(np.uint64)
    keep_lsb = (u >> np.uint64(16)) & np.uint64(1)
    return ((u + np.uint64(0x7FFF) + keep_lsb) >> np.uint64(16)).astype(np.uint16)


def averaged_bf16(theta: np.ndarray) -> np.ndarray:
    """bfloat16 copy of the averaged parameters after Eq. 3: replica 0 of `theta` ([N, numel], double, all rows
    equal after converge) rounded to single precision (the stored master value), then to bfloat16."""
    return bf16_bits(theta[0].astype(np.float32))


# --------------------------------------------------------------------------- #
# Algorithm 1
# --------------------------------------------------------------------------- #
class HdetOracle:
    """Algorithm 1 with N replicas held side by side, step by step, in double.

    Tensors are given as a list of [N, numel] arrays (initial parameters per
    replica) with one optimizer-group id each.  State follows Algorithm 1's
    Init line: velocity 0, accumulated loss 0; Adam moments start at 0; the
    permutations start as the identity (rank r holds rho_r, Algorithm 1's
    second line).

    Readings taken where the paper is silent or ambiguous:

    * update number t uses the schedule value at 0-based index t - 1; converge
      follows update t when t mod T = 0; "t >= S_warm" counts completed updates;
    * gradients may differ per replica (general case) or be shared (Eq. 2); with
      grad_mean the per-replica gradients are first averaged over the replicas
      (Algorithm 1, "AllReduce gradients") and every replica steps with that mean;
    * Adam moments are not averaged at converge (Eq. 3 averages "model
      parameters");
    * L_r is the mean loss over the last round (Section 3.4), so the accumulator
      is reset at every sync, not only inside the auto-LR branch;
    * once the controller has fired, the base rate of a group is the controller's
      eta_bar, held for the next T updates; the one-cycle formula is no longer
      consulted (the decay gamma takes over the anneal);
    * permutations change only when the controller fires (Algorithm 1), one
      independent draw per group for the learning rate (channel 2g) and one for
      the weight decay (channel 2g + 1);
    * the losses are one per replica and shared by all groups;
    * weight decay is spread like the learning rate (Remark 1) with its own
      ratio alpha_wd; its base is adapted by the same controller only with
      auto_wd (Delta from the weight decays, same beta and lambda, gamma = 0);
    * eta_bar is not clamped.
    """

    def __init__(self, params: Sequence[np.ndarray], groups: Sequence[int], n_groups: int, *,
                 optimizer: int, total_steps: int, sched_kind: int, max_lr: Sequence[float],
                 weight_decay: Sequence[float], pct_start: float = 0.3, div_factor: float = 25.0,
                 final_div_factor: float = 1e4, alpha_lr: float = 0.0, alpha_wd: float = 0.0,
                 sync_interval: int = 1, autolr: bool = False, warmup_steps: int = 0,
                 ctrl_beta: float = 0.9, ctrl_sigma: float = 0.1, ctrl_lambda: float = 0.5,
                 f_div: float = 25.0, f_final: float = 1.0, reshuffle: bool = True, seed: int = 0,
                 beta1: float = 0.9, beta2: float = 0.999, eps: float = 1e-8,
                 n_replicas: Optional[int] = None, grad_mean: bool = False, momentum: float = 0.0,
                 auto_wd: bool = False):
        self.theta = [np.array(p, dtype=np.float64, copy=True) for p in params]
        self.n = self.theta[0].shape[0] if self.theta else int(n_replicas)
        self.m = [np.zeros_like(p) for p in self.theta]
        self.v = [np.zeros_like(p) for p in self.theta]
        self.groups = list(groups)
        self.G = n_groups
        self.optimizer = optimizer
        self.S = total_steps
        self.sched_kind = sched_kind
        self.max_lr = list(max_lr)
        self.weight_decay = list(weight_decay)
        self.pct_start, self.div_factor, self.final_div_factor = pct_start, div_factor, final_div_factor
        self.alpha_lr, self.alpha_wd = alpha_lr, alpha_wd
        self.T = sync_interval
        self.autolr, self.S_warm = bool(autolr), warmup_steps
        self.beta, self.sigma, self.lam = ctrl_beta, ctrl_sigma, ctrl_lambda
        self.f_div, self.f_final = f_div, f_final
        self.reshuffle, self.seed = bool(reshuffle), seed
        self.beta1, self.beta2, self.eps = beta1, beta2, eps
        self.grad_mean = bool(grad_mean)
        self.momentum = momentum
        # Algorithm 1, Init
        self.i = 0
        self.fired = False
        self.ctrl_base = [0.0] * n_groups
        self.vel = [0.0] * n_groups
        self.perm_lr = [list(range(self.n)) for _ in range(n_groups)]
        self.perm_wd = [list(range(self.n)) for _ in range(n_groups)]
        self.L_acc = np.zeros(self.n, dtype=np.float64)
        self.n_acc = 0
        # quantities exposed for comparison
        self.lr = None        # [G][N] rates used by the last update
        self.wd = None        # [G][N] weight decays used by the last update
        self.base = None      # [G] base rates used by the last update
        self.w = None         # [N] softmax weights of the last controller firing
        self.delta = [0.0] * n_groups
        # Remark 1: the same controller on the weight-decay channel (off unless auto_wd)
        self.auto_wd = bool(auto_wd)
        self.wd_base = list(weight_decay)      # h_bar of the weight-decay channel, per group
        self.vel_wd = [0.0] * n_groups
        self.delta_wd = [0.0] * n_groups
        self.L_round = None   # [N] mean losses of the last completed round

    def tables(self):
        """Base rates and the per-replica [G][N] tables for the update at the current index."""
        n = self.n
        rho = spread_multipliers(n, self.alpha_lr)          # Eq. 1
        rho_wd = spread_multipliers(n, self.alpha_wd)       # Remark 1
        base = np.empty(self.G)
        lr = np.empty((self.G, n))
        wd = np.empty((self.G, n))
        for g in range(self.G):
            if self.fired:
                base[g] = self.ctrl_base[g]                 # Eq. 7 result, held over the round
            else:
                base[g] = base_lr(self.sched_kind, self.i, self.S, self.max_lr[g], self.pct_start,
                                  self.div_factor, self.final_div_factor)
            for r in range(n):
                lr[g][r] = base[g] * rho[self.perm_lr[g][r]]             # Section 3.2; Eq. 9
                wd[g][r] = self.wd_base[g] * rho_wd[self.perm_wd[g][r]]
        return base, lr, wd

    def step(self, grads: Sequence[np.ndarray], losses: Optional[Sequence[float]] = None) -> bool:
        """One pass of Algorithm 1's loop body; returns True when this update ended a round.

        grads[k] has shape [N, numel_k] (per-replica gradients) or [numel_k]
        (one gradient shared by every replica, Eq. 2).
        """
        base, lr, wd = self.tables()
        n = self.n
        t = self.i + 1
        for k, th in enumerate(self.theta):
            g_id = self.groups[k]
            gk = np.asarray(grads[k], dtype=np.float64)
            if self.grad_mean and gk.ndim == 2:
                g_bar = np.zeros(gk.shape[1], dtype=np.float64)     # Algorithm 1: AllReduce gradients (mean)
                for r in range(n):
                    g_bar += gk[r]
                gk = g_bar / n
            for r in range(n):
                g_r = gk if gk.ndim == 1 else gk[r]
                if self.optimizer == SGD and self.momentum == 0.0 and wd[g_id][r] == 0.0:
                    sgd_update(th[r], g_r, lr[g_id][r])                                   # Eq. 2
                elif self.optimizer == SGD:
                    sgd_momentum_update(th[r], self.m[k][r], g_r, lr[g_id][r], wd[g_id][r], self.momentum)
                else:
                    adamw_update(th[r], self.m[k][r], self.v[k][r], g_r, lr[g_id][r], wd[g_id][r],
                                 self.beta1, self.beta2, self.eps, t)
        self.base, self.lr, self.wd = base, lr, wd
        if losses is not None:
            self.L_acc += np.asarray(losses, dtype=np.float64)      # Algorithm 1: L_acc <- L_acc + loss
        self.n_acc += 1
        self.i += 1
        if t % self.T != 0:
            return False
        for th in self.theta:
            converge(th)                                            # Eq. 3
        self.L_round = self.L_acc / self.n_acc
        self.L_acc = np.zeros(n, dtype=np.float64)
        self.n_acc = 0
        if self.autolr and t >= self.S_warm:
            self.controller(t)
        return True

    def controller(self, t: int) -> None:
        """The auto-LR branch of Algorithm 1 at a sync step (Eq. 4 - Eq. 9)."""
        gamma = decay_gamma(self.f_div, self.f_final, self.S, self.S_warm, self.T)       # Eq. 8
        self.w = softmax_weights(self.L_round, self.sigma)                               # Eq. 4
        for g in range(self.G):
            tilde, bar, delta = hypergradient(self.w, self.lr[g])                        # Eq. 5, Eq. 6
            self.vel[g], self.ctrl_base[g] = meta_update(self.vel[g], bar, delta, self.beta, gamma, self.lam)  # Eq. 7
            self.delta[g] = delta
            if self.auto_wd:
                # Remark 1: Delta = h_tilde - h_bar with h the weight decays of the last update; the same
                # velocity and gain; no decay term, since no floor is scheduled for the weight decay.
                _, bar_wd, delta_wd = hypergradient(self.w, self.wd[g])
                self.vel_wd[g], self.wd_base[g] = meta_update(self.vel_wd[g], bar_wd, delta_wd, self.beta, 0.0, self.lam)
                self.delta_wd[g] = delta_wd
        self.fired = True
        if self.reshuffle:
            k = t // self.T
            for g in range(self.G):
                self.perm_lr[g] = permutation(self.seed, k, 2 * g, self.n)               # Eq. 9
                self.perm_wd[g] = permutation(self.seed, k, 2 * g + 1, self.n)


# --------------------------------------------------------------------------- #
# Section 3.5, Eq. 10: warm noisy initialisation
# --------------------------------------------------------------------------- #
WARM_STREAM = 0x5741524D  # ASCII "WARM": separates these draws from the permutation draws


def warm_sigma(theta0: Sequence[np.ndarray], nu: float) -> float:
    """Standard deviation of Eq. 10: nu * sqrt(||theta_bar_0||^2 / d), d = total number of parameters.

    theta0 is the whole checkpoint as a list of tensors (the norm and d run over all of them).
    """
    norm2 = 0.0
    d = 0
    for t in theta0:
        t = np.asarray(t, dtype=np.float64)
        norm2 += float(np.sum(t * t))
        d += t.size
    return nu * math.sqrt(norm2 / d)


def warm_noise(seed: int, replica: int, tensor: int, start: int, n: int) -> np.ndarray:
    """Standard normal draws epsilon_r / sigma of Eq. 10 for elements start .. start+n-1 of one tensor.

    The paper asks for independent Gaussian noise per replica and parameter; the generator is this
    repository's written definition (counter-based, so any element can be drawn on its own):
    key = mix64(mix64(mix64(mix64(seed) + WARM_STREAM) + replica) + tensor); the element pair
    p = e // 2 takes u = mix64(key + p * 0x9E3779B97F4A7C15), u1 = ((u >> 41) + 0.5) / 2**23,
    u2 = ((u >> 16) & 0xFFFFFF) / 2**24, and the Box-Muller transform gives
    z_even = sqrt(-2 ln u1) cos(2 pi u2), z_odd = sqrt(-2 ln u1) sin(2 pi u2).
    """
    key = mix64(mix64(mix64(mix64(seed) + WARM_STREAM) + replica) + tensor)
    out = np.empty(n, dtype=np.float64)
    for j in range(n):
        e = start + j
        u = mix64(key + (e // 2) * 0x9E3779B97F4A7C15)
        u1 = ((u >> 41) + 0.5) / 8388608.0
        u2 = ((u >> 16) & 0xFFFFFF) / 16777216.0
        radius = math.sqrt(-2.0 * math.log(u1))
        out[j] = radius * (math.cos(2.0 * math.pi * u2) if e % 2 == 0 else math.sin(2.0 * math.pi * u2))
    return out


def warm_noisy_init(theta0_slab: np.ndarray, sigma: float, seed: int, n_replicas: int, tensor: int,
                    start: int = 0) -> np.ndarray:
    """theta_r <- theta_bar_0 + epsilon_r, epsilon_r ~ N(0, sigma^2) independently per replica  (Eq. 10).

    theta0_slab holds elements start .. of tensor `tensor` of the checkpoint; sigma comes from
    warm_sigma over the whole checkpoint.  Returns an [N, len] array.
    """
    t0 = np.asarray(theta0_slab, dtype=np.float64)
    out = np.empty((n_replicas, t0.size), dtype=np.float64)
    for r in range(n_replicas):
        out[r] = t0 + sigma * warm_noise(seed, r, tensor, start, t0.size)
    return out
