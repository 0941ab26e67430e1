"""Mutation check of the oracle's pins: a plausible mistake planted anywhere in the oracle must fail a pin.

Each mutant is a one-line edit of oracle/hdet_oracle.py's source (a dropped term, a wrong sign or index,
a swapped operand), compiled into a scratch module on the CPU.  The pin tests of test_oracle_pins.py are
then run against the mutant and at least one of them has to fail.
"""
import inspect
import itertools
import types

import pytest

import test_oracle_pins as pins
from oracle import hdet_oracle as O

SOURCE = inspect.getsource(O)

MUTANTS = [
    # Eq. 1
    ("rho[r] = 1.0 + alpha * (r - (n - 1) / 2.0) / delta", "rho[r] = 1.0 + alpha * (r - n / 2.0) / delta"),
    ("rho[r] = 1.0 + alpha * (r - (n - 1) / 2.0) / delta", "rho[r] = 1.0 - alpha * (r - (n - 1) / 2.0) / delta"),
    ("delta = max((n - 1) / 2.0, 0.5)", "delta = max((n - 1) / 2.0, 1.0)"),
    ("delta = max((n - 1) / 2.0, 0.5)", "delta = max(n / 2.0, 0.5)"),
    # one-cycle
    ("end_up = float(pct_start * total_steps) - 1.0", "end_up = float(pct_start * total_steps)"),
    ("floor = initial / final_div_factor", "floor = max_lr / final_div_factor"),
    ("return end + (start - end) / 2.0 * (1.0 + math.cos(math.pi * q))",
     "return end + (start - end) / 2.0 * (1.0 - math.cos(math.pi * q))"),
    ("q = (i - end_up) / (end_down - end_up)", "q = (i - end_up) / end_down"),
    ("return start + (end - start) * q", "return end + (start - end) * q"),
    # Eq. 8
    ("k = (total_steps - warmup_steps) / float(sync_interval)", "k = (total_steps - warmup_steps) // sync_interval"),
    ("return 1.0 - math.exp(-math.log(f_div / f_final) / k)", "return 1.0 - math.exp(-math.log(f_final / f_div) / k)"),
    ("k = (total_steps - warmup_steps) / float(sync_interval)", "k = total_steps / float(sync_interval)"),
    # Eq. 4
    ("s = (L.mean() - L) / sigma", "s = (L - L.mean()) / sigma"),
    ("s = (L.mean() - L) / sigma", "s = (L.mean() - L) * sigma"),
    ("return e / e.sum()", "return e / e.max()"),
    # Eq. 5 - 6
    ("return tilde, bar, tilde - bar", "return tilde, bar, bar - tilde"),
    ("bar = float(np.sum(eta) / len(eta))", "bar = float(np.sum(eta) / (len(eta) - 1))"),
    # Eq. 7
    ("v_new = beta * v + (1.0 - beta) * delta", "v_new = beta * v + delta"),
    ("return v_new, bar * (1.0 - gamma) + v_new * lam", "return v_new, bar * (1.0 - gamma) + v * lam"),
    ("return v_new, bar * (1.0 - gamma) + v_new * lam", "return v_new, bar * (1.0 + gamma) + v_new * lam"),
    ("return v_new, bar * (1.0 - gamma) + v_new * lam", "return v_new, (bar + v_new * lam) * (1.0 - gamma)"),
    # Eq. 9
    ("k = u % (j + 1)", "k = u % j"),
    ("for j in range(n - 1, 0, -1):", "for j in range(n - 2, 0, -1):"),
    ("key = mix64(mix64(mix64(seed) + sync_index) + channel)", "key = mix64(mix64(mix64(seed) + sync_index))"),
    ("x = ((x ^ (x >> 27)) * 0x94D049BB133111EB) & _U64", "x = ((x ^ (x >> 29)) * 0x94D049BB133111EB) & _U64"),
    # Eq. 2 / Adam
    ("theta -= lr * g", "theta += lr * g"),
    ("theta *= 1.0 - lr * wd", "theta *= 1.0 - wd"),
    ("bc2 = 1.0 - beta2 ** t", "bc2 = 1.0 - beta2 ** (t - 1) if t > 1 else 1.0 - beta2"),
    ("bc1 = 1.0 - beta1 ** t", "bc1 = 1.0"),
    ("v[...] = beta2 * v + (1.0 - beta2) * g * g", "v[...] = beta2 * v + (1.0 - beta2) * g"),
    ("m[...] = beta1 * m + (1.0 - beta1) * g", "m[...] = beta1 * m + g"),
    ("theta -= lr * (m / bc1) / (np.sqrt(v / bc2) + eps)", "theta -= lr * (m / bc1) / np.sqrt(v / bc2 + eps)"),
    ("theta -= lr * (m / bc1) / (np.sqrt(v / bc2) + eps)", "theta -= lr * (m / bc1) / (np.sqrt(v) / bc2 + eps)"),
    # Eq. 3
    ("mean /= n", "mean /= (n - 1) if n > 1 else 1"),
    ("for r in range(n):\n        mean += theta[r]", "for r in range(n - 1):\n        mean += theta[r]"),
    # Algorithm 1
    ("t = self.i + 1\n        for k, th", "t = self.i\n        for k, th"),
    ("base[g] = base_lr(self.sched_kind, self.i, self.S,", "base[g] = base_lr(self.sched_kind, self.i + 1, self.S,"),
    ("if t % self.T != 0:", "if (t + 1) % self.T != 0:"),
    ("if self.autolr and t >= self.S_warm:", "if self.autolr and t > self.S_warm + self.T:"),
    ("self.L_acc = np.zeros(n, dtype=np.float64)\n        self.n_acc = 0\n        if self.autolr", "if self.autolr"),
    ("self.L_round = self.L_acc / self.n_acc", "self.L_round = self.L_acc / self.T / 2"),
    ("lr[g][r] = base[g] * rho[self.perm_lr[g][r]]", "lr[g][r] = base[g] * rho[r]"),
    ("wd[g][r] = self.wd_base[g] * rho_wd[self.perm_wd[g][r]]", "wd[g][r] = self.wd_base[g] * rho_wd[self.perm_lr[g][r]]"),
    ("wd[g][r] = self.wd_base[g] * rho_wd[self.perm_wd[g][r]]", "wd[g][r] = self.wd_base[g] * rho[self.perm_wd[g][r]]"),
    ("tilde, bar, delta = hypergradient(self.w, self.lr[g])", "tilde, bar, delta = hypergradient(self.w, self.lr[0])"),
    ("self.perm_wd[g] = permutation(self.seed, k, 2 * g + 1, self.n)", "self.perm_wd[g] = permutation(self.seed, k, 2 * g, self.n)"),
    ("        for th in self.theta:\n            converge(th)", "        for th in self.theta + self.m:\n            converge(th)"),
    ("base[g] = self.ctrl_base[g] ", "base[g] = base_lr(self.sched_kind, self.i, self.S, self.ctrl_base[g], self.pct_start, self.div_factor, self.final_div_factor) "),
    ("sgd_update(th[r], g_r, lr[g_id][r])", "sgd_update(th[r], g_r, base[g_id])"),
    ("gk = g_bar / n", "gk = g_bar"),
    # Remark 1, weight-decay channel
    ("_, bar_wd, delta_wd = hypergradient(self.w, self.wd[g])", "_, bar_wd, delta_wd = hypergradient(self.w, self.lr[g])"),
    ("meta_update(self.vel_wd[g], bar_wd, delta_wd, self.beta, 0.0, self.lam)", "meta_update(self.vel_wd[g], bar_wd, delta_wd, self.beta, gamma, self.lam)"),
    ("meta_update(self.vel_wd[g], bar_wd, delta_wd, self.beta, 0.0, self.lam)", "meta_update(self.vel[g], bar_wd, delta_wd, self.beta, 0.0, self.lam)"),
    ("wd[g][r] = self.wd_base[g] * rho_wd[self.perm_wd[g][r]]", "wd[g][r] = self.weight_decay[g] * rho_wd[self.perm_wd[g][r]]"),
    # SGD extension
    ("g_eff = g + wd * theta", "g_eff = g - wd * theta"),
    ("buf[...] = mu * buf + g_eff", "buf[...] = mu * buf + (1 - mu) * g_eff"),
    ("theta -= lr * buf", "theta -= lr * g_eff"),
    ("sgd_momentum_update(th[r], self.m[k][r], g_r, lr[g_id][r], wd[g_id][r], self.momentum)",
     "sgd_momentum_update(th[r], self.m[k][0], g_r, lr[g_id][r], wd[g_id][r], self.momentum)"),
    # Eq. 10
    ("return nu * math.sqrt(norm2 / d)", "return nu * math.sqrt(norm2) / d"),
    ("return nu * math.sqrt(norm2 / d)", "return nu * norm2 / d"),
    ("radius = math.sqrt(-2.0 * math.log(u1))", "radius = math.sqrt(-math.log(u1))"),
    ("u2 = ((u >> 16) & 0xFFFFFF) / 16777216.0", "u2 = ((u >> 41) & 0xFFFFFF) / 16777216.0"),
    ("out[j] = radius * (math.cos(2.0 * math.pi * u2) if e % 2 == 0 else math.sin(2.0 * math.pi * u2))",
     "out[j] = radius * math.cos(2.0 * math.pi * u2)"),
    ("u = mix64(key + (e // 2) * 0x9E3779B97F4A7C15)", "u = mix64(key + j * 0x9E3779B97F4A7C15)"),
    ("out[r] = t0 + sigma * warm_noise(seed, r, tensor, start, t0.size)", "out[r] = t0 + sigma * warm_noise(seed, 0, tensor, start, t0.size)"),
    ("out[r] = t0 + sigma * warm_noise(seed, r, tensor, start, t0.size)", "out[r] = t0 * (1 + sigma * warm_noise(seed, r, tensor, start, t0.size))"),
    ("if self.grad_mean and gk.ndim == 2:", "if False:"),
    ("self.v[k][r], g_r, lr[g_id][r], wd[g_id][r],", "self.v[k][r], g_r, lr[g_id][r], self.weight_decay[g_id],"),
    ("g_r, lr[g_id][r], wd[g_id][r], self.momentum)", "g_r, lr[g_id][r], self.weight_decay[g_id], self.momentum)"),
    # bfloat16 copy of the averaged parameters
    ("return ((u + np.uint64(0x7FFF) + keep_lsb) >> np.uint64(16)).astype(np.uint16)",
     "return (u >> np.uint64(16)).astype(np.uint16)"),
    ("return ((u + np.uint64(0x7FFF) + keep_lsb) >> np.uint64(16)).astype(np.uint16)",
     "return ((u + np.uint64(0x8000)) >> np.uint64(16)).astype(np.uint16)"),
    ("return bf16_bits(theta[0].astype(np.float32))", "return bf16_bits(theta[0].astype(np.float32) * 2)"),
]


def _pin_calls():
    """Every pin test as a zero-argument callable (parametrised tests expanded)."""
    calls = []
    for name, fn in sorted(vars(pins).items()):
        if not (name.startswith("test_") and callable(fn)):
            continue
        marks = [m for m in getattr(fn, "pytestmark", []) if m.name == "parametrize"]
        if not marks:
            calls.append((name, fn, {}))
            continue
        axes = []
        for m in marks:
            names = [a.strip() for a in m.args[0].split(",")]
            axes.append([dict(zip(names, v if len(names) > 1 else (v,))) for v in m.args[1]])
        for combo in itertools.product(*axes):
            kw = {}
            for d in combo:
                kw.update(d)
            calls.append((name, fn, kw))
    return calls


def _mutant_module(old, new):
    assert SOURCE.count(old) == 1, f"mutation site not unique or missing: {old!r}"
    mod = types.ModuleType("hdet_oracle_mutant")
    exec(compile(SOURCE.replace(old, new), "<mutant>", "exec"), mod.__dict__)
    return mod


def test_unmutated_oracle_passes_through_the_same_driver():
    for name, fn, kw in _pin_calls():
        fn(**kw)


@pytest.mark.parametrize("idx", range(len(MUTANTS)))
def test_every_planted_mistake_fails_a_pin(idx, monkeypatch):
    old, new = MUTANTS[idx]
    monkeypatch.setattr(pins, "O", _mutant_module(old, new))
    caught = None
    for name, fn, kw in _pin_calls():
        try:
            fn(**kw)
        except Exception as e:  # an assertion or an arithmetic error both count as caught
            caught = (name, type(e).__name__)
            break
    assert caught is not None, f"mutant survived all pins: {old!r} -> {new!r}"
