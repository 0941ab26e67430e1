"""Pins of the CPU oracle against what the paper and the mathematics fix (no GPU needed).

Each test checks an oracle function against something other than itself: values the
paper prints, closed forms, invariants, a library routine on a special case, or brute force.
"""
import itertools
import math
import os
from fractions import Fraction

import numpy as np
import pytest
import torch

from oracle import hdet_oracle as O

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def _read_kv(name):
    out = {}
    with open(os.path.join(GOLDEN, name)) as f:
        for line in f:
            line = line.strip()
            if not line or line.startswith("#"):
                continue
            k, v = line.split(None, 1)
            out[k] = v
    return out


# ----------------------------------------------------------------------------- Eq. 1
def test_eq1_worked_example_from_the_paper():
    kv = _read_kv("eq1_worked_example.txt")
    n = int(kv["n"])
    alpha = int(kv["alpha_num"]) / int(kv["alpha_den"])
    eta = float(kv["eta"])
    lrs = eta * O.spread_multipliers(n, alpha)
    assert lrs[0] == pytest.approx(float(kv["lr_min"]), rel=1e-13)
    assert lrs[-1] == pytest.approx(float(kv["lr_max"]), rel=1e-13)
    assert lrs.mean() == pytest.approx(float(kv["lr_mean"]), rel=1e-13)
    assert lrs.min() == lrs[0] and lrs.max() == lrs[-1]
    assert np.all(np.diff(lrs) > 0)


def test_eq1_figure1_endpoints():
    n = None
    rows = []
    with open(os.path.join(GOLDEN, "fig1_endpoints.txt")) as f:
        for line in f:
            p = line.split()
            if not p or p[0].startswith("#"):
                continue
            if p[0] == "n":
                n = int(p[1])
            else:
                rows.append((int(p[1]), float(p[3]), float(p[5])))
    for alpha in (0.05, 1 / 9, 0.5):
        rho = O.spread_multipliers(n, alpha)
        for rank, c0, c1 in rows:
            assert rho[rank] == pytest.approx(c0 + c1 * alpha, rel=1e-14)


@pytest.mark.parametrize("n", [1, 2, 3, 4, 7, 8, 16, 31, 32])
@pytest.mark.parametrize("alpha", [0.0, 1 / 9, 0.2, 0.3, 0.5, 0.99])
def test_eq1_sum_range_symmetry_and_exact_rational(n, alpha):
    rho = O.spread_multipliers(n, alpha)
    assert rho.shape == (n,)
    assert rho.sum() == pytest.approx(n, rel=1e-14)
    assert rho.min() >= 1 - alpha - 1e-15 and rho.max() <= 1 + alpha + 1e-15
    for r in range(n):  # symmetric around 1
        assert rho[r] + rho[n - 1 - r] == pytest.approx(2.0, rel=1e-14)
    # exact rational evaluation of Eq. 1, written independently with Fractions
    a = Fraction(alpha)
    delta = max(Fraction(n - 1, 2), Fraction(1, 2))
    for r in range(n):
        exact = 1 + a * (Fraction(r) - Fraction(n - 1, 2)) / delta
        assert rho[r] == pytest.approx(float(exact), rel=1e-14, abs=1e-15)
    if n >= 2:
        assert rho[0] == pytest.approx(1 - alpha, rel=1e-14)
        assert rho[-1] == pytest.approx(1 + alpha, rel=1e-14)


def test_eq1_degenerate_sizes():
    assert list(O.spread_multipliers(1, 0.3)) == [1.0]
    r2 = O.spread_multipliers(2, 0.3)
    assert r2[0] == pytest.approx(0.7) and r2[1] == pytest.approx(1.3)
    assert np.all(O.spread_multipliers(8, 0.0) == 1.0)


# ----------------------------------------------------------------------------- one-cycle schedule
@pytest.mark.parametrize("kind", [O.SCHED_ONECYCLE_COS, O.SCHED_ONECYCLE_LINEAR])
def test_onecycle_closed_form_points(kind):
    S, p, mx, div, fdiv = 1000, 0.3, 3e-4, 25.0, 1e4
    f = lambda i: O.onecycle_lr(i, S, mx, p, div, fdiv, kind)
    assert f(0) == pytest.approx(mx / div, rel=1e-14)
    assert f(299) == pytest.approx(mx, rel=1e-14)          # p*S - 1 = 299
    assert f(S - 1) == pytest.approx(mx / (div * fdiv), rel=1e-10)
    vals = np.array([f(i) for i in range(S)])
    assert np.all(np.diff(vals[:300]) > 0) and np.all(np.diff(vals[299:]) < 0)
    # midpoint of each phase: cosine and linear both pass through the average of the ends
    S2 = 201  # phases [0, 59.3] and [59.3, 200]
    up_end = 0.3 * S2 - 1
    g = lambda x: O.onecycle_lr(x, S2, mx, 0.3, div, fdiv, kind)
    assert g(up_end / 2) == pytest.approx((mx / div + mx) / 2, rel=1e-13)
    mid2 = (up_end + (S2 - 1)) / 2
    assert g(mid2) == pytest.approx((mx + mx / (div * fdiv)) / 2, rel=1e-13)


@pytest.mark.parametrize("S,p", [(1000, 0.3), (500, 0.3), (50, 0.3), (300, 0.3), (37, 0.41), (16, 0.25)])
@pytest.mark.parametrize("kind,name", [(O.SCHED_ONECYCLE_COS, "cos"), (O.SCHED_ONECYCLE_LINEAR, "linear")])
def test_onecycle_matches_the_library_scheduler(S, p, kind, name):
    """Cross-check against the scheduler the paper names (a library routine, not oracle code)."""
    mx, div, fdiv = 3e-4, 25.0, 1e4
    prm = torch.nn.Parameter(torch.zeros(1, dtype=torch.float64))
    opt = torch.optim.SGD([prm], lr=1.0)
    sch = torch.optim.lr_scheduler.OneCycleLR(opt, max_lr=mx, total_steps=S, pct_start=p, anneal_strategy=name,
                                              cycle_momentum=False, div_factor=div, final_div_factor=fdiv)
    for i in range(S):
        lib = opt.param_groups[0]["lr"]
        assert O.onecycle_lr(i, S, mx, p, div, fdiv, kind) == pytest.approx(lib, rel=1e-12, abs=1e-20), i
        opt.step()
        if i < S - 1:
            sch.step()


def test_base_lr_constant():
    assert O.base_lr(O.SCHED_CONSTANT, 5, 16, 1e-2, 0.3, 25.0, 1e4) == 1e-2


# ----------------------------------------------------------------------------- Eq. 2 / Adam
def test_sgd_matches_library_and_closed_form():
    rng = np.random.default_rng(0)
    th0 = rng.normal(size=257)
    gs = rng.normal(size=(5, 257))
    lrs = [0.1, 0.05, 0.2, 0.01, 0.3]
    th = th0.copy()
    for g, lr in zip(gs, lrs):
        O.sgd_update(th, g, lr)
    # closed form: theta_k = theta_0 - sum_i lr_i g_i
    assert np.allclose(th, th0 - np.tensordot(lrs, gs, axes=1), rtol=1e-13, atol=1e-15)
    p = torch.nn.Parameter(torch.tensor(th0))
    opt = torch.optim.SGD([p], lr=0.1)
    for g, lr in zip(gs, lrs):
        opt.param_groups[0]["lr"] = lr
        p.grad = torch.tensor(g)
        opt.step()
    assert np.allclose(th, p.detach().numpy(), rtol=1e-13, atol=1e-15)


@pytest.mark.parametrize("wd", [0.0, 0.01, 0.3])
def test_adamw_matches_library_in_float64(wd):
    rng = np.random.default_rng(1)
    n, steps = 301, 25
    th0 = rng.normal(scale=0.02, size=n)
    b1, b2, eps = 0.9, 0.999, 1e-8
    th, m, v = th0.copy(), np.zeros(n), np.zeros(n)
    p = torch.nn.Parameter(torch.tensor(th0))
    opt = torch.optim.AdamW([p], lr=1e-3, betas=(b1, b2), eps=eps, weight_decay=wd)
    for t in range(1, steps + 1):
        g = rng.normal(scale=1e-3, size=n)
        lr = 1e-4 * (1 + t % 7)
        O.adamw_update(th, m, v, g, lr, wd, b1, b2, eps, t)
        opt.param_groups[0]["lr"] = lr
        p.grad = torch.tensor(g)
        opt.step()
        st = opt.state[p]
        assert np.allclose(th, p.detach().numpy(), rtol=1e-12, atol=1e-18)
        assert np.allclose(m, st["exp_avg"].numpy(), rtol=1e-12, atol=1e-30)
        assert np.allclose(v, st["exp_avg_sq"].numpy(), rtol=1e-12, atol=1e-30)


def test_adamw_first_step_closed_form():
    th0 = np.array([0.5, -0.25, 0.125, 1.0])
    g = np.array([1e-3, -2e-3, 0.0, 4.0])
    lr, wd, eps = 1e-2, 0.1, 1e-8
    th, m, v = th0.copy(), np.zeros(4), np.zeros(4)
    O.adamw_update(th, m, v, g, lr, wd, 0.9, 0.999, eps, 1)
    expect = th0 * (1 - lr * wd) - lr * g / (np.abs(g) + eps)
    assert np.allclose(th, expect, rtol=1e-12, atol=1e-18)
    assert np.allclose(m, 0.1 * g, rtol=1e-13) and np.allclose(v, 0.001 * g * g, rtol=1e-12)


def test_adamw_constant_gradient_closed_form():
    """With a constant gradient the bias-corrected moments are g and g^2 at every step."""
    g = np.array([3e-3, -1e-4, 2.0])
    th0 = np.array([0.1, 0.2, 0.3])
    th, m, v = th0.copy(), np.zeros(3), np.zeros(3)
    lrs = [1e-3, 2e-3, 5e-4, 1e-4, 3e-3, 1e-3]
    for t, lr in enumerate(lrs, 1):
        O.adamw_update(th, m, v, g, lr, 0.0, 0.9, 0.999, 1e-8, t)
    expect = th0 - sum(lrs) * g / (np.abs(g) + 1e-8)
    assert np.allclose(th, expect, rtol=1e-11)


def test_adamw_decay_only_when_gradient_is_zero():
    th0 = np.array([1.0, -2.0])
    th, m, v = th0.copy(), np.zeros(2), np.zeros(2)
    for t in range(1, 4):
        O.adamw_update(th, m, v, np.zeros(2), 0.1, 0.5, 0.9, 0.999, 1e-8, t)
    assert np.allclose(th, th0 * (1 - 0.05) ** 3, rtol=1e-14)


# ----------------------------------------------------------------------------- Eq. 3
def test_converge_brute_force_idempotent_and_order_invariant():
    rng = np.random.default_rng(2)
    th = rng.normal(size=(5, 17))
    ref = [[sum(th[r][j] for r in range(5)) / 5 for j in range(17)] for _ in range(5)]
    a = th.copy()
    O.converge(a)
    assert np.allclose(a, np.array(ref), rtol=1e-14)
    assert np.all(a == a[0])
    b = a.copy()
    O.converge(b)
    assert np.allclose(a, b, rtol=1e-15)
    c = th[[3, 0, 4, 1, 2]].copy()
    O.converge(c)
    assert np.allclose(a, c, rtol=1e-14)


# ----------------------------------------------------------------------------- Eq. 4 - Eq. 6
def test_softmax_weights_properties():
    L = [3.1, 2.9, 3.05, 2.7, 3.3]
    w = O.softmax_weights(L, 0.1)
    assert w.sum() == pytest.approx(1.0, rel=1e-15)
    assert np.argmax(w) == 3 and np.argmin(w) == 4            # lowest loss, highest weight
    w_shift = O.softmax_weights([x + 123.0 for x in L], 0.1)
    assert np.allclose(w, w_shift, rtol=1e-10)
    # ratio of two weights: w_a / w_b = exp((L_b - L_a)/sigma)
    assert w[1] / w[0] == pytest.approx(math.exp((3.1 - 2.9) / 0.1), rel=1e-12)
    assert np.allclose(O.softmax_weights([2.5] * 7, 0.1), 1 / 7, rtol=1e-15)
    # no overflow for a huge loss gap
    w_big = O.softmax_weights([0.0, 1e4], 0.1)
    assert w_big[0] == pytest.approx(1.0) and w_big[1] == 0.0


def test_hypergradient_two_replica_closed_form():
    for b, alpha, L0, L1, sigma in [(1e-3, 0.3, 3.0, 2.8, 0.1), (9e-4, 1 / 9, 2.0, 2.5, 0.2), (0.01, 0.5, 1.0, 1.0, 0.1)]:
        eta = b * O.spread_multipliers(2, alpha)
        w = O.softmax_weights([L0, L1], sigma)
        tilde, bar, delta = O.hypergradient(w, eta)
        assert bar == pytest.approx(b, rel=1e-14)
        assert delta == pytest.approx(b * alpha * math.tanh((L0 - L1) / (2 * sigma)), rel=1e-11, abs=1e-20)
        assert tilde == pytest.approx(bar + delta, rel=1e-14)


def test_hypergradient_sign_rule_and_zero_for_equal_losses():
    eta = 1e-3 * O.spread_multipliers(8, 0.3)
    better_high = 3.0 - 0.1 * np.linspace(-1, 1, 8)    # higher rate, lower loss
    assert O.hypergradient(O.softmax_weights(better_high, 0.1), eta)[2] > 0
    assert O.hypergradient(O.softmax_weights(better_high[::-1], 0.1), eta)[2] < 0
    d = O.hypergradient(O.softmax_weights([2.0] * 8, 0.1), eta)[2]
    assert abs(d) < 1e-18
    # a permuted assignment of rates: Delta still positive when losses follow the rates
    perm = [3, 7, 0, 5, 1, 6, 2, 4]
    assert O.hypergradient(O.softmax_weights(better_high[perm], 0.1), eta[perm])[2] > 0


# ----------------------------------------------------------------------------- Eq. 7 - Eq. 8
def test_meta_update_hand_computed():
    v_new, base = O.meta_update(0.002, 0.01, 0.001, 0.9, 0.1, 0.5)
    assert v_new == pytest.approx(0.0019, rel=1e-13)          # 0.9*0.002 + 0.1*0.001
    assert base == pytest.approx(0.00995, rel=1e-13)          # 0.01*0.9 + 0.0019*0.5


@pytest.mark.parametrize("S,Sw,T,fd,ff", [(1000, 300, 50, 25.0, 1.0), (500, 150, 100, 25.0, 1.0), (300, 90, 7, 10.0, 0.5)])
def test_gamma_reaches_the_floor_after_K_intervals(S, Sw, T, fd, ff):
    gamma = O.decay_gamma(fd, ff, S, Sw, T)
    K = (S - Sw) / T
    assert (1 - gamma) ** K == pytest.approx(ff / fd, rel=1e-12)
    assert 0 < gamma < 1
    # with equal losses (Delta = 0) and v = 0 the base decays by exactly (1 - gamma) per firing
    base, v = 3e-4, 0.0
    for _ in range(int(K)):
        v, base = O.meta_update(v, base, 0.0, 0.9, gamma, 0.5)
    assert v == 0.0
    assert base == pytest.approx(3e-4 * (ff / fd) ** (int(K) / K), rel=1e-12)


def test_gamma_degenerate():
    assert O.decay_gamma(25.0, 1.0, 100, 100, 10) == 0.0
    assert O.decay_gamma(25.0, 1.0, 100, 200, 10) == 0.0
    assert O.decay_gamma(1.0, 1.0, 100, 0, 10) == 0.0
    # literal formula: f_div < f_final gives growth (gamma < 0)
    assert O.decay_gamma(1.0, 25.0, 100, 0, 10) < 0


# ----------------------------------------------------------------------------- Eq. 9
def test_mix64_published_vector():
    vals = []
    with open(os.path.join(GOLDEN, "splitmix64_vector.txt")) as f:
        for line in f:
            line = line.strip()
            if not line or line.startswith("#"):
                continue
            vals.append(line)
    state = int(vals[0].split()[1])
    for k, expect in enumerate(vals[1:], 1):
        assert O.mix64(state + k * 0x9E3779B97F4A7C15) == int(expect)


def test_permutation_is_valid_independent_and_unbiased():
    n = 8
    seen = set()
    counts = np.zeros((n, n))
    trials = 4000
    for k in range(trials):
        p = O.permutation(7, k, 0, n)
        assert sorted(p) == list(range(n))
        seen.add(tuple(p))
        for pos, val in enumerate(p):
            counts[pos][val] += 1
    assert len(seen) > trials * 0.9                       # 8! = 40320 possibilities
    expected = trials / n
    chi2 = ((counts - expected) ** 2 / expected).sum()
    assert chi2 < 120                                     # 49 degrees of freedom; P(chi2 > 120) ~ 1e-7
    # channels and seeds give different draws; the same key repeats
    a = [tuple(O.permutation(7, k, 0, n)) for k in range(50)]
    b = [tuple(O.permutation(7, k, 1, n)) for k in range(50)]
    c = [tuple(O.permutation(8, k, 0, n)) for k in range(50)]
    assert sum(x == y for x, y in zip(a, b)) < 5 and sum(x == y for x, y in zip(a, c)) < 5
    assert O.permutation(7, 3, 2, n) == O.permutation(7, 3, 2, n)
    assert O.permutation(1, 1, 0, 1) == [0]
    # all 6 permutations of 3 elements occur, about equally often
    from collections import Counter
    c3 = Counter(tuple(O.permutation(1, k, 0, 3)) for k in range(6000))
    assert len(c3) == 6 and min(c3.values()) > 850


def test_permutation_follows_its_written_definition():
    """Fisher-Yates from the identity with the documented draws, replayed with explicit swaps."""
    seed, k, ch, n = 5, 9, 3, 6
    key = O.mix64(O.mix64(O.mix64(seed) + k) + ch)
    draws = {j: O.mix64(key + j * 0x9E3779B97F4A7C15) % (j + 1) for j in range(1, n)}
    arr = np.arange(n)
    for j in range(n - 1, 0, -1):
        arr[[j, draws[j]]] = arr[[draws[j], j]]
    assert list(arr) == O.permutation(seed, k, ch, n)


# ----------------------------------------------------------------------------- Algorithm 1
def _mk(n, numels, groups, G, **kw):
    rng = np.random.default_rng(3)
    params = []
    for ne in numels:
        p0 = rng.normal(scale=0.02, size=ne)
        params.append(np.tile(p0, (n, 1)))
    base = dict(optimizer=O.ADAMW, total_steps=40, sched_kind=O.SCHED_ONECYCLE_COS, max_lr=[3e-4] * G,
                weight_decay=[0.01] * G, alpha_lr=0.3, sync_interval=5, seed=1)
    base.update(kw)
    return O.HdetOracle(params, groups, G, **base)


def test_alg1_alpha_zero_keeps_replicas_identical_and_equals_one_replica():
    rng = np.random.default_rng(4)
    many = _mk(4, [33, 5], [0, 0], 1, alpha_lr=0.0, sync_interval=3)
    one = _mk(1, [33, 5], [0, 0], 1, alpha_lr=0.0, sync_interval=3)
    for i in range(10):
        gs = [rng.normal(scale=1e-3, size=33), rng.normal(scale=1e-3, size=5)]
        many.step(gs)          # shared gradient (Eq. 2)
        one.step(gs)
        for k in range(2):
            assert np.all(many.theta[k] == many.theta[k][0])
            assert np.allclose(many.theta[k][0], one.theta[k][0], rtol=1e-14, atol=1e-20)


def test_alg1_sgd_shared_gradient_mean_is_one_trajectory_at_base_rate():
    rng = np.random.default_rng(5)
    n, ne, T, S = 6, 19, 4, 13
    o = _mk(n, [ne], [0], 1, optimizer=O.SGD, alpha_lr=0.4, sync_interval=T, total_steps=S, weight_decay=[0.0])
    ref = o.theta[0][0].copy()
    for i in range(S):
        g = rng.normal(size=ne)
        ended = o.step([g])
        ref -= O.onecycle_lr(i, S, 3e-4, 0.3, 25.0, 1e4, O.SCHED_ONECYCLE_COS) * g
        assert np.allclose(o.theta[0].mean(axis=0), ref, rtol=1e-12, atol=1e-18)
        assert ended == ((i + 1) % T == 0)
        if ended:   # after a sync all ranks hold the same model (Algorithm 1, Return)
            assert np.all(o.theta[0] == o.theta[0][0])
            assert np.allclose(o.theta[0][0], ref, rtol=1e-12, atol=1e-18)
    # between syncs replicas really differ
    o2 = _mk(n, [ne], [0], 1, optimizer=O.SGD, alpha_lr=0.4, sync_interval=T, total_steps=S, weight_decay=[0.0])
    o2.step([np.ones(ne)])
    assert not np.allclose(o2.theta[0][0], o2.theta[0][-1])


def test_alg1_first_update_uses_schedule_index_zero_and_eq1_rates():
    n = 4
    o = _mk(n, [3], [0], 1, optimizer=O.SGD, alpha_lr=0.2, sync_interval=100, total_steps=50, weight_decay=[0.0])
    th0 = o.theta[0].copy()
    o.step([np.ones(3)])
    rho = [0.8, 1 - 0.2 / 3, 1 + 0.2 / 3, 1.2]
    for r in range(n):
        assert np.allclose(th0[r] - o.theta[0][r], (3e-4 / 25.0) * rho[r], rtol=1e-12)
    assert o.lr.mean(axis=1)[0] == pytest.approx(o.base[0], rel=1e-14)


def test_alg1_moments_are_not_averaged_and_params_are():
    rng = np.random.default_rng(6)
    o = _mk(3, [11], [0], 1, sync_interval=2)
    for i in range(2):
        o.step([rng.normal(scale=1e-3, size=(3, 11))])
    assert np.all(o.theta[0] == o.theta[0][0])
    assert not np.allclose(o.m[0][0], o.m[0][1])
    assert not np.allclose(o.v[0][0], o.v[0][1], rtol=1e-6, atol=0.0)


def test_alg1_loss_accumulator_is_the_mean_of_the_last_round():
    o = _mk(2, [4], [0], 1, sync_interval=3, autolr=True, warmup_steps=1000)
    losses = [[1.0, 2.0], [2.0, 4.0], [3.0, 6.0], [10.0, 20.0], [20.0, 40.0], [30.0, 60.0]]
    for i, L in enumerate(losses):
        o.step([np.zeros(4)], L)
        if i == 2:
            assert np.allclose(o.L_round, [2.0, 4.0])
        if i == 5:
            assert np.allclose(o.L_round, [20.0, 40.0])
    assert not o.fired


def test_alg1_controller_timing_hold_and_first_bar():
    S, T, Sw, n = 40, 5, 12, 4
    o = _mk(n, [4], [0], 1, sync_interval=T, total_steps=S, autolr=True, warmup_steps=Sw, alpha_lr=0.3,
            reshuffle=False)
    gamma = O.decay_gamma(25.0, 1.0, S, Sw, T)
    bases = []
    for i in range(S):
        L = 3.0 - 0.1 * np.linspace(-1, 1, n)
        o.step([np.zeros(4)], L)
        bases.append(o.base[0])
        t = i + 1
        assert o.fired == (t >= 15)              # first sync with t >= 12 is t = 15
        if t < 15 or i < 15:
            assert o.base[0] == pytest.approx(O.onecycle_lr(i, S, 3e-4), rel=1e-14)
    # first firing: eta_bar is the schedule value of the last update (index 14)
    w = O.softmax_weights(3.0 - 0.1 * np.linspace(-1, 1, n), 0.1)
    b14 = O.onecycle_lr(14, S, 3e-4)
    delta = float(np.sum(w * b14 * O.spread_multipliers(n, 0.3))) - b14
    assert delta > 0
    v1 = 0.1 * delta
    assert bases[15] == pytest.approx(b14 * (1 - gamma) + 0.5 * v1, rel=1e-12)
    # held constant for the T updates of the round, then changed
    assert all(bases[i] == bases[15] for i in range(15, 20))
    assert bases[20] != bases[15]
    v2 = 0.9 * v1 + 0.1 * (float(np.sum(w * bases[15] * O.spread_multipliers(n, 0.3))) - bases[15])
    assert bases[20] == pytest.approx(bases[15] * (1 - gamma) + 0.5 * v2, rel=1e-12)


def test_alg1_equal_losses_decay_the_base_to_the_floor_ratio():
    S, T, Sw = 60, 5, 10
    o = _mk(4, [2], [0, ], 1, sync_interval=T, total_steps=S, autolr=True, warmup_steps=Sw)
    for i in range(S):
        o.step([np.zeros(2)], [2.5] * 4)
    # firings at t = 10, 15, ..., 60: 11 of them; K = 10 intervals
    b9 = O.onecycle_lr(9, S, 3e-4)
    assert abs(o.vel[0]) < 1e-19 and abs(o.delta[0]) < 1e-19
    assert o.ctrl_base[0] == pytest.approx(b9 * (1.0 / 25.0) ** (11 / 10), rel=1e-11)


def test_alg1_permutations_only_after_firing_and_independent_per_channel():
    n, G = 8, 3
    o = _mk(n, [2, 2, 2], [0, 1, 2], G, sync_interval=2, total_steps=20, autolr=True, warmup_steps=6,
            alpha_wd=0.5, weight_decay=[0.05, 0.0, 0.1])
    ident = list(range(n))
    for i in range(12):
        o.step([np.zeros(2)] * 3, [3.0] * n)
        t = i + 1
        if t < 6:
            assert all(p == ident for p in o.perm_lr + o.perm_wd)
    chans = [tuple(p) for p in o.perm_lr + o.perm_wd]
    assert len(set(chans)) == len(chans)                                # independent draws per channel
    base, lr, wd = o.tables()
    rho = O.spread_multipliers(n, 0.3)
    for g in range(G):
        assert sorted(lr[g] / base[g]) == pytest.approx(sorted(rho), rel=1e-13)   # a permutation of rho
        assert lr[g].mean() == pytest.approx(base[g], rel=1e-14)                  # mean of the spread = base
        assert wd[g].mean() == pytest.approx(o.weight_decay[g], rel=1e-14, abs=1e-20)
        assert lr[g][0] == pytest.approx(base[g] * rho[o.perm_lr[g][0]], rel=1e-14)
        # multipliers grow with their index, so each table is ordered like ITS OWN permutation
        assert list(np.argsort(lr[g])) == list(np.argsort(o.perm_lr[g]))
        if o.weight_decay[g] > 0:
            assert list(np.argsort(wd[g])) == list(np.argsort(o.perm_wd[g]))
            assert sorted(wd[g] / o.weight_decay[g]) == pytest.approx(sorted(O.spread_multipliers(n, 0.5)), rel=1e-13)
    assert np.all(wd[1] == 0.0)


def test_alg1_autolr_off_never_fires_and_keeps_identity():
    o = _mk(4, [2], [0], 1, sync_interval=2, total_steps=10, autolr=False)
    for i in range(10):
        o.step([np.zeros(2)], [3.0, 2.0, 1.0, 0.5])
        assert o.base[0] == pytest.approx(O.onecycle_lr(i, 10, 3e-4), rel=1e-14)
    assert not o.fired and o.perm_lr[0] == [0, 1, 2, 3]


def test_alg1_per_replica_rates_match_per_replica_library_runs():
    """Each replica between syncs is an ordinary AdamW run at its own rate and decay."""
    rng = np.random.default_rng(8)
    n, ne, steps = 4, 9, 4
    o = _mk(n, [ne], [0], 1, sync_interval=100, total_steps=50, alpha_lr=0.3, alpha_wd=0.5, weight_decay=[0.05])
    th0 = o.theta[0][0].copy()
    grads = rng.normal(scale=1e-3, size=(steps, n, ne))
    for i in range(steps):
        o.step([grads[i]])
    rho = O.spread_multipliers(n, 0.3)
    rho_wd = O.spread_multipliers(n, 0.5)
    for r in range(n):
        p = torch.nn.Parameter(torch.tensor(th0))
        opt = torch.optim.AdamW([p], lr=1.0, betas=(0.9, 0.999), eps=1e-8, weight_decay=0.05 * rho_wd[r])
        for i in range(steps):
            opt.param_groups[0]["lr"] = O.onecycle_lr(i, 50, 3e-4) * rho[r]
            p.grad = torch.tensor(grads[i][r])
            opt.step()
        assert np.allclose(o.theta[0][r], p.detach().numpy(), rtol=1e-12, atol=1e-18)


def test_alg1_controller_is_homogeneous_per_group():
    """Eq. 5 - Eq. 7 are linear in the rates: a group whose rates are doubled gets twice Delta, v and eta_bar."""
    n = 4
    o = _mk(n, [2, 2], [0, 1], 2, sync_interval=3, total_steps=30, autolr=True, warmup_steps=3, reshuffle=False,
            max_lr=[3e-4, 6e-4], weight_decay=[0.0, 0.0])
    for i in range(9):
        o.step([np.zeros(2)] * 2, 3.0 - 0.1 * np.linspace(-1, 1, n) + 0.01 * i)
    assert o.fired and o.delta[0] > 0
    assert o.delta[1] == pytest.approx(2 * o.delta[0], rel=1e-12)
    assert o.vel[1] == pytest.approx(2 * o.vel[0], rel=1e-12)
    assert o.ctrl_base[1] == pytest.approx(2 * o.ctrl_base[0], rel=1e-12)


def test_alg1_gradient_mean_equals_a_run_with_the_mean_given_as_shared_gradient():
    """Algorithm 1's gradient AllReduce: stepping with grad_mean on g_r is stepping on the shared mean of the g_r."""
    rng = np.random.default_rng(12)
    n = 5
    a = _mk(n, [13, 4], [0, 0], 1, sync_interval=3, grad_mean=True)
    b = _mk(n, [13, 4], [0, 0], 1, sync_interval=3)
    for i in range(7):
        gs = [rng.normal(scale=1e-3, size=(n, 13)), rng.normal(scale=1e-3, size=(n, 4))]
        a.step(gs)
        b.step([np.array([sum(g[r][j] for r in range(n)) / n for j in range(g.shape[1])]) for g in gs])
        for k in range(2):
            assert np.allclose(a.theta[k], b.theta[k], rtol=1e-13, atol=1e-20)
            assert np.allclose(a.v[k], b.v[k], rtol=1e-12, atol=1e-30)
            # one gradient for everyone: the moments are the same on every replica
            assert np.all(a.m[k] == a.m[k][0]) and np.all(a.v[k] == a.v[k][0])


# ----------------------------------------------------------------------------- Eq. 10
def test_eq10_sigma_matches_the_stated_variance():
    rng = np.random.default_rng(20)
    ts = [rng.normal(scale=0.02, size=1000), rng.normal(scale=0.5, size=37)]
    flat = np.concatenate(ts)
    # nu^2 ||theta||^2 / d written with a library norm
    assert O.warm_sigma(ts, 0.01) ** 2 == pytest.approx(0.01 ** 2 * np.linalg.norm(flat) ** 2 / flat.size, rel=1e-12)
    assert O.warm_sigma(ts, 0.0) == 0.0
    assert O.warm_sigma([np.ones(10)], 0.01) == pytest.approx(0.01, rel=1e-14)   # unit-RMS checkpoint: sigma = nu
    assert O.warm_sigma(ts, 0.02) == pytest.approx(2 * O.warm_sigma(ts, 0.01), rel=1e-14)


def test_eq10_noise_is_standard_normal_and_independent():
    from scipy import stats
    z = O.warm_noise(3, 1, 0, 0, 40000)
    assert abs(z.mean()) < 4 / np.sqrt(z.size) and abs(z.std() - 1) < 0.02
    assert stats.kstest(z, "norm").pvalue > 1e-3                      # library normal distribution
    assert abs(stats.kurtosis(z)) < 0.1 and abs(stats.skew(z)) < 0.05
    # even and odd elements (the two Box-Muller outputs) are uncorrelated, as are replicas and tensors
    assert abs(np.corrcoef(z[0::2], z[1::2])[0, 1]) < 0.03
    assert abs(np.corrcoef(z[:10000], O.warm_noise(3, 2, 0, 0, 10000))[0, 1]) < 0.04
    assert abs(np.corrcoef(z[:10000], O.warm_noise(3, 1, 1, 0, 10000))[0, 1]) < 0.04
    assert abs(np.corrcoef(z[:10000], O.warm_noise(4, 1, 0, 0, 10000))[0, 1]) < 0.04
    # counter-based: a slab equals the same elements of a longer draw, also from an odd start
    assert np.array_equal(O.warm_noise(3, 1, 0, 1001, 50), z[1001:1051])
    # the pair shares its radius: z_even^2 + z_odd^2 = -2 ln u1 is chi-square with 2 degrees of freedom
    r2 = z[0::2] ** 2 + z[1::2] ** 2
    assert stats.kstest(r2, "chi2", args=(2,)).pvalue > 1e-3


def test_eq10_warm_init_statistics_and_limits():
    rng = np.random.default_rng(21)
    theta0 = rng.normal(scale=0.02, size=20000)
    sigma = O.warm_sigma([theta0], 0.01)
    out = O.warm_noisy_init(theta0, sigma, 9, 4, 0)
    assert out.shape == (4, 20000)
    eps = out - theta0
    assert eps.std() == pytest.approx(0.01 * np.sqrt(np.mean(theta0 ** 2)), rel=0.02)     # nu * RMS(theta_0)
    assert abs(eps.mean()) < 4 * sigma / np.sqrt(eps.size)
    assert not np.allclose(out[0], out[1])
    assert np.array_equal(O.warm_noisy_init(theta0, 0.0, 9, 4, 0), np.tile(theta0, (4, 1)))   # nu = 0: plain copies
    # linear in sigma
    out2 = O.warm_noisy_init(theta0, 2 * sigma, 9, 4, 0)
    assert np.allclose(out2 - theta0, 2 * eps, rtol=1e-9, atol=1e-16)
    # a slab of the tensor gives the same values as the whole tensor
    assert np.array_equal(O.warm_noisy_init(theta0[333:444], sigma, 9, 4, 0, start=333), out[:, 333:444])


def test_sgd_momentum_and_weight_decay_match_the_library():
    rng = np.random.default_rng(30)
    n = 101
    th0 = rng.normal(scale=0.02, size=n)
    for mu, wd in [(0.9, 0.0), (0.9, 0.05), (0.0, 0.1), (0.5, 0.01)]:
        th, buf = th0.copy(), np.zeros(n)
        p = torch.nn.Parameter(torch.tensor(th0))
        opt = torch.optim.SGD([p], lr=0.1, momentum=mu, weight_decay=wd)
        for t in range(1, 9):
            g = rng.normal(scale=1e-2, size=n)
            lr = 1e-2 * (1 + t % 3)
            O.sgd_momentum_update(th, buf, g, lr, wd, mu)
            opt.param_groups[0]["lr"] = lr
            p.grad = torch.tensor(g)
            opt.step()
            assert np.allclose(th, p.detach().numpy(), rtol=1e-12, atol=1e-18)
    # mu = wd = 0 is Eq. 2
    a, b, buf = th0.copy(), th0.copy(), np.zeros(n)
    g = rng.normal(size=n)
    O.sgd_momentum_update(a, buf, g, 0.3, 0.0, 0.0)
    O.sgd_update(b, g, 0.3)
    assert np.array_equal(a, b)


def test_alg1_sgd_momentum_per_replica_rates_match_library_runs():
    rng = np.random.default_rng(31)
    n, ne, steps = 3, 7, 5
    o = _mk(n, [ne], [0], 1, optimizer=O.SGD, sync_interval=100, total_steps=50, alpha_lr=0.3, alpha_wd=0.5,
            weight_decay=[0.05], momentum=0.9)
    th0 = o.theta[0][0].copy()
    grads = rng.normal(scale=1e-2, size=(steps, n, ne))
    for i in range(steps):
        o.step([grads[i]])
    rho, rho_wd = O.spread_multipliers(n, 0.3), O.spread_multipliers(n, 0.5)
    for r in range(n):
        p = torch.nn.Parameter(torch.tensor(th0))
        opt = torch.optim.SGD([p], lr=1.0, momentum=0.9, weight_decay=0.05 * rho_wd[r])
        for i in range(steps):
            opt.param_groups[0]["lr"] = O.onecycle_lr(i, 50, 3e-4) * rho[r]
            p.grad = torch.tensor(grads[i][r])
            opt.step()
        assert np.allclose(o.theta[0][r], p.detach().numpy(), rtol=1e-12, atol=1e-18)


def test_remark1_weight_decay_channel_controller():
    n = 4
    kw = dict(sync_interval=2, total_steps=40, autolr=True, warmup_steps=2, reshuffle=False, alpha_wd=0.5,
              weight_decay=[0.05, 0.1], max_lr=[3e-4, 3e-4])
    # identity permutation: replica r holds the r-th smallest weight decay; losses fall with r -> raise the base
    up = _mk(n, [2, 2], [0, 1], 2, auto_wd=True, **kw)
    down = _mk(n, [2, 2], [0, 1], 2, auto_wd=True, **kw)
    flat = _mk(n, [2, 2], [0, 1], 2, auto_wd=True, **kw)
    off = _mk(n, [2, 2], [0, 1], 2, auto_wd=False, **kw)
    for i in range(8):
        up.step([np.zeros(2)] * 2, 3.0 - 0.1 * np.linspace(-1, 1, n))
        down.step([np.zeros(2)] * 2, 3.0 + 0.1 * np.linspace(-1, 1, n))
        flat.step([np.zeros(2)] * 2, [3.0] * n)
        off.step([np.zeros(2)] * 2, 3.0 - 0.1 * np.linspace(-1, 1, n))
    assert up.wd_base[0] > 0.05 and down.wd_base[0] < 0.05 and up.delta_wd[0] > 0 > down.delta_wd[0]
    assert flat.wd_base == pytest.approx([0.05, 0.1], rel=1e-14)              # equal losses: nothing moves (gamma = 0)
    assert max(abs(v) for v in flat.vel_wd) < 1e-17
    assert off.wd_base == [0.05, 0.1]
    # linear in the weight decays: the group with twice the base gets twice Delta, velocity and base
    assert up.delta_wd[1] == pytest.approx(2 * up.delta_wd[0], rel=1e-12)
    assert up.wd_base[1] == pytest.approx(2 * up.wd_base[0], rel=1e-12)
    # first firing by hand: two-replica-style closed form is covered by hypergradient; here Eq. 7 with gamma = 0
    one = _mk(n, [2], [0], 1, auto_wd=True, sync_interval=2, total_steps=40, autolr=True, warmup_steps=2,
              reshuffle=False, alpha_wd=0.5, weight_decay=[0.05])
    L = 3.0 - 0.1 * np.linspace(-1, 1, n)
    for i in range(2):
        one.step([np.zeros(2)], L)
    w = O.softmax_weights(L, 0.1)
    delta = float(np.sum(w * 0.05 * O.spread_multipliers(n, 0.5))) - 0.05
    assert one.wd_base[0] == pytest.approx(0.05 + 0.5 * 0.1 * delta, rel=1e-12)
    # the tables of the next update use the new base
    _, _, wd = one.tables()
    assert wd[0].mean() == pytest.approx(one.wd_base[0], rel=1e-14)


# --------------------------------------------------------------------------- bfloat16 copy of the averaged parameters
def test_bf16_rounding_known_patterns_ties_and_the_library_conversion():
    """Round to nearest, ties to even, on the fp32 bit pattern: textbook cases, the error bound, idempotence,
    and agreement with the library's own fp32 -> bf16 conversion on random and on tie values."""
    import torch

    def f32(bits):
        return np.array(bits, dtype=np.uint32).view(np.float32)

    cases = {0x3F800000: 0x3F80,      # 1.0
             0xBF800000: 0xBF80,      # -1.0
             0x3F808000: 0x3F80,      # exactly half way above an even pattern: stays
             0x3F818000: 0x3F82,      # half way above an odd pattern: goes up to the even one
             0x3F808001: 0x3F81,      # just above half way: up
             0x3F807FFF: 0x3F80,      # just below half way: down
             0x00000000: 0x0000, 0x80000000: 0x8000,
             0x477FE000: 0x4780}      # 65504.0: the carry runs into the exponent
    got = O.bf16_bits(f32(list(cases)))
    assert got.tolist() == list(cases.values())
    rng = np.random.default_rng(5)
    x = (rng.standard_normal(200000) * 10.0 ** rng.integers(-6, 6, 200000)).astype(np.float32)
    ties = f32(((rng.integers(0, 0x7F7F, 4096, dtype=np.int64) << 16) | 0x8000).astype(np.uint32))   # finite exact ties
    for v in (x, ties):
        want = torch.from_numpy(v).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)
        assert np.array_equal(O.bf16_bits(v), want)
    back = (O.bf16_bits(x).astype(np.uint32) << 16).view(np.float32)
    assert np.all(np.abs(back.astype(np.float64) - x) <= np.abs(x.astype(np.float64)) * 2.0 ** -8)   # half an ulp of 8 bits
    assert np.array_equal(O.bf16_bits(back), O.bf16_bits(x))                                         # idempotent


def test_averaged_bf16_is_the_rounded_master_copy_of_the_mean():
    theta = np.array([[1.0, 3.0, 0.1], [2.0, 3.0, 0.3]])
    O.converge(theta)
    bits = O.averaged_bf16(theta)
    assert bits.tolist() == O.bf16_bits(np.array([1.5, 3.0, 0.2], dtype=np.float32)).tolist()
    assert bits[0] == 0x3FC0 and bits[1] == 0x4040
