"""The C-ABI library on the host: exports, argument checks, and its double-precision scalars against the oracle.

A handle created with no tensors touches no device, so all of this runs without a GPU.
"""
import ctypes as C
import os
import re

import numpy as np
import pytest

import harness as H
from hdet_inputs import recipes as R
from hdet_inputs import workloads as W
from paper_2604_24708_b200 import binding as B

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def test_library_exports_every_declared_symbol():
    names = []
    for fn in sorted(os.listdir(os.path.join(ROOT, "include"))):
        if fn.endswith(".h"):
            text = open(os.path.join(ROOT, "include", fn)).read()
            names += re.findall(r"^HDET_API\s+[\w\s\*]+?\b(hdet_\w+)\s*\(", text, flags=re.M)
    assert {"hdet_create", "hdet_set_schedule", "hdet_step", "hdet_converge", "hdet_autolr_update",
            "hdet_destroy"} <= set(names)
    lib = C.CDLL(B.LIB_PATH)
    for n in names:
        assert hasattr(lib, n), n


def test_struct_layouts_match_the_header():
    """Field offsets that the C compiler computes for include/hdet.h equal the ctypes layouts."""
    import subprocess, tempfile
    src = r'''
#include <stdio.h>
#include <stddef.h>
#include "hdet.h"
int main(void) {
  printf("%zu %zu %zu %zu\n", sizeof(hdet_tensor), sizeof(hdet_config), sizeof(hdet_schedule), sizeof(hdet_state));
  printf("%zu %zu %zu %zu\n", offsetof(hdet_tensor, group), offsetof(hdet_config, seed), offsetof(hdet_schedule, f_final), offsetof(hdet_state, gamma));
  printf("%zu %zu %zu\n", offsetof(hdet_state, lr), offsetof(hdet_state, perm_wd), offsetof(hdet_state, loss_round));
  return 0;
}'''
    with tempfile.TemporaryDirectory() as d:
        c = os.path.join(d, "t.c")
        open(c, "w").write(src)
        exe = os.path.join(d, "t")
        subprocess.run(["gcc", "-I", os.path.join(ROOT, "include"), c, "-o", exe], check=True)
        out = subprocess.run([exe], capture_output=True, text=True, check=True).stdout.split()
    got = [int(x) for x in out]
    exp = [C.sizeof(B.hdet_tensor), C.sizeof(B.hdet_config), C.sizeof(B.hdet_schedule), C.sizeof(B.hdet_state),
           B.hdet_tensor.group.offset, B.hdet_config.seed.offset, B.hdet_schedule.f_final.offset,
           B.hdet_state.gamma.offset, B.hdet_state.lr.offset, B.hdet_state.perm_wd.offset,
           B.hdet_state.loss_round.offset]
    assert got == exp


def _cfg(**kw):
    base = dict(n_replicas=4, n_groups=1, optimizer=B.HDET_OPT_ADAMW, grad_dtype=B.HDET_DTYPE_BF16, beta1=0.9,
                beta2=0.999, eps=1e-8, momentum=0.0, alpha_lr=0.2, alpha_wd=0.0, sync_interval=4, reshuffle=1,
                fuse_converge=1, seed=1, device=0)
    base.update(kw)
    return B.hdet_config(**base)


@pytest.mark.parametrize("kw", [dict(n_replicas=0), dict(n_replicas=33), dict(n_groups=0), dict(n_groups=9),
                                dict(optimizer=7), dict(grad_dtype=5), dict(alpha_lr=1.0), dict(alpha_lr=-0.1),
                                dict(alpha_wd=1.5), dict(sync_interval=0), dict(beta1=1.0), dict(eps=-1.0)])
def test_create_rejects_bad_config(kw):
    with pytest.raises(B.HdetError) as e:
        B.hdet_create(_cfg(**kw), [])
    assert e.value.status == B.HDET_ERR_INVALID_ARG and e.value.message


def test_create_rejects_momentum_and_bad_tensors_without_touching_a_device():
    for kw in (dict(momentum=0.9), dict(momentum=1.0, optimizer=B.HDET_OPT_SGD), dict(momentum=-0.1, optimizer=B.HDET_OPT_SGD)):
        with pytest.raises(B.HdetError) as e:
            B.hdet_create(_cfg(**kw), [])                  # momentum with AdamW, or out of range
        assert e.value.status == B.HDET_ERR_INVALID_ARG
    h = B.hdet_create(_cfg(momentum=0.9, optimizer=B.HDET_OPT_SGD), [])
    B.hdet_destroy(h)

    def tens(**kw):
        t = B.hdet_tensor(param=0x1000, grad=0x2000, exp_avg=0x3000, exp_avg_sq=0x4000, numel=100, param_stride=128,
                          grad_stride=128, state_stride=128, group=0)
        for k, v in kw.items():
            setattr(t, k, v)
        return t
    with pytest.raises(B.HdetError) as e:                  # SGD with momentum needs its buffer
        B.hdet_create(_cfg(momentum=0.9, optimizer=B.HDET_OPT_SGD), [tens(exp_avg=None)])
    assert e.value.status == B.HDET_ERR_INVALID_ARG
    cases = [(dict(param=None), B.HDET_ERR_INVALID_ARG), (dict(grad=None), B.HDET_ERR_INVALID_ARG),
             (dict(exp_avg=None), B.HDET_ERR_INVALID_ARG), (dict(numel=0), B.HDET_ERR_INVALID_ARG),
             (dict(group=1), B.HDET_ERR_INVALID_ARG), (dict(group=-1), B.HDET_ERR_INVALID_ARG),
             (dict(param_stride=64), B.HDET_ERR_INVALID_ARG), (dict(grad_stride=-4), B.HDET_ERR_INVALID_ARG),
             (dict(state_stride=10), B.HDET_ERR_INVALID_ARG),
             (dict(param=0x1002), B.HDET_ERR_ALIGN), (dict(grad=0x2001), B.HDET_ERR_ALIGN),
             (dict(exp_avg_sq=0x4001), B.HDET_ERR_ALIGN)]
    for kw, status in cases:
        with pytest.raises(B.HdetError) as e:
            B.hdet_create(_cfg(), [tens(**kw)])
        assert e.value.status == status, kw
    # shared moments (state_stride 0) need a gradient common to all replicas, and all tensors must agree
    with pytest.raises(B.HdetError) as e:
        B.hdet_create(_cfg(), [tens(state_stride=0)])
    assert e.value.status == B.HDET_ERR_INVALID_ARG and "shared moments" in e.value.message
    with pytest.raises(B.HdetError) as e:
        B.hdet_create(_cfg(), [tens(state_stride=0, grad_stride=0), tens(grad_stride=0)])
    assert e.value.status == B.HDET_ERR_UNSUPPORTED
    with pytest.raises(B.HdetError) as e:
        B.hdet_create(_cfg(grad_mode=7), [])
    assert e.value.status == B.HDET_ERR_INVALID_ARG
    # NULL cfg / NULL out through the raw ABI
    lib = B.raw_library()
    h = C.c_void_p()
    assert lib.hdet_create(None, None, 0, C.byref(h)) == B.HDET_ERR_INVALID_ARG
    assert lib.hdet_create(C.byref(_cfg()), None, 0, None) == B.HDET_ERR_INVALID_ARG
    assert lib.hdet_create(C.byref(_cfg()), None, 3, C.byref(h)) == B.HDET_ERR_INVALID_ARG and not h.value
    assert B.hdet_last_error(None)


def test_schedule_checks_and_call_order():
    h = B.hdet_create(_cfg(), [])
    with pytest.raises(B.HdetError) as e:
        B.hdet_step(h)
    assert e.value.status == B.HDET_ERR_STATE
    with pytest.raises(B.HdetError) as e:
        B.hdet_autolr_update(h)
    assert e.value.status == B.HDET_ERR_STATE
    bad = [dict(kind=9), dict(total_steps=0), dict(pct_start=1.0), dict(pct_start=0.001), dict(div_factor=0.0),
           dict(final_div_factor=-1.0), dict(autolr=1, sigma=0.0), dict(autolr=1, f_div=0.0),
           dict(autolr=1, f_final=-2.0), dict(autolr=1, warmup_steps=-1), dict(max_lr=[float("nan")])]
    for kw in bad:
        args = dict(kind=B.HDET_SCHED_ONECYCLE_COS, total_steps=100, max_lr=[1e-3], weight_decay=[0.0])
        args.update(kw)
        with pytest.raises(B.HdetError) as e:
            B.hdet_set_schedule(h, B.make_schedule(**args))
        assert e.value.status == B.HDET_ERR_INVALID_ARG, kw
    lib = B.raw_library()
    assert lib.hdet_set_schedule(h, None) == B.HDET_ERR_INVALID_ARG
    assert lib.hdet_set_schedule(None, None) == B.HDET_ERR_INVALID_ARG
    B.hdet_set_schedule(h, B.make_schedule(B.HDET_SCHED_CONSTANT, 10, [1e-2]))
    for i in range(3):
        assert B.hdet_step(h) is False
        with pytest.raises(B.HdetError) as e:          # not at the end of a round
            B.hdet_autolr_update(h)
        assert e.value.status == B.HDET_ERR_STATE
    assert B.hdet_step(h) is True                      # t = 4 = T
    B.hdet_autolr_update(h)                            # no-op (auto-LR off) but consumes the round
    with pytest.raises(B.HdetError):
        B.hdet_autolr_update(h)
    assert B.hdet_kernel_launches(h) == 0
    with pytest.raises(B.HdetError) as e:              # device-resident stepping needs tensors on a device
        B.hdet_step_device(h)
    assert e.value.status == B.HDET_ERR_UNSUPPORTED
    B.hdet_converge(h)                                 # nothing to do without tensors
    B.hdet_destroy(h)
    B.hdet_destroy(None)


def _scalar_run(w, steps=None):
    """Library (no tensors) and oracle (no tensors) side by side; compares every scalar at every step."""
    h = B.hdet_create(H.lib_config(B, w), [])
    B.hdet_set_schedule(h, H.lib_schedule(B, w))
    o = H.oracle_for(w, [], [])
    n, G = w.n_replicas, w.n_groups
    fired_at = None
    for i in range(steps or w.total_steps):
        perm_lib = list(B.hdet_get_state(h).perm_lr[0])[:n]
        assert perm_lib == o.perm_lr[0]
        losses = R.step_losses(w, i, perm_lib)
        ended = B.hdet_step(h, list(losses))
        ended_o = o.step([], losses)
        assert ended == ended_o
        if ended:
            B.hdet_autolr_update(h)
        st = B.hdet_get_state(h)
        H.compare_scalars(st, o, n, G)
        assert st.step == o.i
        if o.fired and fired_at is None:
            fired_at = i + 1
        if ended:
            assert np.allclose(list(st.loss_round)[:n], o.L_round, rtol=1e-13)
    st = B.hdet_get_state(h)
    B.hdet_destroy(h)
    return st, o, fired_at


def test_scalars_match_oracle_config1():
    st, o, fired = _scalar_run(W.config1())
    assert fired is None and st.base[0] == 1e-2
    lrs = list(st.lr[0])[:4]
    assert lrs[0] == pytest.approx(0.8e-2, rel=1e-14) and lrs[3] == pytest.approx(1.2e-2, rel=1e-14)


def test_scalars_match_oracle_config2_full_run():
    st, o, fired = _scalar_run(W.config2())
    assert fired == 300 and st.fired == 1
    assert st.gamma == pytest.approx(1 - 25.0 ** (-1 / 14.0), rel=1e-12)
    assert all(d > 0 for d in [st.delta[0]])           # higher rate, lower loss -> Delta > 0
    assert sorted(list(st.perm_lr[0])[:8]) == list(range(8))


def test_scalars_match_oracle_config3_and_config5():
    _scalar_run(W.config3())
    st, o, _ = _scalar_run(W.config5(10))
    assert st.fired == 1
    wd = np.array([list(st.wd[g])[:16] for g in range(4)])
    assert np.all(wd[W.GROUP_NO_DECAY] == 0.0)
    assert wd[0].min() == pytest.approx(0.025, rel=1e-12) and wd[0].max() == pytest.approx(0.075, rel=1e-12)
    _scalar_run(W.config5(1), steps=120)
    _scalar_run(W.ragged_workload())


def test_scalars_match_oracle_with_the_weight_decay_channel_controller():
    from dataclasses import replace
    st, o, fired = _scalar_run(replace(W.config5(10), auto_wd=1))
    assert fired == 90 and any(abs(st.wd_delta[g]) > 0 for g in (0, 2, 3))
    assert st.wd_base[W.GROUP_NO_DECAY] == 0.0                      # a zero base stays zero
    assert st.wd_base[0] != 0.05                                    # the base has moved
    _scalar_run(replace(W.ragged_workload(), auto_wd=1))


def test_mean_of_spread_rates_is_the_base_and_alpha_zero_is_uniform():
    w = W.config5(10)
    h = B.hdet_create(H.lib_config(B, w), [])
    B.hdet_set_schedule(h, H.lib_schedule(B, w))
    for i in range(150):
        if B.hdet_step(h, list(R.step_losses(w, i))):
            B.hdet_autolr_update(h)
        st = B.hdet_get_state(h)
        for g in range(4):
            assert np.mean(list(st.lr[g])[:16]) == pytest.approx(st.base[g], rel=1e-13)
    B.hdet_destroy(h)
    h = B.hdet_create(_cfg(alpha_lr=0.0), [])
    B.hdet_set_schedule(h, B.make_schedule(B.HDET_SCHED_ONECYCLE_LINEAR, 50, [1e-3]))
    B.hdet_step(h)
    st = B.hdet_get_state(h)
    assert len(set(list(st.lr[0])[:4])) == 1 and st.lr[0][0] == st.base[0]
    B.hdet_destroy(h)


def test_state_roundtrip_resumes_identically():
    w = W.config5(10)
    def run(upto, h):
        for i in range(upto[0], upto[1]):
            perm = list(B.hdet_get_state(h).perm_lr[0])[:16]
            if B.hdet_step(h, list(R.step_losses(w, i, perm))):
                B.hdet_autolr_update(h)
    a = B.hdet_create(H.lib_config(B, w), [])
    B.hdet_set_schedule(a, H.lib_schedule(B, w))
    run((0, 137), a)
    snap = B.hdet_get_state(a)
    b = B.hdet_create(H.lib_config(B, w), [])
    B.hdet_set_schedule(b, H.lib_schedule(B, w))
    B.hdet_set_state(b, snap)
    run((137, 260), a)
    run((137, 260), b)
    sa, sb = B.hdet_get_state(a), B.hdet_get_state(b)
    assert bytes(sa) == bytes(sb)
    bad = B.hdet_get_state(a)
    bad.perm_lr[0][0] = bad.perm_lr[0][1]
    with pytest.raises(B.HdetError) as e:
        B.hdet_set_state(b, bad)
    assert e.value.status == B.HDET_ERR_INVALID_ARG
    B.hdet_destroy(a)
    B.hdet_destroy(b)


def test_binding_fails_loudly_without_the_library(monkeypatch, tmp_path):
    """No CPU fallback: a missing libhdet.so is an import error, not a silent slow path."""
    monkeypatch.setattr(B, "LIB_PATH", str(tmp_path / "libhdet.so"))
    with pytest.raises(ImportError) as e:
        B._load()
    assert "no CPU fallback" in str(e.value)


def test_arena_refuses_to_run_without_a_device():
    import torch
    if torch.cuda.is_available():
        pytest.skip("a CUDA device is present")
    from paper_2604_24708_b200.arena import StackedArena
    with pytest.raises(RuntimeError):
        StackedArena([8], [0], 2, B.HDET_OPT_SGD, B.HDET_DTYPE_F32)
    # and a handle with tensors cannot be created without a device: the library reports the CUDA error
    t = B.hdet_tensor(param=0x1000, grad=0x2000, numel=8, param_stride=8, grad_stride=8, state_stride=8, group=0)
    cfg = _cfg(optimizer=B.HDET_OPT_SGD, grad_dtype=B.HDET_DTYPE_F32)
    with pytest.raises(B.HdetError) as e:
        B.hdet_create(cfg, [t])
    assert e.value.status == B.HDET_ERR_CUDA


def _fake_descriptors(w, grad_misalign=0):
    """Descriptors of the workload's tensors laid out like a stacked arena at fake addresses (never dereferenced)."""
    from hdet_inputs import workloads as W
    gsz = 2 if w.grad_dtype == W.DTYPE_BF16 else 4
    offs, p_pad = w.arena_offsets(), w.arena_numel()
    base = {"param": 0x7000_0000_0000, "grad": 0x7100_0000_0000 + grad_misalign, "m": 0x7200_0000_0000, "v": 0x7300_0000_0000}
    out = []
    for t, off in zip(w.tensors, offs):
        d = B.hdet_tensor(param=base["param"] + 4 * off, grad=base["grad"] + gsz * off, numel=t.numel,
                          param_stride=p_pad, grad_stride=p_pad, state_stride=p_pad, group=t.group)
        if w.optimizer == W.OPT_ADAMW:
            d.exp_avg, d.exp_avg_sq = base["m"] + 4 * off, base["v"] + 4 * off
        out.append(d)
    return out


@pytest.mark.parametrize("name", ["config1", "config2", "config3", "config4", "config5", "ragged8", "ragged4", "ragged1"])
def test_work_plan_covers_every_element_of_every_tensor_exactly_once(name):
    """Walks the tile table hdet_create builds (host arithmetic only): tiles of 2048 elements, tensor by tensor in
    order, no gap, no overlap, the last tile of a tensor ragged; the access path follows the alignment; the
    partial-sum offsets do not overlap."""
    from hdet_inputs import workloads as W
    from paper_2604_24708_b200 import from_workload
    w = {"ragged8": lambda: W.ragged_workload(align_elems=8), "ragged4": lambda: W.ragged_workload(align_elems=4),
         "ragged1": lambda: W.ragged_workload(align_elems=1)}.get(name, W.ALL_CONFIGS.get(name))()
    descs = _fake_descriptors(w)
    tt, ti, access, poffs = B.hdet_plan_tiles(from_workload.config_for(w), descs)
    covered = np.zeros(len(w.tensors), dtype=np.int64)
    expect_next = {}
    for k, j in zip(tt, ti):
        assert j == expect_next.get(k, 0)                       # tiles of a tensor come in order, none skipped or repeated
        expect_next[k] = j + 1
        lo, hi = 2048 * j, min(w.tensors[k].numel, 2048 * (j + 1))
        assert lo < hi
        covered[k] += hi - lo
    assert tt == sorted(tt)                                      # tensor by tensor
    assert covered.tolist() == [t.numel for t in w.tensors]      # every element exactly once
    assert len(tt) == sum((t.numel + 2047) // 2048 for t in w.tensors)
    gsz = 2 if w.grad_dtype == W.DTYPE_BF16 else 4
    adam = w.optimizer == W.OPT_ADAMW
    for d, a in zip(descs, access):
        vec = d.param % 16 == 0 and d.grad % (4 * gsz) == 0
        if adam:
            vec = vec and d.exp_avg % 16 == 0 and d.exp_avg_sq % 16 == 0
        bulk = vec and adam and d.grad % 16 == 0 and (d.grad_stride * gsz) % 16 == 0
        assert a == (3 if bulk else 1 if vec else 0)
    ends = [o + (t.numel + 3) // 4 * 4 for o, t in zip(poffs, w.tensors)]
    assert poffs[0] == 0 and all(o % 4 == 0 for o in poffs) and poffs[1:] == ends[:-1]


def test_work_plan_rejects_what_create_rejects_and_reports_small_capacity():
    from hdet_inputs import workloads as W
    from paper_2604_24708_b200 import from_workload
    w = W.config2()
    descs = _fake_descriptors(w)
    descs[3].numel = 0
    with pytest.raises(B.HdetError) as e:
        B.hdet_plan_tiles(from_workload.config_for(w), descs)
    assert e.value.status == B.HDET_ERR_INVALID_ARG and "tensor 3" in e.value.message
    descs = _fake_descriptors(w)
    count = C.c_int64(0)
    arr = (B.hdet_tensor * len(descs))(*descs)
    buf = (C.c_int32 * 4)()
    cfg = from_workload.config_for(w)
    assert B._lib.hdet_plan_tiles(C.byref(cfg), arr, len(descs), buf, buf, 4, C.byref(count), None, None) == B.HDET_ERR_INVALID_ARG
    assert count.value == sum((t.numel + 2047) // 2048 for t in w.tensors)


def test_entry_points_that_need_a_device_say_so_on_a_handle_without_tensors():
    """A handle without tensors runs only the scalar part: the diagnostic that launches a kernel is refused, the
    peer-mean has nothing to do, and bad arguments are still reported before any device is touched."""
    from hdet_inputs import workloads as W
    from paper_2604_24708_b200 import from_workload
    w = W.config2()
    h = B.hdet_create(from_workload.config_for(w, n_local=4, replica_offset=0), [])
    B.hdet_set_schedule(h, from_workload.schedule_for(w))
    with pytest.raises(B.HdetError) as e:
        B.hdet_selftest_bounded_wait(h)
    assert e.value.status == B.HDET_ERR_UNSUPPORTED
    B.hdet_apply_mean_peers(h, [0x1000])          # no tiles: nothing to average, no device call
    assert B.hdet_kernel_launches(h) == 0
    B.hdet_destroy(h)
    assert B._lib.hdet_apply_mean_peers(None, None, 0, None) == B.HDET_ERR_INVALID_ARG
    assert B._lib.hdet_selftest_bounded_wait(None, None) == B.HDET_ERR_INVALID_ARG


def test_bf16_copy_pointer_alignment_selects_the_path():
    from hdet_inputs import workloads as W
    from paper_2604_24708_b200 import from_workload
    w = W.ragged_workload(align_elems=8)
    for misalign, want_big in ((0, 3), (8, 1), (2, 0)):
        descs = _fake_descriptors(w)
        for d, off in zip(descs, w.arena_offsets()):
            d.param_bf16 = 0x7400_0000_0000 + 2 * off + misalign
        _, _, access, _ = B.hdet_plan_tiles(from_workload.config_for(w), descs)
        assert set(access) == {want_big}
    descs = _fake_descriptors(w)
    descs[0].param_bf16 = 0x7400_0000_0001
    with pytest.raises(B.HdetError) as e:
        B.hdet_plan_tiles(from_workload.config_for(w), descs)
    assert e.value.status == B.HDET_ERR_ALIGN
