"""GPU parity: the CUDA library, called through its C ABI, against the CPU oracle on the same seeded inputs.

Tolerances (relative error per element with denominator max(|oracle|, RMS of the oracle slab)):
1e-6 after one update, 1e-5 after a full run; schedule and controller scalars 1e-12.
"""
from dataclasses import replace

import numpy as np
import pytest

import harness as H
from hdet_inputs import generator as G
from hdet_inputs import recipes as R
from hdet_inputs import workloads as W

pytestmark = pytest.mark.gpu

TOL_ONE_STEP = 1e-6
TOL_FULL_RUN = 1e-5


def _lockstep(w, slabs, steps=None, fuse=1, shared_grad=False, check_every=None, grad_mean=False, shared_state=False,
              device_resident=False, loss_dtype="float64"):
    """Runs both sides for `steps` updates; checks after the first update, at chosen steps and at the end."""
    g = H.GpuRun(w, fuse=fuse, shared_grad=shared_grad, grad_mean=grad_mean, shared_state=shared_state,
                 device_resident=device_resident, loss_dtype=loss_dtype)
    o = H.OracleRun(w, slabs, shared_grad=shared_grad, grad_mean=grad_mean, loss_dtype=loss_dtype)
    steps = steps or w.total_steps
    worst = 0.0
    try:
        for i in range(steps):
            perm = g.perm0()
            assert perm == o.o.perm_lr[0]
            ended = g.step(perm)
            assert ended == o.step()
            if i == 0:
                worst = max(worst, H.compare_slabs(g, o, TOL_ONE_STEP))
            elif check_every and (i + 1) % check_every == 0:
                worst = max(worst, H.compare_slabs(g, o, TOL_FULL_RUN))
            if ended or i == 0:
                H.compare_scalars(g.state(), o.o, w.n_replicas, w.n_groups)
        worst = max(worst, H.compare_slabs(g, o, TOL_FULL_RUN))
        st = g.state()
        assert st.device_status == 0
        H.compare_scalars(st, o.o, w.n_replicas, w.n_groups)
    finally:
        g.close()
    return worst


def test_device_fill_matches_the_numpy_generator_bit_for_bit():
    import torch
    from hdet_inputs import device as D
    key = G.stream_key(5, G.STREAM_GRAD, 7, 3)
    n, start = 100003, 12345
    for sigma in (1e-3, 0.02):
        sc = G.scale_for_sigma(sigma)
        a = torch.empty(n, dtype=torch.float32, device="cuda")
        D.fill(a, key, start, sc)
        assert np.array_equal(a.cpu().numpy().view(np.uint32), G.fill_f32(key, start, n, sc).view(np.uint32))
        b = torch.empty(n, dtype=torch.bfloat16, device="cuda")
        D.fill(b, key, start, sc)
        assert np.array_equal(b.view(torch.int16).cpu().numpy().view(np.uint16), G.fill_bf16_bits(key, start, n, sc))


def test_config1_sgd_every_element_every_step():
    w = W.config1()
    worst = _lockstep(w, H.whole_tensor_slabs(w), check_every=1)
    assert worst <= TOL_FULL_RUN


@pytest.mark.parametrize("optimizer,grad_dtype", [(W.OPT_ADAMW, W.DTYPE_BF16), (W.OPT_ADAMW, W.DTYPE_F32),
                                                   (W.OPT_SGD, W.DTYPE_F32), (W.OPT_SGD, W.DTYPE_BF16)])
@pytest.mark.parametrize("align", [8, 4, 1])
def test_ragged_list_every_element(optimizer, grad_dtype, align):
    """Odd sizes: tails shorter than a vector, exact tile multiples, one element.  align=8: bulk copies for full
    tiles; align=4: bf16 gradients are then only 8-byte aligned, so 128-bit loads without bulk copies; align=1
    forces scalar accesses."""
    w = W.ragged_workload(n_replicas=3, optimizer=optimizer, grad_dtype=grad_dtype, align_elems=align)
    _lockstep(w, H.whole_tensor_slabs(w), check_every=1)


@pytest.mark.parametrize("n", [1, 2, 5, 32])
def test_replica_counts(n):
    w = W.ragged_workload(n_replicas=n, numels=(4099, 2048, 3))
    _lockstep(w, H.whole_tensor_slabs(w), check_every=3)


def test_shared_gradient_stride_zero():
    w = W.ragged_workload(n_replicas=4, numels=(5000, 17, 2048))
    _lockstep(w, H.whole_tensor_slabs(w), shared_grad=True, check_every=3)
    w = replace(W.config1(), tensors=(W.TensorSpec("flat", 10007, 0),))
    _lockstep(w, H.whole_tensor_slabs(w), shared_grad=True, check_every=4)


def _final_arena(w, fuse=1, shared_grad=False, steps=None, grad_mean=False, shared_state=False, device_resident=False):
    g = H.GpuRun(w, fuse=fuse, shared_grad=shared_grad, grad_mean=grad_mean, shared_state=shared_state,
                 device_resident=device_resident)
    for i in range(steps or w.total_steps):
        g.step(g.perm0())
    a = g.arena
    out = [a.param.clone()] + ([a.exp_avg.clone(), a.exp_avg_sq.clone()] if a.exp_avg is not None else [])
    launches = g.B.hdet_kernel_launches(g.h)
    g.close()
    return out, launches


def test_fused_converge_equals_update_then_converge_bitwise_and_runs_are_deterministic():
    import torch
    w = W.ragged_workload(n_replicas=5, numels=(1, 7, 4097, 2048, 12289))
    fused, l1 = _final_arena(w, fuse=1)
    again, _ = _final_arena(w, fuse=1)
    unfused, l2 = _final_arena(w, fuse=0)
    for a, b, c in zip(fused, again, unfused):
        assert torch.equal(a, b)
        assert torch.equal(a, c)
    assert l1 == w.total_steps and l2 == w.total_steps + w.total_steps // w.sync_interval


@pytest.mark.parametrize("optimizer,grad_dtype", [(W.OPT_ADAMW, W.DTYPE_BF16), (W.OPT_ADAMW, W.DTYPE_F32),
                                                   (W.OPT_SGD, W.DTYPE_F32), (W.OPT_SGD, W.DTYPE_BF16)])
@pytest.mark.parametrize("align", [8, 4, 1])
def test_gradient_replica_mean_every_element(optimizer, grad_dtype, align):
    """grad_mode = replica mean (Algorithm 1's gradient all-reduce on the device), per-replica moments."""
    w = W.ragged_workload(n_replicas=5, optimizer=optimizer, grad_dtype=grad_dtype, align_elems=align)
    _lockstep(w, H.whole_tensor_slabs(w), check_every=1, grad_mean=True)


@pytest.mark.parametrize("grad_dtype", [W.DTYPE_BF16, W.DTYPE_F32])
@pytest.mark.parametrize("align", [8, 1])
@pytest.mark.parametrize("mode", ["shared_grad", "mean"])
@pytest.mark.parametrize("n", [1, 2, 3, 4, 5, 8, 9, 32])
def test_shared_moments_every_element(grad_dtype, align, mode, n):
    """One pair of Adam moments for all replicas (state_stride 0), with a shared gradient or the replica mean."""
    w = W.ragged_workload(n_replicas=n, grad_dtype=grad_dtype, align_elems=align, numels=(4099, 7, 2048, 1, 6150))
    _lockstep(w, H.whole_tensor_slabs(w), check_every=3, shared_grad=(mode == "shared_grad"),
              grad_mean=(mode == "mean"), shared_state=True)


def test_shared_moments_kernel_equals_per_replica_moments_bitwise():
    import torch
    w = W.ragged_workload(n_replicas=6, numels=(4097, 2048, 33, 12289))
    per_replica, _ = _final_arena(w, shared_grad=True)
    shared, _ = _final_arena(w, shared_grad=True, shared_state=True)
    assert torch.equal(per_replica[0], shared[0])
    for a, b in zip(per_replica[1:], shared[1:]):
        assert torch.equal(a, b[None].expand_as(a))
    fused, _ = _final_arena(w, shared_grad=True, shared_state=True, fuse=0)
    assert torch.equal(fused[0], shared[0])


def test_config2_shape_with_gradient_mean_and_shared_moments_sampled():
    """The paper's own arrangement on one GPU: one all-reduced gradient, N rates, moments stored once; 300 updates."""
    w = replace(W.config2(), total_steps=300, warmup_steps=90)
    slabs = [(k, 0, min(2048, t.numel)) for k, t in enumerate(w.tensors) if k % 4 < 2]
    slabs += [(0, 2097152 - 4096, 4096), (10, 1024 * 1024 + 2048 * 7, 2048)]
    _lockstep(w, slabs, check_every=100, grad_mean=True, shared_state=True)


@pytest.mark.parametrize("optimizer,grad_dtype", [(W.OPT_ADAMW, W.DTYPE_BF16), (W.OPT_SGD, W.DTYPE_F32)])
@pytest.mark.parametrize("loss_dtype", ["float64", "float32"])
@pytest.mark.parametrize("fuse", [1, 0])
def test_device_resident_stepping_every_element_and_every_scalar(optimizer, grad_dtype, loss_dtype, fuse):
    """hdet_step_device: schedule, spread, loss accumulation and controller computed by device kernels."""
    w = W.ragged_workload(n_replicas=5, optimizer=optimizer, grad_dtype=grad_dtype)
    _lockstep(w, H.whole_tensor_slabs(w), check_every=1, device_resident=True, loss_dtype=loss_dtype, fuse=fuse)


def test_device_resident_config2_shape_sampled_with_shared_moments():
    w = replace(W.config2(), total_steps=200, warmup_steps=60, sync_interval=20)
    slabs = [(k, 0, min(2048, t.numel)) for k, t in enumerate(w.tensors) if k % 6 < 2]
    _lockstep(w, slabs, check_every=50, device_resident=True, grad_mean=True, shared_state=True)


def test_device_resident_equals_host_stepping_and_mode_switches():
    import torch
    w = W.ragged_workload(n_replicas=4, numels=(4097, 2048, 33))
    host, _ = _final_arena(w)
    dev, _ = _final_arena(w, device_resident=True)
    for a, b in zip(host, dev):
        assert H.rel_err(b.cpu().numpy(), a.cpu().numpy().astype(np.float64)).max() <= 1e-6
    # a handle in device mode refuses host stepping until hdet_set_state hands the state back
    g = H.GpuRun(w, device_resident=True)
    for i in range(5):
        g.step(g.perm0())
    with pytest.raises(g.B.HdetError) as e:
        g.B.hdet_step(g.h, None)
    assert e.value.status == g.B.HDET_ERR_STATE
    with pytest.raises(g.B.HdetError) as e:
        g.B.hdet_autolr_update(g.h)
    assert e.value.status == g.B.HDET_ERR_STATE
    # a schedule change would reach only part of the device-resident state: refused until the state is back on the host
    with pytest.raises(g.B.HdetError) as e:
        g.B.hdet_set_schedule(g.h, H.lib_schedule(g.B, w))
    assert e.value.status == g.B.HDET_ERR_STATE
    st = g.state()
    assert st.step == 5
    g.B.hdet_set_state(g.h, st)
    g.B.hdet_set_schedule(g.h, H.lib_schedule(g.B, w))       # accepted again (same schedule: the run continues unchanged)
    g.B.hdet_set_state(g.h, st)                               # the call reset the base weight decays; restore them
    g.device_resident = False
    for i in range(5, w.total_steps):
        g.step(g.perm0())
    final = [g.arena.param.clone(), g.arena.exp_avg.clone(), g.arena.exp_avg_sq.clone()]
    g.close()
    for a, b in zip(host, final):
        assert H.rel_err(b.cpu().numpy(), a.cpu().numpy().astype(np.float64)).max() <= 1e-6


def test_device_resident_round_replayed_from_a_cuda_graph():
    """A round of T device-resident steps recorded once and replayed gives the same bits as direct calls."""
    import torch
    w = replace(W.ragged_workload(n_replicas=4, numels=(4097, 2048, 33)), total_steps=40, warmup_steps=8,
                sync_interval=4)
    T, rounds = w.sync_interval, 5
    losses = torch.tensor([[3.0 - 0.05 * r + 0.01 * i for r in range(4)] for i in range(T)], dtype=torch.float64,
                          device="cuda")

    def direct():
        g = H.GpuRun(w, device_resident=True)
        g.fill_grads(0)
        s = torch.cuda.current_stream().cuda_stream
        for k in range(rounds * T):
            g.B.hdet_step_device(g.h, losses[k % T], s)
        torch.cuda.synchronize()
        out = [g.arena.param.clone(), g.arena.exp_avg.clone(), g.arena.exp_avg_sq.clone()], g.state()
        g.close()
        return out

    ref, ref_state = direct()
    g = H.GpuRun(w, device_resident=True)
    g.fill_grads(0)
    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    with torch.cuda.stream(side):
        for k in range(T):                                   # first round directly (uploads the state)
            g.B.hdet_step_device(g.h, losses[k], side.cuda_stream)
    torch.cuda.synchronize()
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph, stream=side):
        for k in range(T):
            g.B.hdet_step_device(g.h, losses[k], torch.cuda.current_stream().cuda_stream)
    for _ in range(rounds - 1):
        graph.replay()
    torch.cuda.synchronize()
    st = g.state()                                           # reads the device copy back; host knows the count again
    assert st.step == rounds * T == ref_state.step
    assert bytes(st) == bytes(ref_state)
    for a, b in zip(ref, [g.arena.param, g.arena.exp_avg, g.arena.exp_avg_sq]):
        assert torch.equal(a, b)
    assert st.fired == 1
    g.close()


@pytest.mark.parametrize("grad_dtype", [W.DTYPE_F32, W.DTYPE_BF16])
@pytest.mark.parametrize("align", [8, 1])
@pytest.mark.parametrize("momentum,fuse", [(0.9, 1), (0.9, 0), (0.0, 1)])
def test_sgd_with_weight_decay_and_momentum_every_element(grad_dtype, align, momentum, fuse):
    """SGD beyond Eq. 2: coupled weight decay (spread per replica) and a momentum buffer per replica."""
    w = replace(W.ragged_workload(n_replicas=4, optimizer=W.OPT_SGD, grad_dtype=grad_dtype, align_elems=align),
                momentum=momentum)
    _lockstep(w, H.whole_tensor_slabs(w), check_every=1, fuse=fuse)
    _lockstep(w, H.whole_tensor_slabs(w), check_every=4, fuse=fuse, device_resident=True, grad_mean=True)


@pytest.mark.parametrize("device_resident", [False, True])
def test_weight_decay_channel_controller_every_element(device_resident):
    """Remark 1: the controller also adapts the weight-decay base; host and device-resident stepping."""
    w = replace(W.ragged_workload(n_replicas=5), auto_wd=1, total_steps=18)
    _lockstep(w, H.whole_tensor_slabs(w), check_every=1, device_resident=device_resident)


def test_alpha_zero_keeps_replicas_bitwise_identical():
    import torch
    w = replace(W.ragged_workload(n_replicas=6, numels=(4097, 33)), alpha_lr=0.0, alpha_wd=0.0, autolr=0)
    g = H.GpuRun(w, shared_grad=True)
    for i in range(7):
        g.step()
        for t in (g.arena.param, g.arena.exp_avg, g.arena.exp_avg_sq):
            assert torch.equal(t, t[0:1].expand_as(t))
    g.close()


def test_padding_between_tensors_is_never_written():
    import torch
    w = W.ragged_workload(n_replicas=3)
    g = H.GpuRun(w)
    mask = torch.ones(g.arena.p_pad, dtype=torch.bool, device="cuda")
    for off, t in zip(g.arena.offsets, w.tensors):
        mask[off:off + t.numel] = False
    assert mask.any()
    arrays = (g.arena.param, g.arena.exp_avg, g.arena.exp_avg_sq)
    for t in arrays[1:]:
        t[:, mask] = 7.0                      # canary
    before = [t[:, mask].clone() for t in arrays]
    for i in range(w.total_steps):
        g.step(g.perm0())
    for t, b in zip(arrays, before):
        assert torch.equal(t[:, mask], b)
    g.close()


def test_standalone_converge_matches_oracle_mean():
    import torch
    from oracle import hdet_oracle as O
    w = W.ragged_workload(n_replicas=7, numels=(4099, 5, 2048))
    g = H.GpuRun(w)
    torch.manual_seed(0)
    g.arena.param.copy_(torch.randn_like(g.arena.param))
    before = g.arena.param.cpu().numpy().astype(np.float64)
    m0 = g.arena.exp_avg.clone()
    g.B.hdet_converge(g.h)
    after = g.arena.param.cpu().numpy()
    for off, t in zip(g.arena.offsets, w.tensors):
        ref = before[:, off:off + t.numel].copy()
        O.converge(ref)
        assert H.rel_err(after[:, off:off + t.numel], ref).max() <= 1e-7
    assert torch.equal(g.arena.exp_avg, m0)
    assert g.state().step == 0
    g.close()


def test_nonfinite_parameter_sets_the_status_word():
    import torch
    w = W.ragged_workload(n_replicas=2, numels=(3000,))
    g = H.GpuRun(w)
    g.step()
    assert g.state().device_status == 0
    g.arena.grad[1, 5] = float("inf")
    g.B.hdet_step(g.h, None)
    with pytest.raises(g.B.HdetError) as e:
        g.B.hdet_get_state(g.h)
    assert e.value.status == g.B.HDET_ERR_NONFINITE
    st = g.B.hdet_get_state(g.h, raise_on_nonfinite=False)
    assert st.device_status & 1
    g.B.hdet_set_state(g.h, st)            # clears the word
    assert g.B.hdet_get_state(g.h).device_status == 0
    g.close()


@pytest.mark.parametrize("align", [8, 4])
def test_eps_zero_on_a_ragged_list_sets_no_status_bit(align):
    """eps = 0 is accepted.  Idle lanes of a partial tile hold zeros and would compute 0/0 there; that must
    neither reach memory nor the status word."""
    w = replace(W.ragged_workload(n_replicas=3, align_elems=align), eps=0.0)
    slabs = H.whole_tensor_slabs(w)
    o = H.OracleRun(w, slabs)
    # precondition of the case: no first gradient is exactly zero (v would stay 0 and 0/0 would be genuine)
    assert all(np.all(g != 0.0) for g in o.grads(0))
    g = H.GpuRun(w)
    try:
        for i in range(3):
            assert g.step(g.perm0()) == o.step()
            H.compare_slabs(g, o, TOL_ONE_STEP if i == 0 else TOL_FULL_RUN)
            assert g.state().device_status == 0
    finally:
        g.close()


@pytest.mark.parametrize("align", [8, 4, 1])
@pytest.mark.parametrize("mode", ["fused", "fused_f32_grads", "unfused", "device", "shared_moments", "grad_mean", "sgd"])
def test_bf16_copy_of_the_averaged_parameters(align, mode):
    """hdet_tensor.param_bf16: every converge also writes the averaged parameters as bfloat16.  Bit-exact against
    the oracle's rounding of the fp32 value the GPU stored; against the oracle's own mean at most one bf16 step
    apart (where the two fp32 means differ in their last bit across a rounding boundary); untouched by updates
    that do not converge, and outside the tensors."""
    import torch
    from oracle import hdet_oracle as O
    w = W.ragged_workload(n_replicas=3, align_elems=align,
                          optimizer=W.OPT_SGD if mode == "sgd" else W.OPT_ADAMW,
                          grad_dtype=W.DTYPE_F32 if mode in ("sgd", "fused_f32_grads") else W.DTYPE_BF16)
    kw = dict(shared_grad=(mode == "shared_moments"), shared_state=(mode == "shared_moments"), grad_mean=(mode == "grad_mean"))
    g = H.GpuRun(w, fuse=0 if mode == "unfused" else 1, device_resident=(mode == "device"), bf16_copy=True, **kw)
    o = H.OracleRun(w, H.whole_tensor_slabs(w), shared_grad=kw["shared_grad"], grad_mean=kw["grad_mean"])
    sentinel = 0x7FC1
    bits_view = g.arena.param_bf16.view(torch.int16)
    bits_view.fill_(sentinel)
    used = np.zeros(g.arena.p_pad, dtype=bool)
    for off, ne in zip(g.arena.offsets, g.arena.numels):
        used[off:off + ne] = True
    last, rounds = None, 0
    try:
        for i in range(w.total_steps):
            ended = g.step(g.perm0())
            assert ended == o.step()
            bits = bits_view.cpu().numpy().view(np.uint16)
            assert np.all(bits[~used] == sentinel)                         # padding is never written
            if ended:
                rounds += 1
                stored = g.arena.param[0].cpu().numpy()
                assert np.array_equal(bits[used], O.bf16_bits(stored[used]))     # RNE of the stored fp32 mean, bit for bit
                for k, (off, ne) in enumerate(zip(g.arena.offsets, g.arena.numels)):
                    want = O.averaged_bf16(o.o.theta[k]).astype(np.int32)
                    diff = np.abs(bits[off:off + ne].astype(np.int32) - want)
                    assert diff.max() <= 1 and np.mean(diff == 0) >= 0.99
                last = bits.copy()
            elif last is None:
                assert np.all(bits == sentinel)                            # nothing before the first converge
            else:
                assert np.array_equal(bits, last)                          # plain updates leave the copy alone
        assert rounds == w.total_steps // w.sync_interval
        # the stand-alone converge writes it too
        g.arena.param[1].mul_(1.5)
        bits_view.fill_(sentinel)
        g.B.hdet_converge(g.h)
        torch.cuda.synchronize()
        bits = bits_view.cpu().numpy().view(np.uint16)
        assert np.array_equal(bits[used], O.bf16_bits(g.arena.param[0].cpu().numpy()[used]))
        assert np.all(bits[~used] == sentinel)
        assert g.state().device_status == 0
    finally:
        g.close()


@pytest.mark.parametrize("grad_dtype", [W.DTYPE_BF16, W.DTYPE_F32])
@pytest.mark.parametrize("grad_mean", [False, True])
def test_bulk_register_and_scalar_paths_give_the_same_bits(grad_dtype, grad_mean):
    """The same tensors WITH THE SAME VALUES laid out at 8-, 4- and 1-element alignment go through the bulk-copy
    ring, the 128-bit register pipeline and the scalar path; parameters and both moments must agree bit for bit
    after a whole run (fused converges included), tensor by tensor.  (The seeded generator indexes by arena
    offset, so the values of the 8-aligned run are copied into the other layouts tensor by tensor.)"""
    import torch
    numels = (6150, 2048, 33, 12289, 4097, 8192)
    runs = [H.GpuRun(W.ragged_workload(n_replicas=5, grad_dtype=grad_dtype, align_elems=a, numels=numels), grad_mean=grad_mean)
            for a in (8, 4, 1)]
    src = runs[0]

    def copy_from_src(name):
        for g in runs[1:]:
            for k, ne in enumerate(numels):
                o0, o1 = src.arena.offsets[k], g.arena.offsets[k]
                getattr(g.arena, name)[:, o1:o1 + ne].copy_(getattr(src.arena, name)[:, o0:o0 + ne])

    try:
        copy_from_src("param")
        w = src.w
        for i in range(w.total_steps):
            src.fill_grads(i)
            copy_from_src("grad")
            losses = list(R.step_losses(w, i, src.perm0()))
            for g in runs:
                if g.B.hdet_step(g.h, losses):
                    g.B.hdet_autolr_update(g.h)
        torch.cuda.synchronize()
        for g in runs[1:]:
            for k, ne in enumerate(numels):
                o0, o1 = src.arena.offsets[k], g.arena.offsets[k]
                for name in ("param", "exp_avg", "exp_avg_sq"):
                    assert torch.equal(getattr(src.arena, name)[:, o0:o0 + ne], getattr(g.arena, name)[:, o1:o1 + ne]), \
                        (name, k, g.w.align_elems)
            assert g.state().device_status == 0
    finally:
        for g in runs:
            g.close()


def test_the_first_step_of_a_fresh_handle_can_be_recorded_into_a_cuda_graph():
    """hdet_create prepares the bulk-copy kernels (their shared-memory attribute), so even the very first
    hdet_step of a handle makes no attribute call and can be captured; a replay equals a direct step bit for bit."""
    import torch
    w = replace(W.ragged_workload(n_replicas=4, numels=(4097, 2048, 33, 12289)), sync_interval=1)
    direct = H.GpuRun(w)
    direct.fill_grads(0)
    direct.B.hdet_step(direct.h, None)
    torch.cuda.synchronize()
    g = H.GpuRun(w)
    g.fill_grads(0)
    torch.cuda.synchronize()
    graph, side = torch.cuda.CUDAGraph(), torch.cuda.Stream()
    with torch.cuda.graph(graph, stream=side):
        g.B.hdet_step(g.h, None, torch.cuda.current_stream().cuda_stream)      # recorded, not run
    assert torch.equal(g.arena.exp_avg, torch.zeros_like(g.arena.exp_avg))
    graph.replay()
    torch.cuda.synchronize()
    for a, b in ((g.arena.param, direct.arena.param), (g.arena.exp_avg, direct.arena.exp_avg),
                 (g.arena.exp_avg_sq, direct.arena.exp_avg_sq)):
        assert torch.equal(a, b)
    assert g.state().device_status == 0
    g.close()
    direct.close()


def test_a_wait_that_runs_out_becomes_a_status_and_the_context_stays_usable():
    """Failure handling without a fault: hdet_selftest_bounded_wait makes a kernel wait, with the limit every
    bulk-copy wait has, on a barrier that nothing completes.  The wait ends by itself after about a second, the
    status word carries the timeout bit, update kernels launched meanwhile leave the data alone, hdet_set_state
    clears the bit, and the run then continues in step with the oracle."""
    import time
    import torch
    w = W.ragged_workload(n_replicas=3)
    g = H.GpuRun(w)
    o = H.OracleRun(w, H.whole_tensor_slabs(w))
    try:
        assert g.step(g.perm0()) == o.step()
        clean = g.state()
        before = [g.arena.param.clone(), g.arena.exp_avg.clone(), g.arena.exp_avg_sq.clone()]
        torch.cuda.synchronize()
        t0 = time.perf_counter()
        g.B.hdet_selftest_bounded_wait(g.h, torch.cuda.current_stream().cuda_stream)
        torch.cuda.synchronize()
        waited = time.perf_counter() - t0
        assert 0.3 < waited < 20.0                      # bounded: about 2e9 SM cycles, not forever
        with pytest.raises(g.B.HdetError) as e:
            g.B.hdet_get_state(g.h)
        assert e.value.status == g.B.HDET_ERR_TIMEOUT
        assert g.B.hdet_get_state(g.h, raise_on_nonfinite=False).device_status & 2
        g.fill_grads(1)
        g.B.hdet_step(g.h, None)                        # launched while the bit is set: every CTA leaves at once
        torch.cuda.synchronize()
        for a, b in zip(before, [g.arena.param, g.arena.exp_avg, g.arena.exp_avg_sq]):
            assert torch.equal(a, b)
        g.B.hdet_set_state(g.h, clean)                  # back to the state after update 1; clears the status word
        assert g.state().device_status == 0
        for i in range(1, w.total_steps):
            assert g.step(g.perm0()) == o.step()
        H.compare_slabs(g, o, TOL_FULL_RUN)
        H.compare_scalars(g.state(), o.o, w.n_replicas, w.n_groups)
    finally:
        g.close()


def test_config2_full_run_sampled():
    """N=8, 25.19 M parameters, AdamW, one-cycle over 1000 updates, T=50, controller on: the full run."""
    w = W.config2()
    slabs = [(k, 0, min(2048, t.numel)) for k, t in enumerate(w.tensors)]
    slabs += [(0, 2097152 - 4096, 4096), (10, 1024 * 1024 + 2048 * 7, 2048), (22, 2048 * 513, 2048)]
    worst = _lockstep(w, slabs, check_every=250)
    assert worst <= TOL_FULL_RUN


def _free_gb():
    import gc
    import torch
    gc.collect()
    torch.cuda.empty_cache()
    return torch.cuda.mem_get_info()[0] / 1e9


ONE_STEP_FRACTION = 0.05


def _full_size(w, check_every):
    """A full-size workload against the oracle, with the coverage stated and asserted.

    Whole run, every update: the first tile and the last tile with its ragged tail of EVERY tensor (oracle
    worker processes in lockstep with the GPU; checked after the first update, every `check_every` updates and
    at the end, scalars at every round end).  After the first update, at the one-step tolerance, also at least
    5 % of all elements in random runs of 64 tiles (each run is an independent one-step oracle problem, farmed
    out to a process pool).  Returns the worst relative error seen.
    """
    import multiprocessing as mp
    from oracle import driver as OD
    edge = H.edge_slabs(w)
    assert {k for (k, _, _) in edge} == set(range(len(w.tensors)))            # every tensor is touched
    runs = H.random_run_slabs(w, ONE_STEP_FRACTION, run_tiles=64, seed=w.seed)
    one_step_fraction = H.slab_elements(runs) / w.numel
    whole_run_fraction = H.slab_elements(edge) / w.numel
    assert one_step_fraction >= ONE_STEP_FRACTION
    pool = H.OraclePool(w, edge)
    g = H.GpuRun(w)
    names = ("param", "m", "v")

    def fetch(k, s, n):
        return {name: g.slab(name, k, s, n) for name in names}

    worst, o_perm = 0.0, list(range(w.n_replicas))
    try:
        for i in range(w.total_steps):
            perm = g.perm0()
            assert perm == o_perm
            ended = g.step(perm)
            o_ended, o_perm = pool.step()
            assert ended == o_ended
            if i == 0:
                worst = max(worst, pool.compare(fetch, TOL_ONE_STEP))
                groups = [runs[j:j + 4] for j in range(0, len(runs), 4)]
                tasks = ((w, grp, [fetch(*sl) for sl in grp], TOL_ONE_STEP, {}) for grp in groups)
                with mp.get_context("spawn").Pool(OD.usable_cores()) as farm:
                    for e, msg in farm.imap_unordered(OD.one_step_errors, tasks):
                        assert msg is None, msg
                        worst = max(worst, e)
            elif (i + 1) % check_every == 0:
                worst = max(worst, pool.compare(fetch, TOL_FULL_RUN))
            if ended or i == 0:
                H.compare_scalars(g.state(), pool.scalars(), w.n_replicas, w.n_groups)
        worst = max(worst, pool.compare(fetch, TOL_FULL_RUN))
        st = g.state()
        assert st.device_status == 0
        H.compare_scalars(st, pool.scalars(), w.n_replicas, w.n_groups)
    finally:
        pool.close()
        g.close()
    print(f"\n{w.name}: checked {100 * one_step_fraction:.2f} % of the N x P = {w.n_replicas} x {w.numel} elements after one "
          f"update and {100 * whole_run_fraction:.3f} % through all {w.total_steps} updates (first and last tile of each of "
          f"the {len(w.tensors)} tensors, all touched); worst relative error {worst:.2e}")
    return worst


def test_config3_full_size_sampled():
    """N=8, 354.8 M parameters in 292 tensors (39.7 GB resident), 500 updates, T=100, controller on."""
    w = W.config3()
    if _free_gb() < 45:
        pytest.skip("needs 45 GB of free device memory")
    assert _full_size(w, check_every=250) <= TOL_FULL_RUN


def test_config4_full_size_sampled():
    """N=8, 1.316 B parameters (147.4 GB resident), T=1: every update is the fused update+converge kernel."""
    w = W.config4()
    if _free_gb() < 152:
        pytest.skip("needs 152 GB of free device memory")
    assert _full_size(w, check_every=10) <= TOL_FULL_RUN


@pytest.mark.parametrize("T", [1, 10, 100])
def test_config5_n16_weight_decay_spread(T):
    """N=16, 124.4 M parameters, learning-rate and weight-decay spread, 300 updates, controller on."""
    w = W.config5(T)
    if _free_gb() < 32:
        pytest.skip("needs 32 GB of free device memory")
    assert _full_size(w, check_every=100) <= TOL_FULL_RUN


@pytest.mark.parametrize("align", [8, 1])
def test_warm_noisy_init_every_element(align):
    """Eq. 10 on the device against the oracle's counter-based Box-Muller draws; nu = 0; determinism."""
    import torch
    from oracle import hdet_oracle as O
    w = W.ragged_workload(n_replicas=4, align_elems=align, numels=(4099, 7, 2048, 1, 6150, 33))
    g = H.GpuRun(w)
    offs = g.arena.offsets
    theta0 = [g.arena.param[0, o:o + t.numel].cpu().numpy().astype(np.float64) for o, t in zip(offs, w.tensors)]
    m_before = g.arena.exp_avg.clone()
    g.B.hdet_warm_init(g.h, 0.01, 77)
    sigma = O.warm_sigma(theta0, 0.01)
    worst = 0.0
    for k, (o, t) in enumerate(zip(offs, w.tensors)):
        ref = O.warm_noisy_init(theta0[k], sigma, 77, 4, k)
        got = g.arena.param[:, o:o + t.numel].cpu().numpy()
        worst = max(worst, H.rel_err(got, ref).max())
        # the noise itself, not just theta + noise: compare eps / sigma with the oracle's draws
        z_got = (got.astype(np.float64) - theta0[k]) / sigma
        z_ref = (ref - theta0[k]) / sigma
        assert np.max(np.abs(z_got - z_ref)) < 2e-3          # fp32 rounding of theta + eps limits what can be resolved
    assert worst <= TOL_ONE_STEP
    assert torch.equal(g.arena.exp_avg, m_before) and g.state().step == 0
    first = g.arena.param.clone()
    # same seed on the perturbed replica 0 differs; restore the checkpoint and repeat: bitwise identical
    for k, (o, t) in enumerate(zip(offs, w.tensors)):
        g.arena.param[0, o:o + t.numel] = torch.from_numpy(theta0[k]).float().cuda()
    g.B.hdet_warm_init(g.h, 0.01, 77)
    assert torch.equal(g.arena.param, first)
    # nu = 0: every replica is an exact copy of the checkpoint
    for k, (o, t) in enumerate(zip(offs, w.tensors)):
        g.arena.param[0, o:o + t.numel] = torch.from_numpy(theta0[k]).float().cuda()
    g.B.hdet_warm_init(g.h, 0.0, 77)
    for k, (o, t) in enumerate(zip(offs, w.tensors)):
        blk = g.arena.param[:, o:o + t.numel]
        assert torch.equal(blk, blk[0:1].expand_as(blk))
        assert np.array_equal(blk[0].cpu().numpy().astype(np.float64), theta0[k])
    with pytest.raises(g.B.HdetError):
        g.B.hdet_warm_init(g.h, -1.0, 0)
    g.close()


def test_warm_noisy_init_config2_statistics_and_sampled_parity():
    from oracle import hdet_oracle as O
    w = W.config2()
    g = H.GpuRun(w)
    n = w.n_replicas
    offs = g.arena.offsets
    theta0_full = g.arena.param[0].cpu().numpy().astype(np.float64)
    theta0 = [theta0_full[o:o + t.numel] for o, t in zip(offs, w.tensors)]
    g.B.hdet_warm_init(g.h, 0.01, 2024)
    sigma = O.warm_sigma(theta0, 0.01)
    assert sigma == pytest.approx(0.01 * 0.02, rel=2e-3)          # parameters are N(0, 0.02^2)
    after = g.arena.param.cpu().numpy().astype(np.float64)
    eps = after - theta0_full[None, :]
    assert eps.std() == pytest.approx(sigma, rel=2e-3) and abs(eps.mean()) < 5 * sigma / np.sqrt(eps.size)
    c = np.corrcoef(eps[0, :200000], eps[1, :200000])[0, 1]
    assert abs(c) < 0.01                                           # replicas draw independent noise
    for k, s0, ln in [(0, 0, 2048), (0, 2097152 - 3000, 3000), (1, 0, 2048), (22, 2048 * 500 + 1, 2047), (23, 5, 300)]:
        ref = O.warm_noisy_init(theta0[k][s0:s0 + ln], sigma, 2024, n, k, start=s0)
        got = after[:, offs[k] + s0:offs[k] + s0 + ln]
        assert H.rel_err(got, ref).max() <= TOL_ONE_STEP
    g.close()


def test_step_with_host_gradients_equals_step_with_device_gradients():
    """hdet_step_host_grads: the library uploads each tensor's gradients (strided per replica), then updates."""
    import torch
    for shared in (False, True):
        w = W.ragged_workload(n_replicas=4, numels=(4099, 7, 2048, 33))
        ref, _ = _final_arena(w, shared_grad=shared, steps=6)
        g = H.GpuRun(w, shared_grad=shared)
        gsz = g.arena.grad.element_size()
        for i in range(6):
            g.fill_grads(i)
            host = g.arena.grad.cpu().pin_memory()
            g.arena.grad.zero_()                               # the device copy must come from the host image
            ptrs = [host.data_ptr() + gsz * off for off in g.arena.offsets]
            losses = list(R.step_losses(w, i, g.perm0()))
            if g.B.hdet_step_host_grads(g.h, ptrs, losses):
                g.B.hdet_autolr_update(g.h)
            torch.cuda.synchronize()
            g.i += 1
        for a, b in zip(ref, [g.arena.param, g.arena.exp_avg, g.arena.exp_avg_sq]):
            assert torch.equal(a, b)
        with pytest.raises(g.B.HdetError):
            g.B.hdet_step_host_grads(g.h, [0] * len(w.tensors), None)
        g.close()


def test_maximum_replicas_and_groups():
    """N = 32 replicas and G = 8 groups: every slot of the 8 x 32 launch-scalar tables is in use."""
    w = W.ragged_workload(n_replicas=32, n_groups=8, numels=(2051, 7, 4096, 33, 1, 2048, 515, 9, 130, 4100))
    w = replace(w, total_steps=9, warmup_steps=3)
    _lockstep(w, H.whole_tensor_slabs(w), check_every=3)
    _lockstep(w, H.whole_tensor_slabs(w), check_every=3, device_resident=True)
