"""Replica axis sharded over GPUs: hdet_step_sharded + all-reduce of the local sums + hdet_apply_mean.

Only one GPU is available, so the ranks are emulated as separate handles (separate arenas) stepped one
after the other; their staging buffers are summed with a torch add, which is what an all-reduce computes.
No kernel waits on another.  The host-side scalars are checked without a GPU.
"""
from dataclasses import replace

import numpy as np
import pytest

import harness as H
from hdet_inputs import recipes as R
from hdet_inputs import workloads as W
from paper_2604_24708_b200 import binding as B
from paper_2604_24708_b200 import from_workload
from oracle import hdet_oracle as O


def test_sharded_handles_compute_the_global_scalars_on_every_rank():
    """Each rank's handle (no tensors, no device) must hold the same N-wide tables as an unsharded handle."""
    w = W.config5(10)
    whole = B.hdet_create(from_workload.config_for(w), [])
    parts = [B.hdet_create(from_workload.config_for(w, n_local=4, replica_offset=4 * k), []) for k in range(4)]
    for h in [whole] + parts:
        B.hdet_set_schedule(h, from_workload.schedule_for(w))
    for i in range(120):
        perm = list(B.hdet_get_state(whole).perm_lr[0])[:16]
        losses = list(R.step_losses(w, i, perm))
        ended = B.hdet_step(whole, losses)
        for h in parts:
            assert B.hdet_step_sharded(h, losses, None) == ended
        if ended:
            for h in [whole] + parts:
                B.hdet_autolr_update(h)
        ref = bytes(B.hdet_get_state(whole))
        for h in parts:
            assert bytes(B.hdet_get_state(h)) == ref
    assert B.hdet_get_state(whole).fired == 1
    for kw in (dict(n_local=4, replica_offset=14), dict(n_local=4, replica_offset=-1)):
        with pytest.raises(B.HdetError) as e:
            B.hdet_create(from_workload.config_for(w, **kw), [])
        assert e.value.status == B.HDET_ERR_INVALID_ARG
    with pytest.raises(B.HdetError) as e:
        B.hdet_create(from_workload.config_for(w, n_local=4, replica_offset=0, grad_mode=B.HDET_GRAD_REPLICA_MEAN), [])
    assert e.value.status == B.HDET_ERR_UNSUPPORTED
    with pytest.raises(B.HdetError) as e:              # a shard cannot average on its own
        B.hdet_step(parts[0], None)
    assert e.value.status == B.HDET_ERR_STATE
    for h in [whole] + parts:
        B.hdet_destroy(h)


class _Rank:
    """One emulated rank: its own arena with n_local replicas of the workload and a sharded handle."""

    def __init__(self, w, n_local, offset, shared_grad):
        import torch
        from hdet_inputs import device as D
        from paper_2604_24708_b200.arena import StackedArena
        self.w, self.n_local, self.offset, self.D, self.shared_grad = w, n_local, offset, D, shared_grad
        self.arena = StackedArena([t.numel for t in w.tensors], [t.group for t in w.tensors], n_local, w.optimizer,
                                  w.grad_dtype, align_elems=w.align_elems, shared_grad=shared_grad,
                                  shared_state=shared_grad, bf16_copy=True)
        D.fill(self.arena.param[0], R.param_key(w), 0, R.param_scale(w))
        for r in range(1, n_local):
            self.arena.param[r].copy_(self.arena.param[0])
        self.h = B.hdet_create(from_workload.config_for(w, n_local=n_local, replica_offset=offset),
                               self.arena.descriptors())
        B.hdet_set_schedule(self.h, from_workload.schedule_for(w))
        offs, total = B.hdet_partial_layout(self.h, len(w.tensors))
        self.partial_offsets = offs
        self.partial = torch.zeros(total, dtype=torch.float32, device="cuda")

    def fill_grads(self, step):
        if self.shared_grad:
            self.D.fill(self.arena.grad, R.grad_key(self.w, step, 0), 0, R.grad_scale(self.w))
        else:
            for r in range(self.n_local):      # local replica r is global replica offset + r
                self.D.fill(self.arena.grad[r], R.grad_key(self.w, step, self.offset + r), 0, R.grad_scale(self.w))


@pytest.mark.gpu
@pytest.mark.parametrize("split", [(2, 2, 2), (3, 1, 2), (6,)])
def test_exchange_inside_the_kernel_matches_the_oracle_and_agrees_on_every_rank(split):
    """hdet_apply_mean_peers: every emulated rank reads all staging buffers itself (here all on one device, where a
    peer's buffer is just another pointer) in rank order; no all-reduce.  Every rank must end with the same bits,
    and they must be the oracle's mean within the tolerances."""
    import torch
    w = W.ragged_workload(n_replicas=6, numels=(4099, 7, 2048, 1, 6150, 33))
    ranks, off = [], 0
    for n_local in split:
        ranks.append(_Rank(w, n_local, off, False))
        off += n_local
    o = H.OracleRun(w, H.whole_tensor_slabs(w))
    stream = torch.cuda.current_stream().cuda_stream
    for i in range(w.total_steps):
        perm = list(B.hdet_get_state(ranks[0].h).perm_lr[0])[:6]
        losses = list(R.step_losses(w, i, perm))
        ended = None
        for rk in ranks:
            rk.fill_grads(i)
            ended = B.hdet_step_sharded(rk.h, losses, rk.partial, stream)
        assert ended == o.step()
        if ended:                                # one stream: the launches below follow every rank's update in order
            for rk in ranks:
                B.hdet_apply_mean_peers(rk.h, [q.partial for q in ranks], stream)
                B.hdet_autolr_update(rk.h)
            means = [rk.arena.param[0].clone() for rk in ranks]
            for rk, m in zip(ranks, means):
                for ao, t in zip(rk.arena.offsets, w.tensors):
                    assert torch.equal(m[ao:ao + t.numel], means[0][ao:ao + t.numel])          # same bits on every rank
                    bits = rk.arena.param_bf16[ao:ao + t.numel].view(torch.int16).cpu().numpy().view(np.uint16)
                    assert np.array_equal(bits, O.bf16_bits(m[ao:ao + t.numel].cpu().numpy()))
        tol = 1e-6 if i == 0 else 1e-5
        for rk in ranks:
            for k, (ao, t) in enumerate(zip(rk.arena.offsets, w.tensors)):
                got = rk.arena.param[:, ao:ao + t.numel].cpu().numpy()
                assert H.rel_err(got, o.o.theta[k][rk.offset:rk.offset + rk.n_local]).max() <= tol, (i, k)
    with pytest.raises(B.HdetError) as e:
        B.hdet_apply_mean_peers(ranks[0].h, [], stream)
    assert e.value.status == B.HDET_ERR_INVALID_ARG
    for rk in ranks:
        torch.cuda.synchronize()
        B.hdet_destroy(rk.h)


@pytest.mark.gpu
@pytest.mark.parametrize("shared_grad", [False, True])
@pytest.mark.parametrize("split", [(2, 2, 2), (3, 1, 2), (6,)])
def test_sharded_replica_axis_matches_the_oracle_with_all_replicas(split, shared_grad):
    """6 replicas on 3, 3 (uneven) or 1 emulated rank(s); the all-reduce is a sum of the staging buffers."""
    import torch
    import torch.distributed as dist
    w = W.ragged_workload(n_replicas=6, numels=(4099, 7, 2048, 1, 6150, 33))
    ranks, off = [], 0
    for n_local in split:
        ranks.append(_Rank(w, n_local, off, shared_grad))
        off += n_local
    o = H.OracleRun(w, H.whole_tensor_slabs(w), shared_grad=shared_grad)
    stream = torch.cuda.current_stream().cuda_stream
    nccl = dist.is_initialized()
    if not nccl:                              # a real NCCL all-reduce (world size 1) on the summed buffer, if NCCL comes up
        try:
            import socket
            with socket.socket() as sk:
                sk.bind(("127.0.0.1", 0))
                port = sk.getsockname()[1]
            dist.init_process_group("nccl", init_method=f"tcp://127.0.0.1:{port}", rank=0, world_size=1,
                                    device_id=torch.device("cuda:0"))
            nccl = True
        except Exception:                     # the library does not depend on it; the sum below is the stand-in
            nccl = False
    for i in range(w.total_steps):
        perm = list(B.hdet_get_state(ranks[0].h).perm_lr[0])[:6]
        assert perm == o.o.perm_lr[0]
        losses = list(R.step_losses(w, i, perm))
        ended = None
        for rk in ranks:
            rk.fill_grads(i)
            e = B.hdet_step_sharded(rk.h, losses, rk.partial, stream)
            assert ended in (None, e)
            ended = e
        assert ended == o.step()
        if ended:
            total = torch.stack([rk.partial for rk in ranks]).sum(dim=0)      # what the all-reduce delivers
            if nccl:
                dist.all_reduce(total)                                        # world size 1: unchanged
            for rk in ranks:
                B.hdet_apply_mean(rk.h, total, stream)
                B.hdet_autolr_update(rk.h)
            for rk in ranks:                  # hdet_apply_mean also refreshes the bf16 copy of the averaged parameters
                for ao, t in zip(rk.arena.offsets, w.tensors):
                    stored = rk.arena.param[0, ao:ao + t.numel].cpu().numpy()
                    bits = rk.arena.param_bf16[ao:ao + t.numel].view(torch.int16).cpu().numpy().view(np.uint16)
                    assert np.array_equal(bits, O.bf16_bits(stored))
        tol = 1e-6 if i == 0 else 1e-5
        for rk in ranks:
            for k, (ao, t) in enumerate(zip(rk.arena.offsets, w.tensors)):
                got = rk.arena.param[:, ao:ao + t.numel].cpu().numpy()
                ref = o.o.theta[k][rk.offset:rk.offset + rk.n_local]
                assert H.rel_err(got, ref).max() <= tol, (i, k)
            H.compare_scalars(B.hdet_get_state(rk.h), o.o, 6, w.n_groups)
    assert o.o.fired
    for rk in ranks:
        if len(split) > 1:                    # a shard cannot average on its own
            with pytest.raises(B.HdetError) as e:
                B.hdet_converge(rk.h)
            assert e.value.status == B.HDET_ERR_UNSUPPORTED
        torch.cuda.synchronize()
        B.hdet_destroy(rk.h)


@pytest.fixture(scope="module", autouse=True)
def _close_process_group():
    yield
    import torch.distributed as dist
    if dist.is_available() and dist.is_initialized():
        dist.destroy_process_group()
