"""hdet_converge_static: the replica mean for callers that cannot allocate device memory.

Some users of the library run where cudaMalloc is off limits when the mean is needed: a framework's
caching pool already owns the whole device, or the call sits in a loop that must not risk the
device-wide synchronisation an allocation can trigger.  hdet_converge_static keeps its work tables in
a static device array instead.  These tests call it through the C ABI and check it against the
ordinary entry point (hdet_converge on a handle), twice in a row with different tensor lists, because
the static array still holds the first call's tables when the second call starts.

This file sorts last on purpose: a run that stops at the first failure has then run everything else.
"""
import numpy as np
import pytest

from paper_2604_24708_b200 import binding as B


def _desc(numel, stride=None, param=0x10000):
    return B.hdet_tensor(param=param, numel=numel, param_stride=stride or numel)


def test_static_limits_are_rejected_with_a_message_before_touching_the_device():
    too_many = [_desc(8) for _ in range(B.HDET_STATIC_MAX_TENSORS + 1)]
    with pytest.raises(B.HdetError) as e:
        B.hdet_converge_static(too_many, 4)
    assert e.value.status == B.HDET_ERR_UNSUPPORTED and "1024" in e.value.message
    too_big = [_desc(2048 * B.HDET_STATIC_MAX_TILES + 1)]
    with pytest.raises(B.HdetError) as e:
        B.hdet_converge_static(too_big, 4)
    assert e.value.status == B.HDET_ERR_UNSUPPORTED and "65536" in e.value.message
    for bad, status in [([_desc(0)], B.HDET_ERR_INVALID_ARG), ([_desc(100, stride=50)], B.HDET_ERR_INVALID_ARG),
                        ([_desc(100, param=0x10002)], B.HDET_ERR_ALIGN), ([_desc(100, param=None)], B.HDET_ERR_INVALID_ARG)]:
        with pytest.raises(B.HdetError) as e:
            B.hdet_converge_static(bad, 4)
        assert e.value.status == status
    with pytest.raises(B.HdetError):
        B.hdet_converge_static([_desc(8)], 0)
    with pytest.raises(B.HdetError):
        B.hdet_converge_static([_desc(8)], 33)
    B.hdet_converge_static([], 4)          # nothing to do, no device needed


@pytest.mark.gpu
def test_static_converge_matches_the_handle_entry_point_on_two_calls_in_a_row():
    import torch
    from paper_2604_24708_b200.arena import StackedArena

    def make(numels, n, seed, align):
        a = StackedArena(numels, [0] * len(numels), n, B.HDET_OPT_SGD, B.HDET_DTYPE_F32, align_elems=align)
        g = torch.Generator(device="cuda").manual_seed(seed)
        a.param.copy_(torch.randn(a.param.shape, generator=g, device="cuda"))
        return a

    def reference(a, n, align):
        """The existing entry point: hdet_converge on a handle, run on a copy of the parameters."""
        b = StackedArena(a.numels, a.groups, n, B.HDET_OPT_SGD, B.HDET_DTYPE_F32, align_elems=align)
        assert b.offsets == a.offsets
        b.param.copy_(a.param)
        cfg = B.hdet_config(n_replicas=n, n_groups=1, optimizer=B.HDET_OPT_SGD, grad_dtype=B.HDET_DTYPE_F32,
                            sync_interval=1, fuse_converge=1, device=0)
        h = B.hdet_create(cfg, b.descriptors())
        B.hdet_converge(h)
        torch.cuda.synchronize()
        B.hdet_destroy(h)
        return b.param

    # first call: a long ragged list (vector path, tails); second call: a shorter list with odd
    # offsets (scalar path) and another replica count, so stale tables from call 1 would show.
    first = make([4099, 2048, 3, 70001, 1, 12289], 8, 1, 8)
    second = make([5, 2051, 33, 6151], 3, 2, 1)      # 6151 elements: four tiles on the scalar path
    before_first = first.param.double().cpu().numpy()
    want_first, want_second = reference(first, 8, 8), reference(second, 3, 1)
    stream = torch.cuda.current_stream().cuda_stream
    B.hdet_converge_static(first.descriptors(), 8, 0, stream)
    B.hdet_converge_static(second.descriptors(), 3, 0, stream)
    torch.cuda.synchronize()
    for got, want in ((first.param, want_first), (second.param, want_second)):
        g, w = got.double().cpu().numpy(), want.double().cpu().numpy()
        assert np.max(np.abs(g - w) / np.maximum(np.abs(w), 1.0)) <= 1e-7
        assert torch.equal(got, want)              # same arithmetic in the same order: bitwise equal
    # the mean really was taken: all replicas equal, and close to the float64 mean of the inputs
    # (padding between tensors belongs to no tensor and must be left alone)
    used = np.zeros(first.p_pad, dtype=bool)
    for off, ne in zip(first.offsets, first.numels):
        used[off:off + ne] = True
    after_first = first.param.double().cpu().numpy()
    assert np.all(after_first[:, used] == after_first[0:1, used])
    assert np.array_equal(after_first[:, ~used], before_first[:, ~used])
    assert np.max(np.abs(after_first[0, used] - before_first.mean(axis=0)[used])) <= 1e-6
    # a third call on the first list again is idempotent
    B.hdet_converge_static(first.descriptors(), 8, 0, stream)
    torch.cuda.synchronize()
    assert torch.equal(first.param, want_first)
    # what the entry point is for: further calls leave the device's free memory exactly as it was
    # (the first call above already loaded the module and resolved the array's address)
    free_before = torch.cuda.mem_get_info()[0]
    B.hdet_converge_static(first.descriptors(), 8, 0, stream)
    B.hdet_converge_static(second.descriptors(), 3, 0, stream)
    torch.cuda.synchronize()
    assert torch.cuda.mem_get_info()[0] == free_before
    # a capturing stream is refused (the tables come from host memory that does not outlive the call),
    # and the refusal leaves the capture usable
    side = torch.cuda.Stream()
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph, stream=side):
        with pytest.raises(B.HdetError) as e:
            B.hdet_converge_static(second.descriptors(), 3, 0, torch.cuda.current_stream().cuda_stream)
        assert e.value.status == B.HDET_ERR_UNSUPPORTED and "captured" in e.value.message
        second.param.add_(0.0)                  # something for the graph to hold
    torch.cuda.synchronize()
