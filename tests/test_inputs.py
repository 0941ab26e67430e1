"""The seeded input generator (numpy side): determinism, statistics, exact bf16 rounding."""
import numpy as np
import torch

from hdet_inputs import generator as G
from hdet_inputs import recipes as R
from hdet_inputs import workloads as W


def test_mix64_vectorised_matches_scalar():
    xs = [0, 1, 1234567, (1 << 64) - 1, 0x9E3779B97F4A7C15]
    got = G.mix64(np.array(xs, dtype=np.uint64))
    assert [int(v) for v in got] == [G._mix64_int(x) for x in xs]


def test_normal_int_statistics_and_slab_consistency():
    key = G.stream_key(1, G.STREAM_GRAD, 3, 2)
    z = G.normal_int(key, 0, 400000)
    assert z.min() >= -131070 and z.max() <= 131070
    assert abs(z.mean()) < 3 * G.IRWIN_HALL_STD / np.sqrt(z.size) * 1.5
    assert abs(z.std() / G.IRWIN_HALL_STD - 1) < 5e-3
    # a slab equals the same indices of a longer run
    assert np.array_equal(G.normal_int(key, 1000, 77), z[1000:1077])
    # different cells differ
    assert not np.array_equal(z[:100], G.normal_int(G.stream_key(1, G.STREAM_GRAD, 3, 3), 0, 100))
    assert not np.array_equal(z[:100], G.normal_int(G.stream_key(1, G.STREAM_GRAD, 4, 2), 0, 100))


def test_bf16_rounding_matches_library_conversion():
    key = G.stream_key(9, G.STREAM_GRAD, 0, 0)
    x = G.fill_f32(key, 0, 100000, G.scale_for_sigma(1e-3))
    bits = G.f32_to_bf16_bits(x)
    lib = torch.from_numpy(x).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)
    assert np.array_equal(bits, lib)
    wide = G.bf16_bits_to_f32(bits)
    assert np.array_equal(wide, torch.from_numpy(x).to(torch.bfloat16).float().numpy())


def test_workload_sizes_match_the_stated_configurations():
    assert W.config1().numel == 1_000_000
    assert W.config2().numel == 25_190_400 and len(W.config2().tensors) == 24
    assert W.config3().numel == 354_823_168 and len(W.config3().tensors) == 292
    assert W.config4().numel == 1_315_723_264 and len(W.config4().tensors) == 292
    assert W.config5().numel == 124_439_808 and len(W.config5().tensors) == 148
    w = W.ragged_workload()
    offs = w.arena_offsets()
    assert all(o % 8 == 0 for o in offs) and w.arena_numel() >= w.numel


def test_loss_recipes():
    w = W.config2()
    a = R.step_losses(w, 5)
    assert a.shape == (8,) and np.all(np.diff(a) < 0.05)      # higher rate (higher rank) -> lower loss
    b = R.step_losses(w, 5, [7, 6, 5, 4, 3, 2, 1, 0])
    assert b[0] < b[-1]
    u = R.step_losses(W.config1(), 2)
    assert np.all((u >= 2.0) & (u < 3.0))
    assert np.array_equal(R.step_losses(w, 5), a)
