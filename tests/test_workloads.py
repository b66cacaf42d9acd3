"""Shapes and generators of the synthetic workloads."""
import numpy as np

import workloads as W


def test_model_sizes():
    assert sum(t.numel for t in W.gptneo_8m_shape()) == 8_415_744 and len(W.gptneo_8m_shape()) == 99
    assert sum(t.numel for t in W.resnet50_shape()) == 25_557_032 and len(W.resnet50_shape()) == 161
    assert sum(t.numel for t in W.gptneo_125m_shape()) == 125_226_240 and len(W.gptneo_125m_shape()) == 148
    assert W.get_config("c0_flat_1m").P == 1 << 20


def test_generators_are_seeded_and_order_independent():
    a = W.grads_host(1000, 5678, 3, 2, 0.01)
    _ = W.grads_host(1000, 5678, 9, 1, 0.01)
    b = W.grads_host(1000, 5678, 3, 2, 0.01)
    assert np.array_equal(a, b) and a.dtype == np.float32
    assert not np.array_equal(a, W.grads_host(1000, 5678, 3, 3, 0.01))
    assert abs(a.std() - 0.01) < 1e-3
    x = W.init_params_host(W.resnet50_shape()[:6], 1234, 0.02)
    assert np.all(x[9408:9408 + 64] == 1.0) and np.all(x[9408 + 64:9408 + 128] == 0.0)


def test_bf16_inputs_are_exactly_representable():
    g = W.grads_host(4096, 1, 0, 0, 0.01)
    h = W.bf16_bits_from_f32_host(g)
    back = (h.astype(np.uint32) << 16).view(np.float32)
    assert np.all(np.abs(back - g) <= np.abs(g) * 2.0 ** -7)
    assert np.array_equal(W.bf16_bits_from_f32_host(back), h)


def test_sample_indices_cover_tensor_edges():
    ts = W.gptneo_8m_shape()
    idx = W.sample_indices(ts, 1000, 1)
    assert idx[0] == 0 and idx[-1] == sum(t.numel for t in ts) - 1
    assert np.all(np.diff(idx) > 0)
    off = ts[0].numel
    assert off in idx and off - 1 in idx


def test_sweep_has_192_points_and_respects_memory_cap():
    assert len(list(W.sweep_points())) == 192
    assert all(c.K * c.P * 16 + 8 * c.P <= 2**34 for c in W.sweep_points(2**34))
