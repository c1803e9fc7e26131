"""The seeded input generator: determinism, distributions, bf16 rounding, the five workloads."""
import math

import numpy as np
import torch

import fgr_inputs as gi


def test_counter_based_and_chunk_independent():
    a = gi.normal(0, gi.TENSOR_X, (1 << 20) + 77)
    b = gi.normal(0, gi.TENSOR_X, 1000)
    np.testing.assert_array_equal(a[:1000], b)                       # element i depends on i only
    assert not np.array_equal(b, gi.normal(1, gi.TENSOR_X, 1000))    # seed matters
    assert not np.array_equal(b, gi.normal(0, gi.TENSOR_W, 1000))    # tensor id matters
    # first draws of seed 0, tensor 1: a change of the generator's definition shows up here
    np.testing.assert_allclose(b[:4], [-0.5278119, 1.2314284, -1.4742856, 0.49102512], rtol=1e-6)


def test_distributions():
    a = gi.normal(3, 1, 1 << 20, std=0.5).astype(np.float64)
    assert abs(a.mean()) < 3e-3 and abs(a.std() - 0.5) < 3e-3
    assert abs(((a / 0.5) ** 4).mean() - 3.0) < 0.05                 # Gaussian kurtosis
    u = gi.uniform(3, 3, 1 << 20, -0.1, 0.1).astype(np.float64)
    assert u.min() >= -0.1 and u.max() <= 0.1
    assert abs(u.mean()) < 3e-4 and abs(u.var() - 0.2 ** 2 / 12) < 1e-5


def test_bf16_rounding_matches_library_rne():
    a = gi.normal(5, 1, 100000, std=3.0)
    a[:6] = [0.0, 1.0, 1.00390625, 1.01171875, -1.00390625, 3.3895314e38]   # ties go to even
    bits = gi.f32_to_bf16_bits(a)
    ref = torch.from_numpy(a).to(torch.bfloat16)
    np.testing.assert_array_equal(bits.view(np.int16), ref.view(torch.int16).numpy())
    np.testing.assert_array_equal(gi.bf16_bits_to_f32(bits), ref.float().numpy())


def test_named_workloads():
    c1 = gi.make_config("c1")
    assert c1.X.shape == (1, 256, 256) and c1.X.dtype == np.float32 and c1.bias.shape == (256,)
    assert abs(c1.X.std() - 1 / 16) < 1e-3 and c1.reduce == gi.RED_LSE and c1.act == gi.ACT_GELU_TANH
    shapes = {k: gi.make_config(k, materialize=False) for k in gi.CONFIGS}
    assert shapes["c2"].flop == 2 * 4096 ** 3 and shapes["c2"].write_y == 1
    assert shapes["c3"].bias is None and shapes["c3"].scale == 1 / math.sqrt(2048)
    assert shapes["c4"].min_bytes() == 2 * 16384 * 8192 + 2 * 128 * 8192 + 4 * 16384 + 4 * 128
    assert shapes["c5"].batch == 32 and shapes["c5"].out_width == 2
    small = gi.make_config("c5", batch=2, M=8, N=16, K=8)
    assert small.X.dtype == np.uint16 and small.W.shape == (2, 16, 8)
