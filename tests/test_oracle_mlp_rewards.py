"""Pins for oracle/mlp.py and oracle/rewards.py against library routines."""
import numpy as np
import torch
from scipy.spatial import distance

from oracle import mlp, rewards
from workloads import CONFIGS, make_inputs, bf16_bits


def test_bf16_round_equals_torch_cast():
    rng = np.random.default_rng(0)
    x = np.concatenate([rng.standard_normal(4096).astype(np.float32) * 10.0 ** rng.integers(-6, 6, 4096),
                        np.array([0.0, -0.0, 1.0, 1.00390625, 1.01171875, 3.3895314e38, 1e-40], dtype=np.float32)])
    ref = torch.from_numpy(x).to(torch.bfloat16).to(torch.float32).numpy()
    assert np.array_equal(mlp.bf16_round(x).view(np.uint32), ref.view(np.uint32))


def test_gelu_equals_torch():
    x = np.linspace(-6, 6, 1001)
    ref = torch.nn.functional.gelu(torch.from_numpy(x), approximate="none").numpy()
    assert np.allclose(mlp.gelu_erf(x), ref, rtol=1e-13, atol=1e-15)


def test_mlp_equals_float64_library_composition():
    w = CONFIGS["image"].scaled(hidden=256)
    inp = make_inputs(w)
    rng = np.random.default_rng(1)
    z = rng.standard_normal((37, 64)).astype(np.float32)
    got = mlp.mlp_velocity(z, inp.W1, inp.W2, chunk=16)
    zt = torch.from_numpy(z).to(torch.bfloat16).to(torch.float64)
    h = zt @ torch.from_numpy(inp.W1.astype(np.float64))
    a = torch.nn.functional.gelu(h).to(torch.float32).to(torch.bfloat16).to(torch.float64)
    ref = (a @ torch.from_numpy(inp.W2.astype(np.float64))).to(torch.float32).numpy()
    assert np.array_equal(got, ref)
    assert got.dtype == np.float32 and got.shape == (37, 64)


def test_mlp_special_cases():
    z = np.random.default_rng(2).standard_normal((5, 4)).astype(np.float32)
    assert np.all(mlp.mlp_velocity(z, np.zeros((4, 8)), np.zeros((8, 4))) == 0)
    # W1 = [I, -I], W2 = [I; -I]:  v = GELU(zb) - GELU(-zb) = zb  (GELU(x) - GELU(-x) = x), up to bf16 rounding of GELU
    W1 = np.concatenate([np.eye(4), -np.eye(4)], axis=1)
    W2 = np.concatenate([np.eye(4), -np.eye(4)], axis=0)
    v = mlp.mlp_velocity(z, W1, W2)
    assert np.allclose(v, mlp.bf16_round(z), rtol=2 ** -7, atol=1e-3)
    # a transposed weight matrix must not pass
    W1r = np.random.default_rng(3).standard_normal((4, 8))
    assert mlp.mlp_velocity(z, W1r, W2).shape == (5, 4)


def test_weights_are_bf16_values():
    inp = make_inputs(CONFIGS["image"].scaled(hidden=128))
    assert np.array_equal(mlp.bf16_round(inp.W1), inp.W1)
    assert bf16_bits(inp.W2).dtype == np.uint16
    assert abs(inp.W1.std() - 0.02) < 2e-3


def test_rewards_equal_library():
    rng = np.random.default_rng(4)
    a = rng.standard_normal(1000).astype(np.float32)
    b = rng.standard_normal(1000).astype(np.float32)
    assert np.isclose(rewards.cosine(a, b), 1.0 - distance.cosine(a.astype(np.float64), b.astype(np.float64)), rtol=1e-12)
    assert np.isclose(rewards.neg_mse(a, b), -distance.sqeuclidean(a.astype(np.float64), b.astype(np.float64)) / 1000, rtol=1e-12)
    assert rewards.neg_mse(a, a) == 0.0 and np.isclose(rewards.cosine(a, -2 * a), -1.0)
