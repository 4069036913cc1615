"""Pins for the layer oracle (linear, RMSNorm, rotary embedding, SwiGLU)."""
import numpy as np
import pytest
import torch

from oracle import sdlm_layer_oracle as lo


def test_linear_is_torch_matmul_and_identity_weights_copy_the_input():
    rng = np.random.default_rng(0)
    x, w, b, r = rng.normal(size=(5, 24)), rng.normal(size=(16, 24)), rng.normal(size=16), rng.normal(size=(5, 16))
    ref = torch.from_numpy(x) @ torch.from_numpy(w).T + torch.from_numpy(b) + torch.from_numpy(r)
    assert np.allclose(lo.linear(x, w, b, r), ref.numpy(), rtol=0, atol=1e-13)
    assert np.array_equal(lo.linear(x, np.eye(24)), x)
    assert np.allclose(lo.linear(x, w), (torch.from_numpy(x) @ torch.from_numpy(w).T).numpy(), rtol=0, atol=1e-13)


def test_rms_norm_against_torch_constant_rows_and_rescaling():
    rng = np.random.default_rng(1)
    x, g = rng.normal(size=(7, 40)), rng.normal(size=40)
    ref = torch.nn.functional.rms_norm(torch.from_numpy(x), (40,), torch.from_numpy(g), 1e-6).numpy()
    assert np.allclose(lo.rms_norm(x, g, 1e-6), ref, rtol=0, atol=1e-13)
    const = np.full((2, 16), -3.0)
    assert np.allclose(lo.rms_norm(const, np.ones(16), 0.0), -1.0)               # x / |x|
    assert np.allclose(lo.rms_norm(17.0 * x, g, 0.0), lo.rms_norm(x, g, 0.0), rtol=1e-13, atol=0)   # scale-free when eps = 0


def test_rope_is_a_complex_rotation_of_the_pairs_and_preserves_norms():
    rng = np.random.default_rng(2)
    d, theta = 16, 10000.0
    x = rng.normal(size=(3, 4, 2, d))                         # [B, D, heads, d]
    pos = rng.integers(0, 5000, size=(3, 4))
    y = lo.rope(x, pos, theta)
    z = x[..., :d // 2] + 1j * x[..., d // 2:]
    ang = pos[..., None, None] * theta ** (-2.0 * np.arange(d // 2) / d)
    zr = z * np.exp(1j * ang)
    assert np.allclose(y[..., :d // 2], zr.real, atol=1e-12) and np.allclose(y[..., d // 2:], zr.imag, atol=1e-12)
    assert np.allclose(np.linalg.norm(y, axis=-1), np.linalg.norm(x, axis=-1), rtol=1e-12)
    assert np.array_equal(lo.rope(x, np.zeros((3, 4)), theta), x)


def test_rope_scores_depend_on_the_position_difference_only():
    rng = np.random.default_rng(3)
    d, theta = 32, 1.0e6
    q, k = rng.normal(size=(1, 1, 1, d)), rng.normal(size=(1, 1, 1, d))
    def score(m, n):
        return float(np.sum(lo.rope(q, np.array([[m]]), theta) * lo.rope(k, np.array([[n]]), theta)))
    assert abs(score(10, 3) - score(1007, 1000)) < 1e-9
    assert abs(score(5, 5) - float(np.sum(q * k))) < 1e-12
    assert abs(score(10, 3) - score(3, 10)) > 1e-6            # not symmetric: the sign of the offset matters


def test_swiglu_against_torch_silu_and_limits():
    rng = np.random.default_rng(4)
    gu = rng.normal(size=(6, 20)) * 3
    ref = torch.nn.functional.silu(torch.from_numpy(gu[:, :10])) * torch.from_numpy(gu[:, 10:])
    assert np.allclose(lo.swiglu(gu), ref.numpy(), rtol=0, atol=1e-14)
    assert np.array_equal(lo.swiglu(np.concatenate([np.zeros((1, 4)), np.ones((1, 4))], axis=1)), np.zeros((1, 4)))
    big = np.concatenate([np.full((1, 2), 50.0), np.full((1, 2), 2.5)], axis=1)
    assert np.allclose(lo.swiglu(big), 125.0)                 # silu(g) -> g for large g
    neg = np.concatenate([np.full((1, 2), -50.0), np.full((1, 2), 2.5)], axis=1)
    assert np.all(np.abs(lo.swiglu(neg)) < 1e-18)             # and -> 0 for very negative g


def test_bf16_rounding_helper_is_nearest_even():
    vals = np.array([1.0, 1.0 + 2 ** -8, 1.0 + 2 ** -7, 1.0 + 3 * 2 ** -8, -0.3, 3.0e38])
    want = torch.tensor(vals, dtype=torch.float32).to(torch.bfloat16).to(torch.float64).numpy()
    assert np.array_equal(lo.round_bf16(vals), want)
    bits = torch.tensor(vals, dtype=torch.float32).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)
    assert np.array_equal(lo.to_bits(vals), bits)
