"""Pins of the chain-step oracle: the row factor of the rms-norm and the order of the fused pieces."""

import numpy as np
import pytest

import oracle


def test_rms_scale_closed_forms():
    # a constant row c: mean square c^2; a 3-4 row: mean square 12.5
    x = np.full((1, 64), 3.0, np.float16)
    assert np.allclose(oracle.rms_scale(x, 0.0), [1.0 / 3.0], rtol=1e-15)
    assert np.allclose(oracle.rms_scale(x, 7.0), [0.25], rtol=1e-15)
    x = np.array([[3.0, 4.0], [0.0, 0.0]], np.float16)
    r = oracle.rms_scale(x, 0.5)
    assert np.allclose(r, [1.0 / np.sqrt(13.0), 1.0 / np.sqrt(0.5)], rtol=1e-15)


def test_row_scale_by_hand():
    # x = [3, 4], W = [[1], [2]]: x.W = 11; r = 1 / sqrt(12.5); the addend comes after the factor
    x = np.array([[3.0, 4.0]], np.float16)
    w = np.array([[1.0], [2.0]], np.float16)
    y = oracle.matmul(x, w, row_scale=oracle.rms_scale(x, 0.0))
    assert abs(y[0, 0] - 11.0 / np.sqrt(12.5)) < 1e-14
    y = oracle.matmul(x, w, addend_h=np.array([[2.0]], np.float16), row_scale=oracle.rms_scale(x, 0.0))
    assert abs(y[0, 0] - (11.0 / np.sqrt(12.5) + 2.0)) < 1e-14
    # a factor per ROW: a second row with another norm gets its own
    x2 = np.array([[3.0, 4.0], [6.0, 8.0]], np.float16)
    y2 = oracle.matmul(x2, w, row_scale=oracle.rms_scale(x2, 0.0))
    assert np.allclose(y2[:, 0], [11.0 / np.sqrt(12.5), 22.0 / np.sqrt(50.0)], rtol=1e-15)


def test_folded_norm_equals_the_library_norm_followed_by_the_matmul():
    import torch

    rng = np.random.default_rng(3)
    x = rng.normal(0, 1.5, size=(5, 256)).astype(np.float16)
    w = rng.normal(0, 0.02, size=(256, 48)).astype(np.float16)
    eps = 1e-5
    x64, w64 = torch.from_numpy(x.astype(np.float64)), w.astype(np.float64)
    # gain 1: rms_norm(x) . W  ==  r * (x . W)
    ones = torch.ones(256, dtype=torch.float64)
    ref = torch.nn.functional.rms_norm(x64, (256,), ones, eps).numpy() @ w64
    assert np.allclose(oracle.matmul(x, w, row_scale=oracle.rms_scale(x, eps)), ref, rtol=1e-12, atol=1e-14)
    # a gain folded into the weights (gains 1, 2, 4 keep the folded weights exact in fp16):
    # rms_norm(x, gamma) . W  ==  r * (x . (gamma * W))
    gamma = 2.0 ** rng.integers(0, 3, size=256)
    w_folded = (w64 * gamma[:, None]).astype(np.float16)
    assert np.array_equal(w_folded.astype(np.float64), w64 * gamma[:, None])
    ref = torch.nn.functional.rms_norm(x64, (256,), torch.from_numpy(gamma), eps).numpy() @ w64
    got = oracle.matmul(x, w_folded, row_scale=oracle.rms_scale(x, eps))
    assert np.allclose(got, ref, rtol=1e-12, atol=1e-14)


def test_chain_step_strings_the_pinned_pieces_in_order():
    rng = np.random.default_rng(11)
    x = rng.normal(0, 1, size=(3, 128)).astype(np.float16)
    w = rng.normal(0, 0.05, size=(128, 32)).astype(np.float16)
    bias = rng.normal(0, 1, size=32).astype(np.float16)
    res = rng.normal(0, 1, size=(3, 32)).astype(np.float16)
    base = x.astype(np.float64) @ w.astype(np.float64)
    r = oracle.rms_scale(x, 1e-6)[:, None]
    assert np.allclose(oracle.chain_step(x, w), base, rtol=1e-14)
    assert np.allclose(oracle.chain_step(x, w, "bias", bias, rms_eps=1e-6), base * r + bias.astype(np.float64), rtol=1e-13)
    assert np.allclose(oracle.chain_step(x, w, "add", res), base + res.astype(np.float64), rtol=1e-13)
    # the gate sees the scaled product: swiglu(r * Y), not r * swiglu(Y)
    assert np.allclose(oracle.chain_step(x, w, "swiglu", rms_eps=1e-6), oracle.swiglu_blocks(base * r), rtol=1e-13)
    assert not np.allclose(oracle.chain_step(x, w, "swiglu", rms_eps=1e-6), oracle.swiglu_blocks(base) * r, rtol=1e-3)
    with pytest.raises(ValueError):
        oracle.chain_step(x, w, "add")
    with pytest.raises(ValueError):
        oracle.chain_step(x, w, "none", res)
    with pytest.raises(ValueError):
        oracle.chain_step(x, w, "gelu")
