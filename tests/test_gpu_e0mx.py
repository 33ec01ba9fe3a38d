"""GPU parity of E0M3 and E0M5 (Section 2.3: the construction with three or five fraction bits kept):
quantizer, container and dequantizer bit for bit, the matmul at decode and prefill sizes within the
matmul tolerance, against the oracle run with bits=3 / bits=5."""

import numpy as np
import pytest
import torch

import oracle
from paper_2403_20041_b200 import workloads
from test_gpu_parity import _to_np, _words, assert_matmul_close

pytestmark = pytest.mark.gpu
BITS = [3, 5]


@pytest.fixture(scope="module")
def dev():
    return torch.device("cuda:0")


def _quantized(lib, dev, w_np, bits):
    packed, scales = lib.tl_e0mx_quantize(torch.from_numpy(w_np).to(dev), bits)
    torch.cuda.synchronize()
    return packed, scales, oracle.quantize(w_np, bits=bits)


@pytest.mark.parametrize("bits", BITS)
@pytest.mark.parametrize("K,N", [(128, 16), (384, 48), (1408, 272), (2048, 256), (4096, 1024)])
@pytest.mark.parametrize("dtype", [np.float32, np.float16])
def test_quantize_and_dequant_bit_exact(lib, dev, K, N, dtype, bits):
    w_np = workloads.weights(K, N, seed=workloads.seed_for("e0mx", K, N, bits)).astype(dtype)
    packed, scales, (codes, d_h, b_h) = _quantized(lib, dev, w_np, bits)
    assert (packed.numel(), scales.numel()) == oracle.packed_sizes(K, N, bits=bits)
    assert int(codes.max()) == (1 << bits) - 1
    ref_p, ref_s = oracle.pack(codes, d_h, b_h, bits=bits)
    assert np.array_equal(_words(packed), ref_p)
    assert np.array_equal(_words(scales), ref_s)
    w_hat = lib.tl_e0mx_dequant(packed, scales, K, N, bits)
    torch.cuda.synchronize()
    assert np.array_equal(_to_np(w_hat).view(np.uint16), oracle.dequantize(codes, d_h, b_h, bits=bits).view(np.uint16))


@pytest.mark.parametrize("bits", BITS)
def test_degenerate_groups(lib, dev, bits):
    rng = np.random.default_rng(bits)
    w = rng.normal(0, 0.02, size=(256, 32)).astype(np.float32)
    w[:128, 0] = 0.0                                   # a dead group
    w[:128, 1] = 0.375                                 # one-sided constant group
    w[128:, 2] = -np.abs(w[128:, 2]) - 0.1             # all negative
    w[128:, 3] = np.linspace(-1, 1, 128, dtype=np.float32) * 3e5   # the scale saturates
    w[:128, 4] = np.linspace(-1, 1, 128, dtype=np.float32) * 1e-7  # the scale is an fp16 subnormal
    steps = 1 << bits
    w[:128, 5] = -0.5 + (np.arange(128) % steps) / steps + 0.5 / steps   # ties between neighbouring codes
    w[0, 5], w[1, 5] = -0.5, -0.5 + (2.0 - 2.0 ** -9)
    packed, scales, (codes, d_h, b_h) = _quantized(lib, dev, w, bits)
    ref_p, ref_s = oracle.pack(codes, d_h, b_h, bits=bits)
    assert np.array_equal(_words(packed), ref_p)
    assert np.array_equal(_words(scales), ref_s)
    w_hat = _to_np(lib.tl_e0mx_dequant(packed, scales, 256, 32, bits))
    assert np.array_equal(w_hat.view(np.uint16), oracle.dequantize(codes, d_h, b_h, bits=bits).view(np.uint16))
    assert not w_hat[:128, 0].any()


@pytest.mark.parametrize("bits", BITS)
@pytest.mark.parametrize("M", [1, 3, 8, 9, 16, 40, 128, 144, 300, 520])
def test_matmul_matches_oracle(lib, dev, M, bits):
    K, N = 1408, 272  # 11 tile rows, a ragged panel of one column block
    w_np = workloads.weights(K, N, seed=workloads.seed_for("e0mx-mm", M, bits))
    x_np = workloads.activations(M, K, seed=7, outlier_fraction=0.01 if M > 16 else 0.0)
    packed, scales, (codes, d_h, b_h) = _quantized(lib, dev, w_np, bits)
    y = lib.tl_e0mx_matmul(torch.from_numpy(x_np).to(dev), packed, scales, N, bits)
    torch.cuda.synchronize()
    assert_matmul_close(_to_np(y), oracle.matmul(x_np, oracle.dequantize(codes, d_h, b_h, bits=bits)))
    assert lib.tl_e0m4_device_status() == 0


@pytest.mark.parametrize("bits", BITS)
def test_unit_activation_returns_the_dequantized_row(lib, dev, bits):
    # with x = e_k the product is row k of the dequantized weight, bit for bit
    K, N, M = 512, 144, 4
    w_np = workloads.weights(K, N, seed=workloads.seed_for("e0mx-unit", bits))
    packed, scales, (codes, d_h, b_h) = _quantized(lib, dev, w_np, bits)
    w_hat = oracle.dequantize(codes, d_h, b_h, bits=bits)
    ks = [0, 1, 7, 8, 63, 64, 100, 127, 128, 300, 511]
    for k0 in range(0, len(ks), M):
        sel = ks[k0:k0 + M]
        x = np.zeros((M, K), np.float16)
        for m, k in enumerate(sel):
            x[m, k] = 1.0
        y = _to_np(lib.tl_e0mx_matmul(torch.from_numpy(x).to(dev), packed, scales, N, bits))
        for m, k in enumerate(sel):
            assert np.array_equal(y[m].view(np.uint16), w_hat[k].view(np.uint16)), (bits, k)


@pytest.mark.parametrize("bits", BITS)
@pytest.mark.parametrize("M,K,N", [(1, 4096, 4096), (16, 13696, 1040), (512, 4096, 4608), (2048, 2048, 16384)])
def test_config_sized_sampled(lib, dev, M, K, N, bits):
    w = workloads.weights_torch(K, N, workloads.seed_for("e0mx-cfg", K, N, bits), dev)
    x = workloads.activations_torch(M, K, 3, dev, outlier_fraction=0.01 if M > 16 else 0.0)
    packed, scales = lib.tl_e0mx_quantize(w, bits)
    ws = lib.tl_e0m4_workspace(max(int(lib.lib().tl_e0mx_matmul_workspace(M, K, N, bits)), 256), dev)
    y = lib.tl_e0mx_matmul(x, packed, scales, N, bits, workspace=ws)
    torch.cuda.synchronize()
    assert not _to_np(ws).any()
    rng = np.random.default_rng(bits)
    nbs = sorted(set([0, N // 16 - 1] + rng.integers(0, N // 16, size=8).tolist()))
    cols = np.concatenate([np.arange(nb * 16, nb * 16 + 16) for nb in nbs])
    rows = np.arange(M) if M <= 64 else np.unique(np.concatenate([[0, M - 1], rng.integers(0, M, size=24)]))
    codes, d_h, b_h = oracle.quantize(_to_np(w[:, torch.from_numpy(cols).to(dev)]), bits=bits)
    y_ref = oracle.matmul(_to_np(x)[rows], oracle.dequantize(codes, d_h, b_h, bits=bits))
    assert_matmul_close(_to_np(y)[np.ix_(rows, cols)], y_ref)
    assert lib.tl_e0m4_device_status() == 0


def test_mean_absolute_error_halves_per_bit(lib, dev):
    # the error of the GPU round trip falls about 2x per kept bit: E0M3 > E0M4 > E0M5 > E0M8
    K, N = 2048, 512
    w = workloads.weights_torch(K, N, 99, dev)
    mae = {}
    for bits in (3, 5):
        mae[bits] = float((lib.tl_e0mx_dequant(*lib.tl_e0mx_quantize(w, bits), K, N, bits).float() - w).abs().mean())
    mae[4] = float((lib.tl_e0m4_dequant(*lib.tl_e0m4_quantize(w), K, N).float() - w).abs().mean())
    mae[8] = float((lib.tl_e0m8_dequant(*lib.tl_e0m8_quantize(w), K, N).float() - w).abs().mean())
    assert 1.7 < mae[3] / mae[4] < 2.3 and 1.7 < mae[4] / mae[5] < 2.3 and 6.0 < mae[5] / mae[8] < 10.0


def test_argument_errors(lib, dev):
    L = lib.lib()
    a = 0x10000
    assert L.tl_e0mx_quantize(a, 0, 128, 16, 128, 4, a, a, None) == 2   # bits must be 3 or 5
    assert L.tl_e0mx_quantize(a, 0, 128, 16, 64, 5, a, a, None) == 2    # groups of 128 only
    assert L.tl_e0mx_dequant(a, a, 128, 16, 128, 5, None, None) == 1
    assert L.tl_e0mx_matmul(a, a, a, a, 1, 128, 16, 128, 6, None, 0, None) == 2
    assert lib.tl_e0mx_packed_sizes(4096, 4096, 5) == (4096 * 4096 * 5 // 8, 32 * 4096 * 4)
    assert lib.tl_e0mx_packed_sizes(4096, 4096, 3) == (4096 * 4096 * 3 // 8, 32 * 4096 * 4)
