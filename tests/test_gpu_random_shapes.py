"""GPU parity on seeded random shapes: single calls with every fused epilogue, lists and chains,
against the oracle on WHOLE outputs.

The parametrized tests elsewhere pick their shapes by hand; here a seeded generator draws token
counts, K, N, group size and epilogue together, so that combinations nobody thought of (a ragged
last panel with a ragged last stage at three tokens and group 32, say) are exercised as well.
Sizes stay small enough for the oracle to recompute every output element.
Tolerance: max|y - y_ref| <= 1e-2 max|y_ref| and relative Frobenius error <= 1e-3.
"""

import numpy as np
import pytest

import oracle
from paper_2403_20041_b200 import workloads

torch = pytest.importorskip("torch")
pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def dev():
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    return torch.device("cuda:0")


def _np(t):
    return t.detach().cpu().numpy()


def assert_close(y, y_ref):
    y = np.asarray(y, dtype=np.float64)
    assert np.isfinite(y).all()
    scale = np.abs(y_ref).max()
    assert np.abs(y - y_ref).max() <= 1e-2 * scale
    assert np.linalg.norm(y - y_ref) / np.linalg.norm(y_ref) <= 1e-3


def _draw(rng, max_m=40):
    group = int(rng.choice([128, 128, 64, 32]))
    K = 128 * int(rng.integers(1, 25))            # up to 3072, any number of groups (ragged stages)
    N = 16 * int(rng.integers(1, 100))            # up to 1584, mostly not a multiple of 128
    M = int(rng.choice([1, 1, 2, 3, 4, 5, 7, 8, 9, 12, 16, int(rng.integers(17, max_m + 1))]))
    return M, K, N, group


def _w_hat(w_np, group):
    return oracle.dequantize(*oracle.quantize(w_np, group=group), group=group)


@pytest.mark.parametrize("case", range(48))
def test_single_call_with_a_random_epilogue(lib, dev, case):
    rng = np.random.default_rng(workloads.seed_for("random single", case))
    M, K, N, group = _draw(rng)
    epi = ["none", "add", "bias", "swiglu"][case % 4]
    if epi == "swiglu":
        N = 16 * max(1, N // 16)  # gate/up alternate in blocks of eight columns: any multiple of 16
    w_np = workloads.weights(K, N, workloads.seed_for("random single w", case))
    x_np = workloads.activations(M, K, workloads.seed_for("random single x", case))
    packed, scales = lib.tl_e0m4_quantize(torch.from_numpy(w_np).to(dev), group=group)
    x = torch.from_numpy(x_np).to(dev)
    w_hat = _w_hat(w_np, group)
    if epi == "none":
        y = lib.tl_e0m4_matmul(x, packed, scales, N, group=group)
        ref = oracle.matmul(x_np, w_hat)
    elif epi == "add":
        a_np = workloads.activations(M, N, workloads.seed_for("random single a", case))
        y = lib.tl_e0m4_matmul_add(x, packed, scales, N, torch.from_numpy(a_np).to(dev),
                                   y=torch.empty((M, N), dtype=torch.float16, device=dev), group=group)
        ref = oracle.matmul(x_np, w_hat, a_np)
    elif epi == "bias":
        b_np = workloads.activations(1, N, workloads.seed_for("random single b", case))[0].copy()
        y = lib.tl_e0m4_matmul_bias(x, packed, scales, N, torch.from_numpy(b_np).to(dev), group=group)
        ref = oracle.matmul(x_np, w_hat, b_np)
    else:
        y = lib.tl_e0m4_matmul_swiglu(x, packed, scales, N, group=group)
        ref = oracle.swiglu_blocks(oracle.matmul(x_np, w_hat))
    torch.cuda.synchronize()
    assert lib.tl_e0m4_device_status() == 0
    assert_close(_np(y), ref)


@pytest.mark.parametrize("case", range(12))
def test_list_of_random_problems(lib, dev, case):
    """One tl_e0m4_matmul_batch call over 3..40 problems of unrelated shapes (one M and group per call)."""
    rng = np.random.default_rng(workloads.seed_for("random list", case))
    M, _, _, group = _draw(rng, max_m=64)
    count = int(rng.integers(3, 41))
    probs, refs = [], []
    for j in range(count):
        _, K, N, _ = _draw(rng)
        w_np = workloads.weights(K, N, workloads.seed_for("random list w", case, j))
        x_np = workloads.activations(M, K, workloads.seed_for("random list x", case, j))
        packed, scales = lib.tl_e0m4_quantize(torch.from_numpy(w_np).to(dev), group=group)
        y = torch.full((M, N), float("nan"), dtype=torch.float16, device=dev)
        probs.append((torch.from_numpy(x_np).to(dev), packed, scales, y))
        refs.append(oracle.matmul(x_np, _w_hat(w_np, group)))
    ws = lib.tl_e0m4_workspace(lib.tl_e0m4_matmul_batch_workspace(), dev)
    lib.tl_e0m4_matmul_batch(probs, M, ws, group=group)
    torch.cuda.synchronize()
    assert lib.tl_e0m4_device_status() == 0
    assert not _np(ws).any()
    for (_, _, _, y), ref in zip(probs, refs):
        assert_close(_np(y), ref)


@pytest.mark.parametrize("case", range(10))
def test_chain_of_random_steps(lib, dev, case):
    """A chain whose steps feed one another (x of a step = y of the one before, so K follows N),
    with a random epilogue and sometimes a folded rms-norm per step; every step is checked against
    the oracle on the fp16 input the GPU really gave it."""
    rng = np.random.default_rng(workloads.seed_for("random chain", case))
    M = int(rng.integers(1, 9))
    group = int(rng.choice([128, 64, 32]))
    steps_n = int(rng.integers(2, 9))
    K = 128 * int(rng.integers(1, 13))
    x = torch.from_numpy(workloads.activations(M, K, workloads.seed_for("random chain x", case))).to(dev)
    steps, w_hats = [], []
    for j in range(steps_n):
        epi = str(rng.choice(["none", "add", "bias", "swiglu"]))
        N_out = 128 * int(rng.integers(1, 13))       # the next step's K: a multiple of 128
        N = 2 * N_out if epi == "swiglu" else N_out   # the joined gate/up projection is twice as wide
        # a small gain keeps the values of a long chain inside fp16
        w_np = workloads.weights(K, N, workloads.seed_for("random chain w", case, j), std=1.0 / np.sqrt(K))
        packed, scales = lib.tl_e0m4_quantize(torch.from_numpy(w_np).to(dev), group=group)
        y = torch.full((M, N_out), float("nan"), dtype=torch.float16, device=dev)
        st = dict(x=x, packed=packed, scales=scales, y=y, epilogue=epi, after_previous=True)
        if epi == "add":
            st["addend"] = torch.from_numpy(workloads.activations(M, N, workloads.seed_for("random chain a", case, j))).to(dev)
        elif epi == "bias":
            st["addend"] = torch.from_numpy(
                workloads.activations(1, N, workloads.seed_for("random chain b", case, j))[0].copy()).to(dev)
        if rng.random() < 0.5:
            st["rms_eps"] = 1e-5
        steps.append(st)
        w_hats.append(_w_hat(w_np, group))
        x, K = y, N_out
    ws = lib.tl_e0m4_workspace(lib.tl_e0m4_matmul_chain_workspace(), dev)
    lib.tl_e0m4_matmul_chain(steps, M, ws, group=group)
    torch.cuda.synchronize()
    assert lib.tl_e0m4_device_status() == 0
    assert not _np(ws).any()
    for st, w_hat in zip(steps, w_hats):
        epi = st["epilogue"]
        addend = _np(st["addend"]) if "addend" in st else None
        ref = oracle.chain_step(_np(st["x"]), w_hat, epi, addend, st.get("rms_eps"))
        assert_close(_np(st["y"]), ref)


@pytest.mark.parametrize("case", range(16))
def test_single_call_at_prefill_sizes(lib, dev, case):
    """41..700 tokens: the tensor-core kernel's token tiles, split-K, pairs of CTAs and rounds of a
    group, on shapes with ragged panels and ragged token tiles, with every epilogue."""
    rng = np.random.default_rng(workloads.seed_for("random prefill", case))
    _, K, N, group = _draw(rng)
    M = int(rng.integers(41, 701))
    epi = ["none", "add", "bias", "swiglu"][case % 4]
    w_np = workloads.weights(K, N, workloads.seed_for("random prefill w", case))
    x_np = workloads.activations(M, K, workloads.seed_for("random prefill x", case), outlier_fraction=0.01)
    packed, scales = lib.tl_e0m4_quantize(torch.from_numpy(w_np).to(dev), group=group)
    x = torch.from_numpy(x_np).to(dev)
    w_hat = _w_hat(w_np, group)
    if epi == "none":
        y = lib.tl_e0m4_matmul(x, packed, scales, N, group=group)
        ref = oracle.matmul(x_np, w_hat)
    elif epi == "add":
        a_np = workloads.activations(M, N, workloads.seed_for("random prefill a", case))
        y = lib.tl_e0m4_matmul_add(x, packed, scales, N, torch.from_numpy(a_np).to(dev),
                                   y=torch.empty((M, N), dtype=torch.float16, device=dev), group=group)
        ref = oracle.matmul(x_np, w_hat, a_np)
    elif epi == "bias":
        b_np = workloads.activations(1, N, workloads.seed_for("random prefill b", case))[0].copy()
        y = lib.tl_e0m4_matmul_bias(x, packed, scales, N, torch.from_numpy(b_np).to(dev), group=group)
        ref = oracle.matmul(x_np, w_hat, b_np)
    else:
        y = lib.tl_e0m4_matmul_swiglu(x, packed, scales, N, group=group)
        ref = oracle.swiglu_blocks(oracle.matmul(x_np, w_hat))
    torch.cuda.synchronize()
    assert lib.tl_e0m4_device_status() == 0
    assert_close(_np(y), ref)


@pytest.mark.parametrize("case", range(24))
def test_other_code_widths_on_random_shapes(lib, dev, case):
    """E0M8, E0M3 and E0M5 (groups of 128): quantizer words bit for bit and the matmul within
    tolerance, 1..300 tokens, shapes drawn like the 4-bit cases."""
    rng = np.random.default_rng(workloads.seed_for("random widths", case))
    _, K, N, _ = _draw(rng)
    group = 128
    M = int(rng.choice([1, 2, 5, 8, 9, 16, int(rng.integers(17, 301))]))
    bits = [8, 3, 5][case % 3]
    w_np = workloads.weights(K, N, workloads.seed_for("random widths w", case))
    x_np = workloads.activations(M, K, workloads.seed_for("random widths x", case))
    w, x = torch.from_numpy(w_np).to(dev), torch.from_numpy(x_np).to(dev)
    codes, d_h, b_h = oracle.quantize(w_np, group=group, bits=bits)
    ref_p, ref_s = oracle.pack(codes, d_h, b_h, group=group, bits=bits)
    if bits == 8:
        packed, scales = lib.tl_e0m8_quantize(w, group=group)
        y = lib.tl_e0m8_matmul(x, packed, scales, N, group=group)
    else:
        packed, scales = lib.tl_e0mx_quantize(w, bits)
        y = lib.tl_e0mx_matmul(x, packed, scales, N, bits)
    torch.cuda.synchronize()
    assert lib.tl_e0m4_device_status() == 0
    assert np.array_equal(_np(packed).view(np.uint32), ref_p)
    assert np.array_equal(_np(scales).view(np.uint32), ref_s)
    assert_close(_np(y), oracle.matmul(x_np, oracle.dequantize(codes, d_h, b_h, group=group, bits=bits)))
