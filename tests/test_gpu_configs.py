"""GPU parity on the full-size layer shapes of every benchmark configuration.

Two kinds of checks, both through the C ABI against the CPU oracle:
  * packing and dequantization of WHOLE matrices, bit for bit (the oracle works through the matrix
    in column slabs; columns are independent);
  * the matmul in the launch configuration the benchmark times (single calls at every M of the
    sweeps, and whole stacks as one list call), compared on sampled output columns and token rows:
    an output column depends on its own weight column only, so the oracle recomputes the sample
    exactly.
Tolerance of the matmul: max|y - y_ref| <= 1e-2 max|y_ref| and relative Frobenius error <= 1e-3.
"""

import numpy as np
import pytest

import oracle
from paper_2403_20041_b200 import workloads

torch = pytest.importorskip("torch")
pytestmark = pytest.mark.gpu

MAX_ABS_FRAC = 1e-2
REL_FRO = 1e-3


@pytest.fixture(scope="module")
def dev():
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    return torch.device("cuda:0")


def _np(t):
    return t.detach().cpu().numpy()


def _shape(stack, name):
    return next((k, n) for nm, k, n in workloads.STACKS[stack]["matrices"] if nm == name)


def assert_matmul_close(y, y_ref):
    y = np.asarray(y, dtype=np.float64)
    assert np.isfinite(y).all()
    assert np.abs(y - y_ref).max() <= MAX_ABS_FRAC * np.abs(y_ref).max()
    assert np.linalg.norm(y - y_ref) / np.linalg.norm(y_ref) <= REL_FRO


# ------------------------------------------------------------------ whole matrices, bit for bit
FULL_TENSORS = [
    ("gemv4096", "w"),
    ("gemma2b", "q"), ("gemma2b", "k"), ("gemma2b", "gate"), ("gemma2b", "down"),
    ("chatglm2_6b", "qkv"), ("chatglm2_6b", "gate_up"), ("chatglm2_6b", "down"),
    ("llm14b", "qkv"), ("llm14b", "o"), ("llm14b", "gate_up"), ("llm14b", "down"),
]


@pytest.mark.parametrize("stack,name", FULL_TENSORS)
def test_full_tensor_packing_and_dequant_bit_exact(lib, dev, stack, name):
    """Every packed word, every scale word and every dequantized fp16 value of a whole layer matrix."""
    K, N = _shape(stack, name)
    w = workloads.weights_torch(K, N, workloads.seed_for("fulltensor", stack, name), dev)
    packed, scales = lib.tl_e0m4_quantize(w)
    w_hat = lib.tl_e0m4_dequant(packed, scales, K, N)
    torch.cuda.synchronize()
    pw, sw = _np(packed).view(np.uint32), _np(scales).view(np.uint32)
    ng = K // 128
    slab = 1024  # columns per oracle pass: a multiple of the 128-column panel, so a slab's tiles are contiguous
    for n0 in range(0, N, slab):
        n1 = min(N, n0 + slab)
        codes, d_h, b_h = oracle.quantize(_np(w[:, n0:n1]).copy())
        ref_p, ref_s = oracle.pack(codes, d_h, b_h)
        t0, t1 = (n0 // 16) * ng, (n1 // 16) * ng  # tiles before the slab / up to its end
        assert np.array_equal(pw[t0 * 256:t1 * 256], ref_p), (n0, "packed")
        assert np.array_equal(sw[t0 * 16:t1 * 16], ref_s), (n0, "scales")
        assert np.array_equal(_np(w_hat[:, n0:n1]).view(np.uint16),
                              oracle.dequantize(codes, d_h, b_h).view(np.uint16)), (n0, "dequant")


# ------------------------------------------------------------------ single calls at config sizes
def _sampled_case(lib, dev, stack, name, M, n_blocks=10):
    K, N = _shape(stack, name)
    seed = workloads.seed_for("cfg", stack, name, M)
    w = workloads.weights_torch(K, N, seed, dev)
    x = workloads.activations_torch(M, K, seed + 1, dev, outlier_fraction=0.01 if M > 16 else 0.0)
    packed, scales = lib.tl_e0m4_quantize(w)
    y = lib.tl_e0m4_matmul(x, packed, scales, N)
    torch.cuda.synchronize()
    rng = np.random.default_rng(seed)
    nbs = sorted(set([0, N // 16 - 1] + rng.integers(0, N // 16, size=n_blocks).tolist()))
    cols = np.concatenate([np.arange(nb * 16, nb * 16 + 16) for nb in nbs])
    # token rows: all of them up to 64; beyond that rows 0 and M - 1, one per 128-token tile and a random few
    rows = np.arange(M) if M <= 64 else np.unique(np.concatenate(
        [[0, M - 1], np.arange(0, M, 128) + rng.integers(0, 128, size=(M + 127) // 128), rng.integers(0, M, size=16)]))
    rows = rows[rows < M]
    codes, d_h, b_h = oracle.quantize(_np(w[:, torch.from_numpy(cols).to(dev)]))
    y_ref = oracle.matmul(_np(x)[rows], oracle.dequantize(codes, d_h, b_h))
    assert_matmul_close(_np(y)[np.ix_(rows, cols)], y_ref)
    assert lib.tl_e0m4_device_status() == 0


@pytest.mark.parametrize("M", [1, 2, 4, 8, 16, 64, 256, 1024, 4096])
@pytest.mark.parametrize("name", ["qkv", "o", "gate_up", "down"])
def test_llm14b_sweep_sampled(lib, dev, name, M):
    """The 14B-class layer at every M of its sweep: the register kernel (M <= 8), the tensor-core
    kernel with rounds of a group (16, 64), token tiles and pairs of CTAs (256 .. 4096)."""
    _sampled_case(lib, dev, "llm14b", name, M)


@pytest.mark.parametrize("M", [1, 4, 16, 128, 512, 2048])
@pytest.mark.parametrize("name", ["qkv", "o", "gate_up", "down"])
def test_chatglm2_sweep_sampled(lib, dev, name, M):
    _sampled_case(lib, dev, "chatglm2_6b", name, M)


@pytest.mark.parametrize("name", ["q", "k", "o", "gate", "down"])
def test_gemma2b_decode_sampled(lib, dev, name):
    _sampled_case(lib, dev, "gemma2b", name, 1)


# ------------------------------------------------------------------ whole stacks as one list call
@pytest.mark.parametrize("stack,layers,M", [("llm14b", 40, 1), ("llm14b", 3, 16), ("gemma2b", 18, 1), ("gemma2b", 30, 2),
                                            ("chatglm2_6b", 28, 4)])
def test_stack_as_one_list_sampled(lib, dev, stack, layers, M):
    """The benchmark's headline launch: every matrix of every layer as one tl_e0m4_matmul_batch call
    (one persistent kernel per 192 problems, each with its own weights and activations).  The oracle
    recomputes sampled column blocks of a sample of the problems, first and last included."""
    spec = workloads.STACKS[stack]
    shapes = [(layer, name, K, N) for layer in range(layers) for name, K, N in spec["matrices"]]
    probs, keep = [], {}
    rng = np.random.default_rng(workloads.seed_for("list", stack, M))
    checked = set([0, len(shapes) - 1] + rng.integers(0, len(shapes), size=10).tolist())
    # the neighbourhood of every 128th problem too
    checked |= {j for j in range(len(shapes)) if j % 128 in (0, 127)}
    for j, (layer, name, K, N) in enumerate(shapes):
        w = workloads.weights_torch(K, N, workloads.seed_for("list", stack, layer, name), dev)
        packed, scales = lib.tl_e0m4_quantize(w)
        x = workloads.activations_torch(M, K, workloads.seed_for("list", stack, layer, name, "x"), dev)
        y = torch.full((M, N), float("nan"), dtype=torch.float16, device=dev)
        probs.append((x, packed, scales, y))
        if j in checked:
            nbs = sorted(set([0, N // 16 - 1] + rng.integers(0, N // 16, size=6).tolist()))
            cols = np.concatenate([np.arange(nb * 16, nb * 16 + 16) for nb in nbs])
            keep[j] = (cols, _np(w[:, torch.from_numpy(cols).to(dev)]))
        del w
    ws = lib.tl_e0m4_workspace(lib.tl_e0m4_matmul_batch_workspace(), dev)
    lib.tl_e0m4_matmul_batch(probs, M, ws)
    torch.cuda.synchronize()
    assert not _np(ws).any()
    assert lib.tl_e0m4_device_status() == 0
    for j, (cols, w_np) in keep.items():
        x, _, _, y = probs[j]
        codes, d_h, b_h = oracle.quantize(w_np)
        y_ref = oracle.matmul(_np(x), oracle.dequantize(codes, d_h, b_h))
        assert_matmul_close(_np(y)[:, cols], y_ref)
    # every output was written (no NaN left anywhere)
    for _, _, _, y in probs[::7]:
        assert torch.isfinite(y).all()
