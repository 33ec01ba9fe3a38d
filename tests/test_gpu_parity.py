"""GPU parity: the CUDA library, called through its C ABI, against the CPU oracle.

Integer/byte results (packed codes, scale words, dequantized fp16 bits) must be bit-exact.
Matmul results must satisfy  max|y - y_ref| <= 1e-2 * max|y_ref|  and
||y - y_ref||_F / ||y_ref||_F <= 1e-3  with y_ref the oracle's double-precision product.
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


def _to_np(t):
    return t.detach().cpu().numpy()


def _words(t):
    return _to_np(t).view(np.uint32)


def assert_matmul_close(y, y_ref):
    y = np.asarray(y, dtype=np.float64)
    scale = np.abs(y_ref).max()
    assert np.isfinite(y).all()
    if scale == 0:
        assert not y.any()
        return
    assert np.abs(y - y_ref).max() <= MAX_ABS_FRAC * scale
    assert np.linalg.norm(y - y_ref) / np.linalg.norm(y_ref) <= REL_FRO


def _quantize_both(lib, dev, w_np):
    w = torch.from_numpy(w_np).to(dev)
    packed, scales = lib.tl_e0m4_quantize(w)
    torch.cuda.synchronize()
    codes, d_h, b_h = oracle.quantize(w_np)
    return packed, scales, (codes, d_h, b_h)


# ---------------------------------------------------------------- quantize / pack / dequant
@pytest.mark.parametrize("K,N", [(128, 16), (384, 48), (1408, 272), (256, 400), (2048, 256), (4096, 4096)])
@pytest.mark.parametrize("dtype", [np.float32, np.float16])
def test_quantize_and_dequant_bit_exact(lib, dev, K, N, dtype):
    if dtype == np.float16 and K * N > 1 << 20:
        pytest.skip("fp16 input covered on the small shapes")
    w_np = workloads.weights(K, N, seed=workloads.seed_for("q", K, N)).astype(dtype)
    packed, scales, (codes, d_h, b_h) = _quantize_both(lib, dev, w_np)
    ref_packed, ref_scales = oracle.pack(codes, d_h, b_h)
    assert np.array_equal(_words(packed), ref_packed)
    assert np.array_equal(_words(scales), ref_scales)
    w_hat = lib.tl_e0m4_dequant(packed, scales, K, N)
    torch.cuda.synchronize()
    ref = oracle.dequantize(codes, d_h, b_h)
    assert np.array_equal(_to_np(w_hat).view(np.uint16), ref.view(np.uint16))


def test_quantize_degenerate_groups(lib, dev):
    K, N = 512, 32
    w = workloads.weights(K, N, seed=1)
    w[:128, :] = 0.0                     # dead groups
    w[128:256, 3] = 0.0
    w[128 + 7, 3] = 0.37                 # single non-zero
    w[256:384, :] = np.abs(w[256:384])   # all positive
    w[384:, :] = -np.abs(w[384:])        # all negative
    w[300, 5] = 3.0e5                    # scale saturates
    w[130:140, 9] = np.float32(2.0 ** -30)  # vanishing group -> scale underflows to subnormal/zero
    w[128:256, 10] = 0.0
    w[131, 10] = np.float32(1.0e-9)
    packed, scales, (codes, d_h, b_h) = _quantize_both(lib, dev, w)
    ref_packed, ref_scales = oracle.pack(codes, d_h, b_h)
    assert np.array_equal(_words(packed), ref_packed)
    assert np.array_equal(_words(scales), ref_scales)
    w_hat = lib.tl_e0m4_dequant(packed, scales, K, N)
    assert np.array_equal(_to_np(w_hat).view(np.uint16),
                          oracle.dequantize(codes, d_h, b_h).view(np.uint16))


def test_quantize_exact_ties_and_zeros(lib, dev):
    # the hand-worked mixed group of the oracle pins, repeated over a tile
    K, N = 128, 16
    w = np.zeros((K, N), np.float32)
    vals = [-13.0 / 256.0, 815.0 / 4096.0, 0.0, 1 / 64, -1 / 64, 0.5 / 64, -0.5 / 64]
    w[: len(vals), :] = np.asarray(vals, np.float32)[:, None]
    packed, scales, (codes, d_h, b_h) = _quantize_both(lib, dev, w)
    assert codes[: len(vals), 0].tolist() == [0, 15, 3, 4, 2, 4, 3]
    assert np.array_equal(_words(packed), oracle.pack(codes, d_h, b_h)[0])
    w_hat = _to_np(lib.tl_e0m4_dequant(packed, scales, K, N))
    assert w_hat[: len(vals), 5].astype(np.float64).tolist() == [-3 / 64, 12 / 64, 0.0, 1 / 64, -1 / 64, 1 / 64, 0.0]


@pytest.mark.parametrize("K,N", [(4096, 27392), (13696, 4096), (16384, 2048)])
def test_quantize_full_size_sampled_blocks(lib, dev, K, N):
    """Config-sized matrices: all of the matrix is quantized on the GPU; the oracle recomputes
    sampled 16-column blocks (columns are independent) and their packed tiles must match."""
    w = workloads.weights_torch(K, N, workloads.seed_for("full", K, N), dev)
    packed, scales = lib.tl_e0m4_quantize(w)
    w_hat = lib.tl_e0m4_dequant(packed, scales, K, N)
    torch.cuda.synchronize()
    rng = np.random.default_rng(0)
    panels = sorted(set([0, N // 128 - 1] + rng.integers(0, N // 128, size=4).tolist()))
    ng = K // 128
    pw, sw = _words(packed), _words(scales)
    for p in panels:  # every config N is a multiple of 128: a panel is 8 tiles per group
        cols = slice(p * 128, p * 128 + 128)
        w_np = _to_np(w[:, cols]).copy()
        codes, d_h, b_h = oracle.quantize(w_np)
        ref_p, ref_s = oracle.pack(codes, d_h, b_h)
        assert np.array_equal(pw[p * 8 * ng * 256:(p + 1) * 8 * ng * 256], ref_p)
        assert np.array_equal(sw[p * 8 * ng * 16:(p + 1) * 8 * ng * 16], ref_s)
        assert np.array_equal(_to_np(w_hat[:, cols]).view(np.uint16),
                              oracle.dequantize(codes, d_h, b_h).view(np.uint16))


# ---------------------------------------------------------------- matmul
def _matmul_case(lib, dev, M, K, N, seed, outliers=0.0):
    w_np = workloads.weights(K, N, seed)
    x_np = workloads.activations(M, K, seed + 1, outlier_fraction=outliers)
    packed, scales, (codes, d_h, b_h) = _quantize_both(lib, dev, w_np)
    y = lib.tl_e0m4_matmul(torch.from_numpy(x_np).to(dev), packed, scales, N)
    torch.cuda.synchronize()
    y_ref = oracle.matmul(x_np, oracle.dequantize(codes, d_h, b_h))
    return _to_np(y), y_ref


@pytest.mark.parametrize("M", [1, 2, 3, 8, 9, 16])
@pytest.mark.parametrize("K,N", [(128, 16), (384, 48), (1408, 272), (4096, 512)])
def test_decode_matmul_matches_oracle(lib, dev, M, K, N):
    y, y_ref = _matmul_case(lib, dev, M, K, N, seed=workloads.seed_for("mm", M, K, N))
    assert y.shape == (M, N)
    assert_matmul_close(y, y_ref)


@pytest.mark.parametrize("M", [17, 40, 128, 200])
@pytest.mark.parametrize("K,N", [(384, 48), (1408, 272), (2048, 512)])
def test_prefill_matmul_matches_oracle(lib, dev, M, K, N):
    y, y_ref = _matmul_case(lib, dev, M, K, N, seed=workloads.seed_for("pf", M, K, N), outliers=0.01)
    assert y.shape == (M, N)
    assert_matmul_close(y, y_ref)


@pytest.mark.parametrize("M", [1, 16, 64])
def test_unit_vector_returns_dequantized_row_bit_exactly(lib, dev, M):
    K, N = 512, 64
    w_np = workloads.weights(K, N, seed=21)
    packed, scales, (codes, d_h, b_h) = _quantize_both(lib, dev, w_np)
    w_hat = oracle.dequantize(codes, d_h, b_h)
    ks = [0, 1, 127, 128, 300, 511]
    for k in ks:
        x = np.zeros((M, K), np.float16)
        x[M - 1, k] = 1.0
        y = _to_np(lib.tl_e0m4_matmul(torch.from_numpy(x).to(dev), packed, scales, N))
        assert np.array_equal(y[M - 1].view(np.uint16), w_hat[k].view(np.uint16))
        assert not y[: M - 1].view(np.uint16).any()


def test_matmul_with_zero_weights_and_zero_activations(lib, dev):
    K, N = 256, 32
    packed, scales, _ = _quantize_both(lib, dev, np.zeros((K, N), np.float32))
    x = torch.from_numpy(workloads.activations(4, K, 3)).to(dev)
    assert not _to_np(lib.tl_e0m4_matmul(x, packed, scales, N)).any()
    packed, scales, _ = _quantize_both(lib, dev, workloads.weights(K, N, 4))
    y = lib.tl_e0m4_matmul(torch.zeros((4, K), dtype=torch.float16, device=dev), packed, scales, N)
    assert not _to_np(y).any()


def test_matmul_overwrites_output(lib, dev):
    K, N = 256, 32
    w_np = workloads.weights(K, N, 5)
    x_np = workloads.activations(2, K, 6)
    packed, scales, (codes, d_h, b_h) = _quantize_both(lib, dev, w_np)
    y = torch.full((2, N), float("nan"), dtype=torch.float16, device=dev)
    lib.tl_e0m4_matmul(torch.from_numpy(x_np).to(dev), packed, scales, N, y=y)
    assert_matmul_close(_to_np(y), oracle.matmul(x_np, oracle.dequantize(codes, d_h, b_h)))


@pytest.mark.parametrize("stack,name,M", [
    ("gemv4096", "w", 1), ("gemma2b", "k", 1), ("gemma2b", "gate", 1), ("gemma2b", "down", 1),
    ("chatglm2_6b", "gate_up", 16), ("chatglm2_6b", "down", 4), ("llm14b", "qkv", 16),
    ("chatglm2_6b", "qkv", 128), ("chatglm2_6b", "down", 512), ("llm14b", "o", 2048),
])
def test_config_shapes_sampled_columns(lib, dev, stack, name, M):
    """Full-size layers in the benchmark's launch configuration; the oracle recomputes a
    sample of output column blocks (each output column depends on its own weights only)."""
    K, N = next((k, n) for nm, k, n in workloads.STACKS[stack]["matrices"] if nm == name)
    seed = workloads.seed_for(stack, name, M)
    w = workloads.weights_torch(K, N, seed, dev)
    x = workloads.activations_torch(M, K, seed + 1, dev, outlier_fraction=0.01 if M > 16 else 0.0)
    packed, scales = lib.tl_e0m4_quantize(w)
    y = lib.tl_e0m4_matmul(x, packed, scales, N)
    torch.cuda.synchronize()
    rng = np.random.default_rng(1)
    nbs = sorted(set([0, N // 16 - 1] + rng.integers(0, N // 16, size=14).tolist()))
    cols = np.concatenate([np.arange(nb * 16, nb * 16 + 16) for nb in nbs])
    rows = np.arange(M) if M <= 64 else np.unique(np.concatenate(
        [[0, M - 1], rng.integers(0, M, size=30), np.arange(0, M, 128)]))
    w_np = _to_np(w[:, torch.from_numpy(cols).to(dev)])
    codes, d_h, b_h = oracle.quantize(w_np)
    y_ref = oracle.matmul(_to_np(x)[rows], oracle.dequantize(codes, d_h, b_h))
    assert_matmul_close(_to_np(y)[np.ix_(rows, cols)], y_ref)


def test_host_buffer_variant_matches_device_variant(lib, dev):
    M, K, N = 4, 1408, 272
    w_np = workloads.weights(K, N, 31)
    packed, scales, _ = _quantize_both(lib, dev, w_np)
    x_host = torch.from_numpy(workloads.activations(M, K, 32)).pin_memory()
    y_host = torch.empty((M, N), dtype=torch.float16).pin_memory()
    staging = lib.tl_e0m4_workspace(lib.tl_e0m4_matmul_host_staging(M, K, N), dev)
    lib.tl_e0m4_matmul_host(x_host, packed, scales, N, y_host, staging)
    torch.cuda.synchronize()
    y_dev = lib.tl_e0m4_matmul(x_host.to(dev), packed, scales, N)
    # split-K partial sums meet in fp32 atomics, so two runs may differ in the last bit
    assert_matmul_close(y_host.numpy(), _to_np(y_dev).astype(np.float64))
    assert np.abs(y_host.numpy().astype(np.float64) - _to_np(y_dev).astype(np.float64)).max() <= \
        2.0 ** -9 * np.abs(_to_np(y_dev).astype(np.float64)).max()


def test_workspace_is_returned_zeroed_and_status_clean(lib, dev):
    # a shape that splits column blocks across CTAs, so partial sums go through the scratch
    M, K, N = 3, 2048, 2048
    w = workloads.weights_torch(K, N, 77, dev)
    packed, scales = lib.tl_e0m4_quantize(w)
    x = workloads.activations_torch(M, K, 78, dev)
    ws = lib.tl_e0m4_workspace(lib.tl_e0m4_matmul_workspace(M, K, N), dev)
    y1 = lib.tl_e0m4_matmul(x, packed, scales, N, workspace=ws).clone()
    torch.cuda.synchronize()
    assert not _to_np(ws).any()
    y2 = lib.tl_e0m4_matmul(x, packed, scales, N, workspace=ws)
    torch.cuda.synchronize()
    assert not _to_np(ws).any()
    assert_matmul_close(_to_np(y2), _to_np(y1).astype(np.float64))
    assert lib.tl_e0m4_device_status() == 0


def _split_case(lib, dev, M, K, N, seed):
    w = workloads.weights_torch(K, N, seed, dev)
    packed, scales = lib.tl_e0m4_quantize(w)
    x = workloads.activations_torch(M, K, seed + 1, dev, outlier_fraction=0.01)
    ws = lib.tl_e0m4_workspace(lib.tl_e0m4_matmul_workspace(M, K, N), dev)
    codes, d_h, b_h = oracle.quantize(_to_np(w))
    y_ref = oracle.matmul(_to_np(x), oracle.dequantize(codes, d_h, b_h))
    for _ in range(2):
        y = lib.tl_e0m4_matmul(x, packed, scales, N, workspace=ws)
        torch.cuda.synchronize()
        assert not _to_np(ws).any()
        assert_matmul_close(_to_np(y), y_ref)
    assert lib.tl_e0m4_device_status() == 0


@pytest.mark.parametrize("M,K,N", [(16, 4096, 512), (40, 16384, 256), (256, 8192, 1024)])
def test_tensor_core_split_k_leaves_workspace_zero(lib, dev, M, K, N):
    # few output tiles and a long K: the library's own policy shares each tile between several
    # CTAs along K; partial sums meet in the scratch, which must be zero again afterwards
    _split_case(lib, dev, M, K, N, seed=91)


@pytest.mark.parametrize("ks", [2, 3, 4])
@pytest.mark.parametrize("M,K,N", [(9, 2048, 272), (200, 2048, 512), (300, 2176, 144), (520, 2560, 400)])
def test_tensor_core_split_k_forced(lib, dev, tuning, ks, M, K, N):
    # the tuning override forces the number of k slices (read at every call), so that ragged
    # panels, several token tiles and uneven group slices all go through the shared-tile path
    tuning("ksplit", ks)
    _split_case(lib, dev, M, K, N, seed=workloads.seed_for("ks", ks, M, K, N))


@pytest.mark.parametrize("M", [255, 256, 257, 300, 513, 1030])
def test_tensor_core_token_tile_boundaries(lib, dev, tuning, M):
    # M around the 256-token tile: equal tiles of a multiple of 16 tokens with a ragged last
    # one, 17 column blocks (two full panels and one of a single block), an odd number of groups
    tuning("ksplit", 1)
    y, y_ref = _matmul_case(lib, dev, M, 640 + 128, 272, seed=workloads.seed_for("tb", M), outliers=0.01)
    assert y.shape == (M, 272)
    assert_matmul_close(y, y_ref)


def test_back_to_back_calls_share_one_workspace(lib, dev):
    # consecutive decode launches overlap through programmatic dependent launch; results must
    # not depend on it
    K = 2048
    shapes = [2048, 256, 256, 2048, 4096]
    x = workloads.activations_torch(1, K, 5, dev)
    mats = []
    for i, N in enumerate(shapes):
        w = workloads.weights_torch(K, N, 100 + i, dev)
        mats.append((N, *lib.tl_e0m4_quantize(w), w))
    ws = lib.tl_e0m4_workspace(max(lib.tl_e0m4_matmul_workspace(1, K, N) for N in shapes), dev)
    torch.cuda.synchronize()
    ys = [lib.tl_e0m4_matmul(x, p, s, N, workspace=ws) for N, p, s, _ in mats]
    torch.cuda.synchronize()
    for (N, p, s, w), y in zip(mats, ys):
        cols = np.arange(0, N, 7)
        codes, d_h, b_h = oracle.quantize(_to_np(w)[:, cols])
        y_ref = oracle.matmul(_to_np(x), oracle.dequantize(codes, d_h, b_h))
        assert_matmul_close(_to_np(y)[:, cols], y_ref)


@pytest.mark.parametrize("M", [24, 300])
def test_tensor_core_chain_of_dependent_calls(lib, dev, M):
    # consecutive tensor-core launches overlap through programmatic dependent launch; a launch
    # whose input is the previous launch's output, and launches that share one split-K scratch,
    # must give what the same calls give with a synchronize between them
    dims = [1024, 2048, 512, 1024]          # x[M,1024] -> [M,2048] -> [M,512] -> [M,1024]
    mats = []
    for i in range(3):
        w = workloads.weights_torch(dims[i], dims[i + 1], 700 + i, dev) * (2.0 / dims[i] ** 0.5)
        mats.append(lib.tl_e0m4_quantize(w))
    ws = lib.tl_e0m4_workspace(max(lib.tl_e0m4_matmul_workspace(M, dims[i], dims[i + 1]) for i in range(3)), dev)
    x = workloads.activations_torch(M, dims[0], 710, dev)

    def run(sync):
        h = x
        for i, (p, s) in enumerate(mats):
            h = lib.tl_e0m4_matmul(h, p, s, dims[i + 1], workspace=ws)
            if sync:
                torch.cuda.synchronize()
        torch.cuda.synchronize()
        return _to_np(h).astype(np.float64)

    ref = run(sync=True)
    assert np.isfinite(ref).all() and np.abs(ref).max() > 0
    for _ in range(3):
        got = run(sync=False)
        # split-K sums meet in atomics: allow the last fp16 bit of each of the three layers
        assert np.abs(got - ref).max() <= 2.0 ** -7 * np.abs(ref).max()
    assert not _to_np(ws).any()
    assert lib.tl_e0m4_device_status() == 0


@pytest.mark.parametrize("M", [1, 5, 16, 17, 40, 100, 128])
def test_batch_matches_oracle_and_single_calls(lib, dev, M):
    # shapes chosen so that range boundaries cut panels, ragged panels and odd group counts occur
    shapes = [(1408, 272), (256, 400), (2048, 2048), (2048, 256), (13696, 512), (384, 48), (4096, 4096)]
    ws = lib.tl_e0m4_workspace(lib.tl_e0m4_matmul_batch_workspace(), dev)
    probs, refs = [], []
    for i, (K, N) in enumerate(shapes):
        w = workloads.weights_torch(K, N, 500 + i, dev)
        packed, scales = lib.tl_e0m4_quantize(w)
        x = workloads.activations_torch(M, K, 600 + i, dev)
        y = torch.full((M, N), float("nan"), dtype=torch.float16, device=dev)
        probs.append((x, packed, scales, y))
        cols = np.unique(np.concatenate([np.arange(0, N, 5), np.arange(N - 16, N)]))
        codes, d_h, b_h = oracle.quantize(_to_np(w)[:, cols])
        refs.append((cols, oracle.matmul(_to_np(x), oracle.dequantize(codes, d_h, b_h))))
    lib.tl_e0m4_matmul_batch(probs, M, ws)
    torch.cuda.synchronize()
    assert not _to_np(ws).any()
    for (x, packed, scales, y), (cols, y_ref) in zip(probs, refs):
        assert_matmul_close(_to_np(y)[:, cols], y_ref)
        y_single = lib.tl_e0m4_matmul(x, packed, scales, y.shape[1], workspace=ws)
        assert_matmul_close(_to_np(y), _to_np(y_single).astype(np.float64))
    assert lib.tl_e0m4_device_status() == 0


def test_batch_host_variant(lib, dev):
    M, shapes = 2, [(384, 48), (1408, 272)]
    xs = torch.empty(sum(M * K for K, _ in shapes), dtype=torch.float16, device=dev)
    ys = torch.empty(sum(M * N for _, N in shapes), dtype=torch.float16, device=dev)
    hx = torch.from_numpy(workloads.activations(1, xs.numel(), 9)[0]).pin_memory()
    hy = torch.empty(ys.numel(), dtype=torch.float16).pin_memory()
    ws = lib.tl_e0m4_workspace(lib.tl_e0m4_matmul_batch_workspace(), dev)
    probs, refs, xo, yo = [], [], 0, 0
    for i, (K, N) in enumerate(shapes):
        w_np = workloads.weights(K, N, 40 + i)
        packed, scales, (codes, d_h, b_h) = _quantize_both(lib, dev, w_np)
        x = xs[xo:xo + M * K].view(M, K)
        y = ys[yo:yo + M * N].view(M, N)
        refs.append((yo, N, oracle.matmul(hx[xo:xo + M * K].view(M, K).numpy(),
                                          oracle.dequantize(codes, d_h, b_h))))
        probs.append((x, packed, scales, y))
        xo += M * K
        yo += M * N
    lib.tl_e0m4_matmul_batch_host(probs, M, hx, xs, hy, ys, ws)
    torch.cuda.synchronize()
    for yo, N, y_ref in refs:
        assert_matmul_close(hy[yo:yo + M * N].view(M, N).numpy(), y_ref)


def test_gpu_entry_points_launch_kernels(lib, dev):
    before = lib.tl_e0m4_launch_count()
    w = workloads.weights_torch(128, 16, 1, dev)
    p, s = lib.tl_e0m4_quantize(w)
    lib.tl_e0m4_dequant(p, s, 128, 16)
    lib.tl_e0m4_matmul(torch.ones((1, 128), dtype=torch.float16, device=dev), p, s, 16)
    assert lib.tl_e0m4_launch_count() >= before + 3


# ---------------------------------------------------------------- matmul with the residual add fused in
@pytest.mark.parametrize("M", [1, 3, 8, 9, 40, 257])
@pytest.mark.parametrize("K,N", [(1408, 272), (2048, 2048)])
def test_matmul_add_matches_oracle(lib, dev, M, K, N):
    # 2048 x 2048 at M <= 8 cuts panels between CTAs (sums through the scratch); 272 columns end
    # in a panel of one block; M = 257 gives two token tiles of 144
    w_np = workloads.weights(K, N, seed=workloads.seed_for("add", K, N))
    x_np = workloads.activations(M, K, seed=workloads.seed_for("add", "x", M, K))
    r_np = workloads.activations(M, N, seed=workloads.seed_for("add", "r", M, N))
    packed, scales, (codes, d_h, b_h) = _quantize_both(lib, dev, w_np)
    y_ref = oracle.matmul(x_np, oracle.dequantize(codes, d_h, b_h), addend_h=r_np)
    x, r = torch.from_numpy(x_np).to(dev), torch.from_numpy(r_np).to(dev)
    y = torch.full((M, N), float("nan"), dtype=torch.float16, device=dev)
    lib.tl_e0m4_matmul_add(x, packed, scales, N, r, y=y)
    torch.cuda.synchronize()
    assert_matmul_close(_to_np(y), y_ref)
    assert np.array_equal(_to_np(r), r_np)          # the addend is only read
    # in place: the residual stream is updated where it lives
    lib.tl_e0m4_matmul_add(x, packed, scales, N, r)
    torch.cuda.synchronize()
    assert_matmul_close(_to_np(r), y_ref)


@pytest.mark.parametrize("ks", [2, 4])
def test_matmul_add_with_split_k(lib, dev, tuning, ks):
    tuning("ksplit", ks)
    M, K, N = 200, 2048, 400
    w_np = workloads.weights(K, N, seed=61)
    x_np = workloads.activations(M, K, seed=62, outlier_fraction=0.01)
    r_np = workloads.activations(M, N, seed=63)
    packed, scales, (codes, d_h, b_h) = _quantize_both(lib, dev, w_np)
    ws = lib.tl_e0m4_workspace(lib.tl_e0m4_matmul_workspace(M, K, N), dev)
    r = torch.from_numpy(r_np).to(dev)
    lib.tl_e0m4_matmul_add(torch.from_numpy(x_np).to(dev), packed, scales, N, r, workspace=ws)
    torch.cuda.synchronize()
    assert not _to_np(ws).any()
    assert_matmul_close(_to_np(r), oracle.matmul(x_np, oracle.dequantize(codes, d_h, b_h), addend_h=r_np))


def test_matmul_add_is_rounded_once(lib, dev):
    # x = e_0: the fp32 accumulator holds the exact product (code - zero point) / 8 * d, which
    # has more bits than an fp16.  The addend must meet that value, not its fp16 rounding: the
    # result is one fp32 sum rounded once to fp16.
    K, N = 256, 32
    w_np = workloads.weights(K, N, seed=71)
    packed, scales, (codes, d_h, b_h) = _quantize_both(lib, dev, w_np)
    exact = ((oracle.e0m4_value(codes[0]).astype(np.float64) - b_h[0].astype(np.float64)) *
             d_h[0].astype(np.float64))
    assert np.any(exact.astype(np.float16).astype(np.float64) != exact)    # the case is not vacuous
    x_np = np.zeros((1, K), np.float16)
    x_np[0, 0] = 1.0
    r_np = (exact * 2.0 ** -9).astype(np.float16)[None, :]
    y = lib.tl_e0m4_matmul_add(torch.from_numpy(x_np).to(dev), packed, scales, N,
                               torch.from_numpy(r_np).to(dev), y=torch.empty((1, N), dtype=torch.float16, device=dev))
    torch.cuda.synchronize()
    once = (exact.astype(np.float32) + r_np[0].astype(np.float32)).astype(np.float16)
    twice = (exact.astype(np.float16).astype(np.float32) + r_np[0].astype(np.float32)).astype(np.float16)
    assert np.any(once.view(np.uint16) != twice.view(np.uint16))           # rounding twice would show
    assert np.array_equal(_to_np(y)[0].view(np.uint16), once.view(np.uint16))


# ---------------------------------------------------------------- matmul with SwiGLU fused in
def _swiglu_case(lib, dev, M, K, F, seed):
    wg = workloads.weights_torch(K, F, seed, dev)
    wu = workloads.weights_torch(K, F, seed + 1, dev)
    w = lib.interleave_gate_up(wg, wu)
    packed, scales = lib.tl_e0m4_quantize(w)
    x = workloads.activations_torch(M, K, seed + 2, dev, outlier_fraction=0.01 if M > 16 else 0.0)
    codes, d_h, b_h = oracle.quantize(_to_np(w))
    y_ref = oracle.swiglu_blocks(oracle.matmul(_to_np(x), oracle.dequantize(codes, d_h, b_h)))
    return x, packed, scales, y_ref


@pytest.mark.parametrize("M", [1, 3, 8, 9, 40, 257])
@pytest.mark.parametrize("K,F", [(1408, 136), (2048, 1024)])
def test_matmul_swiglu_matches_oracle(lib, dev, M, K, F):
    # F = 136: N = 272 ends in a panel of one column block; 2048 x 2048 at M <= 8 cuts panels
    # between CTAs; M = 257 gives two token tiles of 144
    x, packed, scales, y_ref = _swiglu_case(lib, dev, M, K, F, seed=workloads.seed_for("glu", M, K, F))
    y = lib.tl_e0m4_matmul_swiglu(x, packed, scales, 2 * F)
    torch.cuda.synchronize()
    assert y.shape == (M, F)
    assert_matmul_close(_to_np(y), y_ref)


@pytest.mark.parametrize("ks", [2, 4])
def test_matmul_swiglu_with_split_k(lib, dev, tuning, ks):
    tuning("ksplit", ks)
    M, K, F = 200, 2048, 200
    x, packed, scales, y_ref = _swiglu_case(lib, dev, M, K, F, seed=81)
    ws = lib.tl_e0m4_workspace(lib.tl_e0m4_matmul_workspace(M, K, 2 * F), dev)
    y = lib.tl_e0m4_matmul_swiglu(x, packed, scales, 2 * F, workspace=ws)
    torch.cuda.synchronize()
    assert not _to_np(ws).any()
    assert_matmul_close(_to_np(y), y_ref)


def test_matmul_swiglu_paired_ctas(lib, dev, tuning):
    tuning("tc_pair", 1)
    tuning("ksplit", 1)
    x, packed, scales, y_ref = _swiglu_case(lib, dev, 300, 1024, 200, seed=85)   # 400 columns: 4 panels, the last of one block
    y = lib.tl_e0m4_matmul_swiglu(x, packed, scales, 400)
    torch.cuda.synchronize()
    assert_matmul_close(_to_np(y), y_ref)


# ---------------------------------------------------------------- seeded sweep over shapes, modes and epilogues
def test_seeded_sweep_of_shapes_modes_and_epilogues(lib, dev, tuning):
    """Fifty seeded cases: M across both kernels and the tile boundaries, K of 1..24 groups, N of
    1..70 column blocks, split-K forced or not, paired CTAs forced or not, each of the three
    epilogues; every result against the oracle."""
    import random

    rnd = random.Random(7)
    for it in range(50):
        M = rnd.choice([1, 2, 5, 8, 9, 15, 16, 17, 31, 33, 64, 100, 127, 128, 129, 200, 255, 256, 257, 300, 513, 700])
        K, N = 128 * rnd.randint(1, 24), 16 * rnd.randint(1, 70)
        tuning("ksplit", -1)
        tuning("tc_pair", -1)
        mode = rnd.choice(["auto", "ks", "pair", "nopair"])
        if mode == "ks":
            tuning("ksplit", rnd.choice([1, 2, 3, 4, 6, 8]))
        elif mode == "pair":
            tuning("tc_pair", 1)
            tuning("ksplit", 1)
        elif mode == "nopair":
            tuning("tc_pair", 0)
        epi = rnd.choice(["plain", "plain", "add", "swiglu"])
        w_np = workloads.weights(K, N, seed=1000 + it)
        x_np = workloads.activations(M, K, seed=2000 + it, outlier_fraction=0.01)
        packed, scales, (codes, d_h, b_h) = _quantize_both(lib, dev, w_np)
        w_hat = oracle.dequantize(codes, d_h, b_h)
        x = torch.from_numpy(x_np).to(dev)
        if epi == "plain":
            y, ref = lib.tl_e0m4_matmul(x, packed, scales, N), oracle.matmul(x_np, w_hat)
        elif epi == "add":
            r_np = workloads.activations(M, N, seed=3000 + it)
            y = lib.tl_e0m4_matmul_add(x, packed, scales, N, torch.from_numpy(r_np).to(dev))
            ref = oracle.matmul(x_np, w_hat, addend_h=r_np)
        else:
            y, ref = lib.tl_e0m4_matmul_swiglu(x, packed, scales, N), oracle.swiglu_blocks(oracle.matmul(x_np, w_hat))
        torch.cuda.synchronize()
        try:
            assert_matmul_close(_to_np(y), ref)
        except AssertionError as e:
            raise AssertionError(f"case {it}: M={M} K={K} N={N} mode={mode} epilogue={epi}") from e
    assert lib.tl_e0m4_device_status() == 0


@pytest.mark.parametrize("M", [3, 33])
def test_batch_longer_than_one_launch(lib, dev, M):
    # more problems than one launch of either list kernel takes: every problem must still meet its
    # own activations (the tensor-core kernel carries one tensor map per problem)
    rng = np.random.default_rng(M)
    count = 150
    ws = lib.tl_e0m4_workspace(lib.tl_e0m4_matmul_batch_workspace(), dev)
    shapes = [(128 * int(rng.integers(1, 4)), 16 * int(rng.integers(1, 12))) for _ in range(count)]
    probs, refs = [], []
    for i, (K, N) in enumerate(shapes):
        w_np = workloads.weights(K, N, seed=3000 + i)
        x_np = workloads.activations(M, K, seed=4000 + i)
        packed, scales = lib.tl_e0m4_quantize(torch.from_numpy(w_np).to(dev))
        y = torch.full((M, N), float("nan"), dtype=torch.float16, device=dev)
        probs.append((torch.from_numpy(x_np).to(dev), packed, scales, y))
        codes, d_h, b_h = oracle.quantize(w_np)
        refs.append(oracle.matmul(x_np, oracle.dequantize(codes, d_h, b_h)))
    lib.tl_e0m4_matmul_batch(probs, M, ws)
    torch.cuda.synchronize()
    assert not _to_np(ws).any()
    for (x, packed, scales, y), y_ref in zip(probs, refs):
        assert_matmul_close(_to_np(y), y_ref)
    assert lib.tl_e0m4_device_status() == 0


@pytest.mark.parametrize("stack,layers,M", [("gemma2b", 18, 1), ("chatglm2_6b", 6, 16), ("chatglm2_6b", 6, 96)])
def test_whole_stack_as_one_list_sampled(lib, dev, stack, layers, M):
    """The benchmark's launch configuration: every matrix of every layer in one
    tl_e0m4_matmul_batch call (full-size weights; own activations per matrix).  The oracle
    recomputes two column blocks of every problem."""
    spec = workloads.STACKS[stack]
    rng = np.random.default_rng(7)
    ws = lib.tl_e0m4_workspace(lib.tl_e0m4_matmul_batch_workspace(), dev)
    probs, refs = [], []
    for layer in range(layers):
        for name, K, N in spec["matrices"]:
            seed = workloads.seed_for("list", stack, layer, name)
            w = workloads.weights_torch(K, N, seed, dev)
            packed, scales = lib.tl_e0m4_quantize(w)
            x = workloads.activations_torch(M, K, seed + 1, dev)
            y = torch.full((M, N), float("nan"), dtype=torch.float16, device=dev)
            nbs = sorted({int(rng.integers(0, N // 16)), N // 16 - 1})
            cols = np.concatenate([np.arange(nb * 16, nb * 16 + 16) for nb in nbs])
            w_cols = _to_np(w[:, torch.from_numpy(cols).to(dev)])
            del w
            probs.append((x, packed, scales, y))
            refs.append((cols, w_cols))
    lib.tl_e0m4_matmul_batch(probs, M, ws)
    torch.cuda.synchronize()
    assert not _to_np(ws).any()
    assert lib.tl_e0m4_device_status() == 0
    for (x, packed, scales, y), (cols, w_cols) in zip(probs, refs):
        y_np = _to_np(y)
        assert np.isfinite(y_np).all()
        codes, d_h, b_h = oracle.quantize(w_cols)
        assert_matmul_close(y_np[:, cols], oracle.matmul(_to_np(x), oracle.dequantize(codes, d_h, b_h)))


@pytest.mark.parametrize("M", [1, 3, 8, 9, 40, 257, 520])
@pytest.mark.parametrize("K,N", [(1408, 272), (2048, 2048)])
def test_matmul_bias_matches_oracle(lib, dev, M, K, N):
    # a bias row shared by all tokens: the oracle adds it as a broadcast addend
    w_np = workloads.weights(K, N, seed=workloads.seed_for("bias", M, K, N))
    x_np = workloads.activations(M, K, seed=21)
    b_np = workloads.activations(1, N, seed=22)[0]
    packed, scales, (codes, d_h, b_h) = _quantize_both(lib, dev, w_np)
    y = lib.tl_e0m4_matmul_bias(torch.from_numpy(x_np).to(dev), packed, scales, N, torch.from_numpy(b_np).to(dev))
    torch.cuda.synchronize()
    y_ref = oracle.matmul(x_np, oracle.dequantize(codes, d_h, b_h), addend_h=np.tile(b_np, (M, 1)))
    assert_matmul_close(_to_np(y), y_ref)
    assert lib.tl_e0m4_device_status() == 0


@pytest.mark.parametrize("ks", [2, 4])
def test_matmul_bias_with_split_k(lib, dev, tuning, ks):
    tuning("ksplit", ks)
    M, K, N = 200, 2048, 512
    w_np = workloads.weights(K, N, seed=31)
    x_np = workloads.activations(M, K, seed=32)
    b_np = workloads.activations(1, N, seed=33)[0]
    packed, scales, (codes, d_h, b_h) = _quantize_both(lib, dev, w_np)
    y = lib.tl_e0m4_matmul_bias(torch.from_numpy(x_np).to(dev), packed, scales, N, torch.from_numpy(b_np).to(dev))
    torch.cuda.synchronize()
    assert_matmul_close(_to_np(y), oracle.matmul(x_np, oracle.dequantize(codes, d_h, b_h), addend_h=np.tile(b_np, (M, 1))))


@pytest.mark.parametrize("pair", ["0", "1"])
@pytest.mark.parametrize("M", [9, 33, 70, 97, 128])
def test_list_kernel_with_and_without_paired_ctas(lib, dev, tuning, pair, M):
    # both forms of the tensor-core list kernel at every token count, odd panel counts included
    tuning("list_pair", int(pair))
    shapes = [(1408, 272), (256, 400), (2048, 256), (384, 48), (2048, 2048), (640, 128), (13696, 144)]
    ws = lib.tl_e0m4_workspace(lib.tl_e0m4_matmul_batch_workspace(), dev)
    probs, refs = [], []
    for i, (K, N) in enumerate(shapes):
        w_np = workloads.weights(K, N, seed=5000 + i)
        x_np = workloads.activations(M, K, seed=5100 + i)
        packed, scales = lib.tl_e0m4_quantize(torch.from_numpy(w_np).to(dev))
        y = torch.full((M, N), float("nan"), dtype=torch.float16, device=dev)
        probs.append((torch.from_numpy(x_np).to(dev), packed, scales, y))
        cols = np.unique(np.concatenate([np.arange(0, N, 3), np.arange(N - 16, N)]))
        codes, d_h, b_h = oracle.quantize(w_np[:, cols])
        refs.append((cols, oracle.matmul(x_np, oracle.dequantize(codes, d_h, b_h))))
    for _ in range(2):
        lib.tl_e0m4_matmul_batch(probs, M, ws)
    torch.cuda.synchronize()
    assert not _to_np(ws).any()
    for (x, packed, scales, y), (cols, y_ref) in zip(probs, refs):
        y_np = _to_np(y)
        assert np.isfinite(y_np).all()
        assert_matmul_close(y_np[:, cols], y_ref)
    assert lib.tl_e0m4_device_status() == 0


# ---------------------------------------------------------------- panels shared by a cluster of CTAs
@pytest.mark.parametrize("cluster", [0, 1])
@pytest.mark.parametrize("group", [128, 32])
@pytest.mark.parametrize("M", [1, 5, 8])
def test_shared_panels_meet_in_scratch_or_in_a_cluster(lib, dev, tuning, M, group, cluster):
    """The CTAs that share a panel's k groups add their partial sums up either in the global scratch
    (cluster = 0) or, launched as a thread-block cluster, in one another's shared memory (1: forced
    wherever the shape allows it).  2128 columns: sixteen full panels and one of five column blocks,
    so some CTAs of the last cluster have no tile to finish.  Plain, residual and SwiGLU epilogues."""
    tuning("decode_cluster", cluster)
    K, N = 2048, 2128
    w_np = workloads.weights(K, N, seed=workloads.seed_for("cluster", group))
    x_np = workloads.activations(M, K, seed=workloads.seed_for("cluster", "x", M))
    r_np = workloads.activations(M, N, seed=workloads.seed_for("cluster", "r", M))
    codes, d_h, b_h = oracle.quantize(w_np, group=group)
    w_hat = oracle.dequantize(codes, d_h, b_h, group=group)
    packed, scales = lib.tl_e0m4_quantize(torch.from_numpy(w_np).to(dev), group=group)
    x, r = torch.from_numpy(x_np).to(dev), torch.from_numpy(r_np).to(dev)
    ws = lib.tl_e0m4_workspace(lib.tl_e0m4_matmul_workspace(M, K, N), dev)
    for _ in range(2):
        y = lib.tl_e0m4_matmul(x, packed, scales, N, workspace=ws, group=group)
        y_add = lib.tl_e0m4_matmul_add(x, packed, scales, N, r, y=torch.empty_like(r), workspace=ws, group=group)
        y_glu = lib.tl_e0m4_matmul_swiglu(x, packed, scales, N, workspace=ws, group=group)
        torch.cuda.synchronize()
        assert not _to_np(ws).any()
        y_ref = oracle.matmul(x_np, w_hat)
        assert_matmul_close(_to_np(y), y_ref)
        assert_matmul_close(_to_np(y_add), oracle.matmul(x_np, w_hat, addend_h=r_np))
        assert_matmul_close(_to_np(y_glu), oracle.swiglu_blocks(y_ref))
    assert lib.tl_e0m4_device_status() == 0
