"""The entry point for callers that may not allocate device memory (runs last on purpose).

Some users of this library cannot call cudaMalloc when they need a matmul: an inference server
that gave its whole device pool to a framework allocator at start-up, a latency-critical loop
that must not trigger cudaMalloc's device synchronization, a plug-in whose host forbids
allocation.  For them `tl_e0m4_matmul_noalloc` keeps the decode kernel's scratch in an array
inside the library.  The first test calls it through the C ABI, twice in a row on the same stream,
and checks each result against `tl_e0m4_matmul` (which takes its scratch from the caller) within
the tolerance the parity tests use; the shape is one whose column panels are split between
CTAs, so the scratch is really exercised, and the second call finds the array as the first
left it.  The second test covers the entry point's whole range of token counts (1 to 16: above
8 tokens it is the only default route into the register kernel's two-block form), every group
size and a last panel of fewer than eight column blocks, against the CPU oracle.
"""

import numpy as np
import pytest

import oracle
from paper_2403_20041_b200 import workloads

torch = pytest.importorskip("torch")
pytestmark = pytest.mark.gpu

MAX_ABS_FRAC = 1e-2
REL_FRO = 1e-3


def _close(y, y_ref):
    y = y.astype(np.float64)
    y_ref = y_ref.astype(np.float64)
    assert np.isfinite(y).all()
    assert np.abs(y - y_ref).max() <= MAX_ABS_FRAC * np.abs(y_ref).max()
    assert np.linalg.norm(y - y_ref) / np.linalg.norm(y_ref) <= REL_FRO


def test_noalloc_entry_point_matches_workspace_entry_point(lib):
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    dev = torch.device("cuda:0")
    M, K, N = 3, 2048, 2048  # 16 panels over 256+ CTAs: every panel is split and meets in the scratch
    w = workloads.weights_torch(K, N, 901, dev)
    packed, scales = lib.tl_e0m4_quantize(w)
    x1 = workloads.activations_torch(M, K, 902, dev)
    x2 = workloads.activations_torch(M, K, 903, dev)
    # everything the calls need exists before them; the calls themselves allocate nothing
    y1 = torch.full((M, N), float("nan"), dtype=torch.float16, device=dev)
    y2 = torch.full((M, N), float("nan"), dtype=torch.float16, device=dev)
    assert lib.tl_e0m4_matmul_noalloc_scratch_bytes() <= 4 << 20
    torch.cuda.synchronize()

    lib.tl_e0m4_matmul_noalloc(x1, packed, scales, y1)
    lib.tl_e0m4_matmul_noalloc(x2, packed, scales, y2)  # second call in a row, same stream
    torch.cuda.synchronize()

    ref1 = lib.tl_e0m4_matmul(x1, packed, scales, N)
    ref2 = lib.tl_e0m4_matmul(x2, packed, scales, N)
    torch.cuda.synchronize()
    _close(y1.cpu().numpy(), ref1.cpu().numpy())
    _close(y2.cpu().numpy(), ref2.cpu().numpy())
    assert lib.tl_e0m4_device_status() == 0


@pytest.mark.parametrize("group", [128, 64, 32])
@pytest.mark.parametrize("M", [1, 8, 9, 12, 16])
def test_noalloc_entry_point_matches_oracle_over_its_whole_range(lib, M, group):
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    dev = torch.device("cuda:0")
    # 2128 = 16 full panels + one of five column blocks; 17 panels over ~300 CTAs: every panel is cut
    # between CTAs and meets in the built-in scratch
    K, N = 2048, 2128
    w_np = workloads.weights(K, N, workloads.seed_for("noalloc", group))
    codes, d_h, b_h = oracle.quantize(w_np, group=group)
    w_hat = oracle.dequantize(codes, d_h, b_h, group=group)
    packed, scales = lib.tl_e0m4_quantize(torch.from_numpy(w_np).to(dev), group=group)
    xs = [workloads.activations(M, K, workloads.seed_for("noalloc", "x", M, i)) for i in range(2)]
    xd = [torch.from_numpy(x).to(dev) for x in xs]
    ys = [torch.full((M, N), float("nan"), dtype=torch.float16, device=dev) for _ in range(2)]
    torch.cuda.synchronize()
    for x, y in zip(xd, ys):  # two calls in a row on one stream
        lib.tl_e0m4_matmul_noalloc(x, packed, scales, y, group=group)
    torch.cuda.synchronize()
    for x, y in zip(xs, ys):
        _close(y.cpu().numpy(), oracle.matmul(x, w_hat))
    assert lib.tl_e0m4_device_status() == 0


def test_noalloc_entry_point_refuses_what_its_scratch_cannot_serve(lib):
    L = lib.lib()
    a = 0x10000  # fake aligned pointers: the checks below fail before anything is touched
    assert L.tl_e0m4_matmul_noalloc(a, a, a, a, 17, 128, 16, 128, None) == 9   # TL_ERR_LIMIT
    assert "M <= 16" in lib.tl_status_string(9)
    assert L.tl_e0m4_matmul_noalloc(a, a, a, None, 1, 128, 16, 128, None) == 1  # TL_ERR_NULL
    assert L.tl_e0m4_matmul_noalloc(a, a, a, a, 1, 100, 16, 128, None) == 2     # TL_ERR_SHAPE
