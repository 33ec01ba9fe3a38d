"""A bounded device-side wait that runs out, made to happen in the safe form.

Every mbarrier wait of the matmul kernels gives up after a cycle budget, raises TL_ERR_TIMEOUT in the
device status word and lets its CTA leave in order (tensor memory freed).  To see that path work
without faulting or hanging anything, the tests shorten the budget to a fraction of a millisecond
and tell the kernels' producers to issue no copies at all (tl_e0m4_tuning_set "wait_limit_cycles"
and "skip_copies"): every consumer then waits for data that is never requested, nothing is in
flight when it gives up, and the kernel returns by itself.  Afterwards the same workspace, cleared
again, must serve a normal call, and a following tensor-core launch shows that tensor memory was
handed back.
"""

import numpy as np
import pytest

import oracle
from paper_2403_20041_b200 import workloads

torch = pytest.importorskip("torch")
pytestmark = pytest.mark.gpu

TL_ERR_TIMEOUT = 8
SHORT = 200_000  # SM cycles: about 0.1 ms


@pytest.fixture(scope="module")
def dev():
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    return torch.device("cuda:0")


def _case(lib, dev, M, K, N, seed):
    w_np = workloads.weights(K, N, seed)
    x_np = workloads.activations(M, K, seed + 1)
    packed, scales = lib.tl_e0m4_quantize(torch.from_numpy(w_np).to(dev))
    codes, d_h, b_h = oracle.quantize(w_np)
    y_ref = oracle.matmul(x_np, oracle.dequantize(codes, d_h, b_h))
    return torch.from_numpy(x_np).to(dev), packed, scales, y_ref


def _check(y, y_ref):
    y = y.cpu().numpy().astype(np.float64)
    assert np.isfinite(y).all()
    assert np.abs(y - y_ref).max() <= 1e-2 * np.abs(y_ref).max()
    assert np.linalg.norm(y - y_ref) / np.linalg.norm(y_ref) <= 1e-3


@pytest.mark.parametrize("M,K,N,pair", [
    (1, 128, 16, False),     # register kernel, a single CTA
    (32, 256, 128, False),   # tensor-core kernel, one small token tile
    (200, 256, 128, False),  # tensor-core kernel, more tokens than one round of a whole group serves
    (64, 256, 256, True),    # a pair of CTAs on one work item (cluster of two)
])
def test_wait_runs_out_status_is_raised_and_the_next_call_is_correct(lib, dev, tuning, M, K, N, pair):
    x, packed, scales, y_ref = _case(lib, dev, M, K, N, seed=workloads.seed_for("timeout", M, K, N))
    if pair:
        tuning("tc_pair", 1)
        tuning("ksplit", 1)
    ws = lib.tl_e0m4_workspace(max(lib.tl_e0m4_matmul_workspace(M, K, N), 256), dev)
    y = torch.zeros((M, N), dtype=torch.float16, device=dev)
    assert lib.tl_e0m4_device_status() == 0
    tuning("wait_limit_cycles", SHORT)
    tuning("skip_copies", 1)
    lib.tl_e0m4_matmul(x, packed, scales, N, y=y, workspace=ws)   # returns: the launch itself is fine
    assert lib.tl_e0m4_device_status() == TL_ERR_TIMEOUT           # synchronizes; the kernel gave up by itself
    assert lib.tl_e0m4_device_status() == 0                        # reading the word cleared it
    tuning("skip_copies", -1)
    tuning("wait_limit_cycles", -1)
    # the same workspace, cleared again, serves a normal call (and, for the tensor-core shapes, the
    # launch finds its tensor memory free)
    lib.lib().tl_e0m4_workspace_init(ws.data_ptr(), ws.numel(), None)
    y = lib.tl_e0m4_matmul(x, packed, scales, N, workspace=ws)
    torch.cuda.synchronize()
    _check(y, y_ref)
    assert lib.tl_e0m4_device_status() == 0


@pytest.mark.parametrize("M", [4, 24, 100])
def test_wait_runs_out_in_the_list_kernels(lib, dev, tuning, M):
    # M = 4: register list kernel; 24: tensor-core list kernel; 100: its paired form
    shapes = [(256, 128), (384, 48)]
    cases = [_case(lib, dev, M, K, N, seed=workloads.seed_for("timeout-list", M, K, N)) for K, N in shapes]
    ys = [torch.zeros((M, N), dtype=torch.float16, device=dev) for _, N in shapes]
    probs = [(x, p, s, y) for (x, p, s, _), y in zip(cases, ys)]
    ws = lib.tl_e0m4_workspace(lib.tl_e0m4_matmul_batch_workspace(), dev)
    tuning("wait_limit_cycles", SHORT)
    tuning("skip_copies", 1)
    lib.tl_e0m4_matmul_batch(probs, M, ws)
    assert lib.tl_e0m4_device_status() == TL_ERR_TIMEOUT
    tuning("skip_copies", -1)
    tuning("wait_limit_cycles", -1)
    lib.lib().tl_e0m4_workspace_init(ws.data_ptr(), ws.numel(), None)
    lib.tl_e0m4_matmul_batch(probs, M, ws)
    torch.cuda.synchronize()
    for (_, _, _, y_ref), y in zip(cases, ys):
        _check(y, y_ref)
    assert lib.tl_e0m4_device_status() == 0


def test_wait_runs_out_in_the_chain_kernel(lib, dev, tuning):
    # two dependent steps; with the producers silent every consumer gives up on its first stage, the
    # kernel returns, and the re-initialised workspace (scratch slots and phase counters) serves a normal call
    M, K, N = 2, 256, 256
    x, p1, s1, ref1 = _case(lib, dev, M, K, N, seed=71)
    w2 = workloads.weights(N, 128, 72)
    p2, s2 = lib.tl_e0m4_quantize(torch.from_numpy(w2).to(dev))
    t = torch.zeros((M, N), dtype=torch.float16, device=dev)
    y = torch.zeros((M, 128), dtype=torch.float16, device=dev)
    steps = [dict(x=x, packed=p1, scales=s1, y=t), dict(x=t, packed=p2, scales=s2, y=y, after_previous=True)]
    ws = lib.tl_e0m4_workspace(lib.tl_e0m4_matmul_chain_workspace(), dev)
    tuning("wait_limit_cycles", SHORT)
    tuning("skip_copies", 1)
    lib.tl_e0m4_matmul_chain(steps, M, ws)
    assert lib.tl_e0m4_device_status() == TL_ERR_TIMEOUT
    tuning("skip_copies", -1)
    tuning("wait_limit_cycles", -1)
    lib.lib().tl_e0m4_workspace_init(ws.data_ptr(), ws.numel(), None)
    lib.tl_e0m4_matmul_chain(steps, M, ws)
    torch.cuda.synchronize()
    _check(t, ref1)
    codes, d_h, b_h = oracle.quantize(w2)
    _check(y, oracle.matmul(t.cpu().numpy(), oracle.dequantize(codes, d_h, b_h)))
    assert lib.tl_e0m4_device_status() == 0
    assert not ws.cpu().numpy().any()
