"""GPU parity of tl_e0m4_matmul_chain (a list of decode steps that consume one another's outputs,
run by one persistent kernel) against the oracle's chain step.

Every step is checked on its own: the oracle recomputes the step from the fp16 inputs the GPU
really fed it (the outputs of the earlier steps, read back), so a step's error is not mixed with
the rounding of the steps before it.  Tolerance per step: max|y - y_ref| <= 1e-2 max|y_ref| and
relative Frobenius error <= 1e-3, as for every matmul of the library.
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


class Mat:
    """A quantized weight on the GPU plus what the oracle needs to recompute sampled output columns."""

    def __init__(self, lib, dev, K, N, seed, n_blocks=None, std=0.02):
        w = workloads.weights_torch(K, N, seed, dev, std=std)
        self.K, self.N = K, N
        self.packed, self.scales = lib.tl_e0m4_quantize(w)
        rng = np.random.default_rng(seed)
        nbs = np.arange(N // 16) if n_blocks is None or N // 16 <= n_blocks else np.unique(
            np.concatenate([[0, N // 16 - 1], rng.integers(0, N // 16, size=n_blocks)]))
        self.blocks = nbs
        self.cols = np.concatenate([np.arange(nb * 16, nb * 16 + 16) for nb in nbs])
        codes, d_h, b_h = oracle.quantize(_np(w[:, torch.from_numpy(self.cols).to(dev)]))
        self.w_hat = oracle.dequantize(codes, d_h, b_h)  # fp16 [K, len(cols)]

    def out_cols(self, swiglu):
        """Output columns that the sampled weight columns determine."""
        if not swiglu:
            return self.cols
        return np.concatenate([np.arange(nb * 8, nb * 8 + 8) for nb in self.blocks])


def check_steps(lib, steps, mats):
    """steps: the dicts given to the library (tensors hold the GPU's results); mats: the Mat of each."""
    for st, mat in zip(steps, mats):
        epi = st.get("epilogue", "none")
        addend = None
        if epi == "add":
            # the addend the GPU saw: the step's own addend buffer, unless it was overwritten in place
            addend = _np(st["addend_before"] if "addend_before" in st else st["addend"])[:, mat.cols]
        elif epi == "bias":
            addend = _np(st["addend"])[mat.cols]
        ref = oracle.chain_step(_np(st["x"]), mat.w_hat, epi, addend, st.get("rms_eps"))
        assert_close(_np(st["y"])[:, mat.out_cols(epi == "swiglu")], ref)


def _layer_steps(lib, dev, M, H, QKV, F, layers, seed, n_blocks, split_qkv):
    """Transformer-shaped decode layers: rms-norm folded into qkv (+ bias), o + residual, rms-norm
    folded into gate_up (+ SwiGLU), down + residual.  Attention is left out: the first H features of
    the qkv output stand in for its result.  Every layer writes its own buffers, so every
    intermediate survives for the check."""
    steps, mats = [], []
    h = workloads.activations_torch(M, H, seed, dev)
    for layer in range(layers):
        def mat(name, K, N):
            return Mat(lib, dev, K, N, workloads.seed_for("chain", seed, layer, name), n_blocks)

        bias = workloads.activations_torch(1, QKV, seed + 7 * layer + 1, dev)[0].contiguous()
        new = lambda n: torch.full((M, n), float("nan"), dtype=torch.float16, device=dev)
        if split_qkv:
            # the projection as two independent steps of one phase: q (what "attention" passes on) and kv
            mq, mkv = mat("q", H, H), mat("kv", H, QKV - H)
            a, kv = new(H), new(QKV - H)
            steps.append(dict(x=h, packed=mq.packed, scales=mq.scales, y=a, epilogue="bias", addend=bias[:H].contiguous(),
                              rms_eps=1e-5, after_previous=True))
            steps.append(dict(x=h, packed=mkv.packed, scales=mkv.scales, y=kv, epilogue="bias",
                              addend=bias[H:].contiguous(), rms_eps=1e-5))
            mats += [mq, mkv]
        else:
            mqkv = mat("qkv", H, QKV)
            qkv = new(QKV)
            steps.append(dict(x=h, packed=mqkv.packed, scales=mqkv.scales, y=qkv, epilogue="bias", addend=bias,
                              rms_eps=1e-5, after_previous=True))
            mats.append(mqkv)
            a = qkv[:, :H]  # contiguous for one token only
        mo, mgu, md = mat("o", H, H), mat("gate_up", H, 2 * F), mat("down", F, H)
        h1, g, h2 = new(H), new(F), new(H)
        steps.append(dict(x=a, packed=mo.packed, scales=mo.scales, y=h1, epilogue="add", addend=h, after_previous=True))
        steps.append(dict(x=h1, packed=mgu.packed, scales=mgu.scales, y=g, epilogue="swiglu", rms_eps=1e-5,
                          after_previous=True))
        steps.append(dict(x=g, packed=md.packed, scales=md.scales, y=h2, epilogue="add", addend=h1, after_previous=True))
        mats += [mo, mgu, md]
        h = h2
    return steps, mats


@pytest.mark.parametrize("M", [1, 4, 8])
def test_small_layers_every_step_against_the_oracle(lib, dev, M):
    # small shapes with ragged last panels (528 = four panels and one column block; split: 384 and 144),
    # every output column checked; most phases have fewer chunks than the launch has CTAs
    steps, mats = _layer_steps(lib, dev, M, H=384, QKV=528, F=640, layers=3, seed=11 + M, n_blocks=None,
                               split_qkv=M > 1)
    ws = lib.tl_e0m4_workspace(lib.tl_e0m4_matmul_chain_workspace(), dev)
    lib.tl_e0m4_matmul_chain(steps, M, ws)
    torch.cuda.synchronize()
    assert lib.tl_e0m4_device_status() == 0
    assert not _np(ws).any()
    check_steps(lib, steps, mats)


@pytest.mark.parametrize("M", [1, 4])
def test_chatglm2_shaped_layers_sampled_columns(lib, dev, M):
    """Six ChatGLM2-6B-shaped layers (24 or 30 dependent steps, 650 MB of weights) through ONE call."""
    steps, mats = _layer_steps(lib, dev, M, H=4096, QKV=4608, F=13696, layers=6, seed=100 + M, n_blocks=8,
                               split_qkv=M > 1)
    ws = lib.tl_e0m4_workspace(lib.tl_e0m4_matmul_chain_workspace(), dev)
    before = lib.tl_e0m4_launch_count()
    lib.tl_e0m4_matmul_chain(steps, M, ws)
    assert lib.tl_e0m4_launch_count() == before + 1
    torch.cuda.synchronize()
    assert lib.tl_e0m4_device_status() == 0
    assert not _np(ws).any()
    check_steps(lib, steps, mats)
    # the same list again on the same workspace: same results up to the order of the atomics
    first = [_np(st["y"]).astype(np.float64) for st in steps]
    lib.tl_e0m4_matmul_chain(steps, M, ws)
    torch.cuda.synchronize()
    for st, y0 in zip(steps, first):
        assert np.abs(_np(st["y"]).astype(np.float64) - y0).max() <= 2.0 ** -8 * np.abs(y0).max()


def test_in_place_residual_stream_and_more_steps_than_one_launch_takes(lib, dev):
    # 70 layers x 2 steps = 140 steps (two launches), the residual stream h updated where it lives:
    # h = fp16(rms(h) (h . W1) . W2 + h); the oracle replays the chain with its own fp16 roundings
    M, H = 2, 256
    layers = 70
    h0 = workloads.activations(M, H, 5)
    h = torch.from_numpy(h0).to(dev)
    t = torch.empty((M, H), dtype=torch.float16, device=dev)
    steps, mats = [], []
    for layer in range(layers):
        m1 = Mat(lib, dev, H, H, workloads.seed_for("inplace", layer, 1), std=0.05)
        m2 = Mat(lib, dev, H, H, workloads.seed_for("inplace", layer, 2), std=0.01)
        steps.append(dict(x=h, packed=m1.packed, scales=m1.scales, y=t, rms_eps=1e-6, after_previous=True))
        steps.append(dict(x=t, packed=m2.packed, scales=m2.scales, y=h, epilogue="add", addend=h, after_previous=True))
        mats += [m1, m2]
    ws = lib.tl_e0m4_workspace(lib.tl_e0m4_matmul_chain_workspace(), dev)
    before = lib.tl_e0m4_launch_count()
    lib.tl_e0m4_matmul_chain(steps, M, ws)
    assert lib.tl_e0m4_launch_count() == before + 2
    torch.cuda.synchronize()
    assert lib.tl_e0m4_device_status() == 0
    assert not _np(ws).any()
    ref = h0
    for layer in range(layers):
        tt = oracle.chain_step(ref, mats[2 * layer].w_hat, rms_eps=1e-6).astype(np.float16)
        ref = oracle.chain_step(tt, mats[2 * layer + 1].w_hat, "add", ref).astype(np.float16)
    got = _np(h).astype(np.float64)
    ref = ref.astype(np.float64)
    # 140 dependent roundings: a looser bar than a single step's
    assert np.linalg.norm(got - ref) / np.linalg.norm(ref) <= 2e-2


@pytest.mark.parametrize("group", [64, 32])
def test_smaller_groups(lib, dev, group):
    M, K, N = 3, 512, 272
    w_np = workloads.weights(K, N, 77 + group)
    w2_np = workloads.weights(N - 16, 128, 78 + group)
    x_np = workloads.activations(M, K, 79)
    p1, s1 = lib.tl_e0m4_quantize(torch.from_numpy(w_np).to(dev), group=group)
    p2, s2 = lib.tl_e0m4_quantize(torch.from_numpy(w2_np).to(dev), group=group)
    x = torch.from_numpy(x_np).to(dev)
    y1 = torch.empty((M, N), dtype=torch.float16, device=dev)
    ws = lib.tl_e0m4_workspace(lib.tl_e0m4_matmul_chain_workspace(), dev)
    y2 = torch.empty((M, 128), dtype=torch.float16, device=dev)
    # the second step reads the first 256 columns' worth of K from a buffer of its own
    x2 = torch.empty((M, N - 16), dtype=torch.float16, device=dev)
    lib.tl_e0m4_matmul_chain([dict(x=x, packed=p1, scales=s1, y=y1, rms_eps=1e-5)], M, ws, group=group)
    x2.copy_(y1[:, :N - 16])
    lib.tl_e0m4_matmul_chain([dict(x=x2, packed=p2, scales=s2, y=y2)], M, ws, group=group)
    torch.cuda.synchronize()
    w_hat = oracle.dequantize(*oracle.quantize(w_np, group=group), group=group)
    assert_close(_np(y1), oracle.chain_step(x_np, w_hat, rms_eps=1e-5))
    w2_hat = oracle.dequantize(*oracle.quantize(w2_np, group=group), group=group)
    assert_close(_np(y2), oracle.chain_step(_np(x2), w2_hat))
