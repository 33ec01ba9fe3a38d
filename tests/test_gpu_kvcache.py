"""GPU parity of the in-place KV-cache append against the oracle (byte-exact: pure data movement)."""

import numpy as np
import pytest
import torch

import oracle

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def dev():
    return torch.device("cuda:0")


@pytest.mark.parametrize("B,H,L,S,D", [(1, 2, 64, 1, 128), (3, 4, 40, 5, 64), (2, 32, 2048, 128, 128), (5, 1, 7, 7, 8)])
def test_kv_append_matches_oracle(lib, dev, B, H, L, S, D):
    rng = np.random.default_rng(B * 1000 + S)
    cache = rng.normal(size=(B, H, L, D)).astype(np.float16)
    new = rng.normal(size=(B, H, S, D)).astype(np.float16)
    pos = rng.integers(0, L - S + 1, size=B).astype(np.int32)
    pos[0] = L - S                                  # the last rows of the cache
    ref = oracle.kv_append(cache, new, pos)
    c = torch.from_numpy(cache).to(dev)
    lib.tl_kv_append(c, torch.from_numpy(new).to(dev), torch.from_numpy(pos).to(dev))
    torch.cuda.synchronize()
    assert np.array_equal(c.cpu().numpy().view(np.uint16), ref.view(np.uint16))
    assert lib.tl_e0m4_device_status() == 0


def test_decode_steps_fill_the_cache_like_one_prefill(lib, dev):
    rng = np.random.default_rng(4)
    B, H, L, D = 2, 3, 16, 32
    new = rng.normal(size=(B, H, 6, D)).astype(np.float16)
    whole = torch.zeros((B, H, L, D), dtype=torch.float16, device=dev)
    lib.tl_kv_append(whole, torch.from_numpy(new).to(dev), torch.tensor([3, 9], dtype=torch.int32, device=dev))
    steps = torch.zeros_like(whole)
    for s in range(6):
        lib.tl_kv_append(steps, torch.from_numpy(np.ascontiguousarray(new[:, :, s:s + 1])).to(dev),
                         torch.tensor([3 + s, 9 + s], dtype=torch.int32, device=dev))
    torch.cuda.synchronize()
    assert torch.equal(whole, steps)


def test_rows_beyond_the_cache_are_refused_without_a_fault(lib, dev):
    B, H, L, S, D = 2, 2, 8, 3, 16
    c = torch.ones((B, H, L, D), dtype=torch.float16, device=dev)
    new = torch.full((B, H, S, D), 2.0, dtype=torch.float16, device=dev)
    lib.tl_kv_append(c, new, torch.tensor([6, 1], dtype=torch.int32, device=dev))   # entry 0 would end at row 9
    torch.cuda.synchronize()
    out = c.cpu().numpy()
    assert (out[0] == 1.0).all()                         # untouched
    assert (out[1, :, 1:4] == 2.0).all() and (out[1, :, 4:] == 1.0).all()
    assert lib.tl_e0m4_device_status() == 2              # TL_ERR_SHAPE, raised on the device
    assert lib.tl_e0m4_device_status() == 0              # reading the word clears it
    with pytest.raises(lib.TlError):                     # more new rows than the cache has: refused on the host
        lib.tl_kv_append(c, torch.zeros((B, H, L + 1, D), dtype=torch.float16, device=dev),
                         torch.zeros(B, dtype=torch.int32, device=dev))


@pytest.mark.parametrize("bad", [2**31 - 1, 2**31 - 2, -(2**31), -1, 6])
def test_positions_at_the_ends_of_int32_are_refused(lib, dev, bad):
    # position + S would wrap around in 32-bit arithmetic; the guard compares position with L - S
    # instead, skips the entry's stores and raises the status word
    B, H, L, S, D = 2, 2, 8, 3, 16
    c = torch.ones((B, H, L, D), dtype=torch.float16, device=dev)
    new = torch.full((B, H, S, D), 2.0, dtype=torch.float16, device=dev)
    lib.tl_kv_append(c, new, torch.tensor([bad, 5], dtype=torch.int32, device=dev))
    torch.cuda.synchronize()
    out = c.cpu().numpy()
    assert (out[0] == 1.0).all()
    assert (out[1, :, 5:8] == 2.0).all() and (out[1, :, :5] == 1.0).all()
    assert lib.tl_e0m4_device_status() == 2
