"""ctypes binding of libtl_e0m4.so: argument marshalling only.

Functions carry the names of the C entry points declared in include/tl_e0m4.h.  Torch is
used for device memory and streams; every computation happens inside the library's CUDA
kernels.  If the shared library has not been built the first call raises: there is no
fallback path.
"""

from __future__ import annotations

import ctypes
import os

_PKG = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_PKG, "libtl_e0m4.so")

TL_OK = 0
TL_F32, TL_F16 = 0, 1
TL_KERNEL_REGISTER, TL_KERNEL_TENSOR = 0, 1
TL_STAGE_DECODE, TL_STAGE_PREFILL = 0, 1
GROUP = 128

STATUS_NAMES = {
    0: "TL_OK", 1: "TL_ERR_NULL", 2: "TL_ERR_SHAPE", 3: "TL_ERR_ALIGN", 4: "TL_ERR_DTYPE",
    5: "TL_ERR_WORKSPACE", 6: "TL_ERR_ARCH", 7: "TL_ERR_CUDA", 8: "TL_ERR_TIMEOUT",
    9: "TL_ERR_LIMIT", 10: "TL_ERR_KEY",
}

# every symbol include/tl_e0m4.h declares: name -> (restype, argtypes)
_vp, _i64, _int, _sz = ctypes.c_void_p, ctypes.c_int64, ctypes.c_int, ctypes.c_size_t
SYMBOLS = {
    "tl_e0m4_packed_sizes": (_int, [_i64, _i64, _int, ctypes.POINTER(_sz), ctypes.POINTER(_sz)]),
    "tl_e0m4_quantize": (_int, [_vp, _int, _i64, _i64, _int, _vp, _vp, _vp]),
    "tl_int4_quantize": (_int, [_vp, _int, _i64, _i64, _int, _vp, _vp, _vp]),
    "tl_e0m4_matmul_add": (_int, [_vp, _vp, _vp, _vp, _vp, _i64, _i64, _i64, _int, _vp, _sz, _vp]),
    "tl_e0m4_matmul_bias": (_int, [_vp, _vp, _vp, _vp, _vp, _i64, _i64, _i64, _int, _vp, _sz, _vp]),
    "tl_e0m4_matmul_swiglu": (_int, [_vp, _vp, _vp, _vp, _i64, _i64, _i64, _int, _vp, _sz, _vp]),
    "tl_kv_append": (_int, [_vp, _vp, _vp, _i64, _i64, _i64, _i64, _i64, _vp]),
    "tl_rmsnorm": (_int, [_vp, _vp, _vp, _vp, _vp, _i64, _i64, ctypes.c_float, _vp]),
    "tl_layernorm": (_int, [_vp, _vp, _vp, _vp, _vp, _vp, _i64, _i64, ctypes.c_float, _vp]),
    "tl_e0m4_dequant": (_int, [_vp, _vp, _i64, _i64, _int, _vp, _vp]),
    "tl_e0m4_matmul_kernel": (_int, [_i64, _i64, _i64]),
    "tl_e0m4_matmul_stage": (_int, [_i64]),
    "tl_e0m4_tuning_set": (_int, [ctypes.c_char_p, _i64]),
    "tl_e0m4_matmul_workspace": (_sz, [_i64, _i64, _i64]),
    "tl_e0m4_workspace_init": (_int, [_vp, _sz, _vp]),
    "tl_e0m4_device_status": (_int, [_vp]),
    "tl_e0m4_matmul": (_int, [_vp, _vp, _vp, _vp, _i64, _i64, _i64, _int, _vp, _sz, _vp]),
    "tl_e0m4_matmul_batch_workspace": (_sz, []),
    "tl_e0m4_matmul_batch": (_int, [_vp, _int, _i64, _int, _vp, _sz, _vp]),
    "tl_e0m4_matmul_batch_host": (_int, [_vp, _int, _i64, _int, _vp, _vp, _sz, _vp, _vp, _sz, _vp, _sz, _vp]),
    "tl_e0m4_matmul_chain_workspace": (_sz, []),
    "tl_e0m4_matmul_chain": (_int, [_vp, _int, _i64, _int, _vp, _sz, _vp]),
    "tl_e0m4_matmul_noalloc": (_int, [_vp, _vp, _vp, _vp, _i64, _i64, _i64, _int, _vp]),
    "tl_e0m4_matmul_noalloc_scratch_bytes": (_sz, []),
    "tl_e0m4_matmul_host_staging": (_sz, [_i64, _i64, _i64]),
    "tl_e0m4_matmul_host": (_int, [_vp, _vp, _vp, _vp, _i64, _i64, _i64, _int, _vp, _sz, _vp]),
    "tl_e0m8_packed_sizes": (_int, [_i64, _i64, _int, ctypes.POINTER(_sz), ctypes.POINTER(_sz)]),
    "tl_e0m8_quantize": (_int, [_vp, _int, _i64, _i64, _int, _vp, _vp, _vp]),
    "tl_e0m8_dequant": (_int, [_vp, _vp, _i64, _i64, _int, _vp, _vp]),
    "tl_e0m8_matmul_workspace": (_sz, [_i64, _i64, _i64]),
    "tl_e0m8_matmul": (_int, [_vp, _vp, _vp, _vp, _i64, _i64, _i64, _int, _vp, _sz, _vp]),
    "tl_e0m8_matmul_batch": (_int, [_vp, _int, _i64, _int, _vp, _sz, _vp]),
    "tl_e0m8_matmul_add": (_int, [_vp, _vp, _vp, _vp, _vp, _i64, _i64, _i64, _int, _vp, _sz, _vp]),
    "tl_e0m8_matmul_bias": (_int, [_vp, _vp, _vp, _vp, _vp, _i64, _i64, _i64, _int, _vp, _sz, _vp]),
    "tl_e0m8_matmul_swiglu": (_int, [_vp, _vp, _vp, _vp, _i64, _i64, _i64, _int, _vp, _sz, _vp]),
    "tl_e0mx_packed_sizes": (_int, [_i64, _i64, _int, _int, ctypes.POINTER(_sz), ctypes.POINTER(_sz)]),
    "tl_e0mx_quantize": (_int, [_vp, _int, _i64, _i64, _int, _int, _vp, _vp, _vp]),
    "tl_e0mx_dequant": (_int, [_vp, _vp, _i64, _i64, _int, _int, _vp, _vp]),
    "tl_e0mx_matmul_workspace": (_sz, [_i64, _i64, _i64, _int]),
    "tl_e0mx_matmul": (_int, [_vp, _vp, _vp, _vp, _i64, _i64, _i64, _int, _int, _vp, _sz, _vp]),
    "tl_e0m4_launch_count": (ctypes.c_uint64, []),
    "tl_status_string": (ctypes.c_char_p, [_int]),
}



class Problem(ctypes.Structure):
    """Mirror of the C struct tl_e0m4_problem."""

    _fields_ = [("x_dev", _vp), ("packed_dev", _vp), ("scales_dev", _vp), ("y_dev", _vp),
                ("K", _i64), ("N", _i64)]


class Step(ctypes.Structure):
    """Mirror of the C struct tl_e0m4_step."""

    _fields_ = [("x_dev", _vp), ("packed_dev", _vp), ("scales_dev", _vp), ("y_dev", _vp), ("addend_dev", _vp),
                ("K", _i64), ("N", _i64), ("epilogue", ctypes.c_int32), ("after_previous", ctypes.c_int32),
                ("rms_scale", ctypes.c_int32), ("rms_eps", ctypes.c_float)]


TL_EPILOGUE_NONE, TL_EPILOGUE_ADD, TL_EPILOGUE_BIAS, TL_EPILOGUE_SWIGLU = 0, 1, 2, 3
_EPILOGUES = {"none": 0, "add": 1, "bias": 2, "swiglu": 3}

_lib = None


class TlError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        text = lib().tl_status_string(status).decode()
        super().__init__(f"{where}: {STATUS_NAMES.get(status, status)} ({text})")


def lib() -> ctypes.CDLL:
    """Load the shared library (once).  Raises if it has not been built."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise RuntimeError(
                f"{LIB_PATH} is missing: build it with `python -m paper_2403_20041_b200.build` "
                "(needs nvcc). There is no CPU fallback.")
        handle = ctypes.CDLL(LIB_PATH)
        for name, (res, args) in SYMBOLS.items():
            fn = getattr(handle, name)
            fn.restype = res
            fn.argtypes = args
        _lib = handle
    return _lib


def _check(status: int, where: str) -> None:
    if status != TL_OK:
        raise TlError(status, where)


def _stream(stream) -> int:
    import torch

    if stream is None:
        stream = torch.cuda.current_stream()
    return stream.cuda_stream if hasattr(stream, "cuda_stream") else int(stream)


def _dev_ptr(t, name: str) -> int:
    if not t.is_cuda or not t.is_contiguous():
        raise ValueError(f"{name} must be a contiguous CUDA tensor")
    return t.data_ptr()


def tl_e0m4_packed_sizes(K: int, N: int, group: int = GROUP):
    """(packed_bytes, scales_bytes) for a [K, N] weight."""
    a, b = _sz(0), _sz(0)
    _check(lib().tl_e0m4_packed_sizes(K, N, group, ctypes.byref(a), ctypes.byref(b)),
           "tl_e0m4_packed_sizes")
    return a.value, b.value


def tl_e0m4_quantize(w, packed=None, scales=None, group: int = GROUP, stream=None):
    """Quantize a CUDA weight tensor [K, N] (fp32 or fp16).  Returns (packed, scales) as
    uint8 CUDA tensors in the library's packed layout."""
    return _quantize("tl_e0m4_quantize", w, packed, scales, group, stream)


def tl_int4_quantize(w, packed=None, scales=None, group: int = GROUP, stream=None):
    """Same container, codes of the group-wise asymmetric INT4 comparison format."""
    return _quantize("tl_int4_quantize", w, packed, scales, group, stream)


def _quantize(symbol, w, packed, scales, group, stream):
    import torch

    K, N = w.shape
    pb, sb = tl_e0m4_packed_sizes(K, N, group)
    if packed is None:
        packed = torch.empty(pb, dtype=torch.uint8, device=w.device)
    if scales is None:
        scales = torch.empty(sb, dtype=torch.uint8, device=w.device)
    if w.dtype == torch.float32:
        dt = TL_F32
    elif w.dtype == torch.float16:
        dt = TL_F16
    else:
        raise ValueError("weights must be float32 or float16")
    _check(getattr(lib(), symbol)(_dev_ptr(w, "w"), dt, K, N, group, _dev_ptr(packed, "packed"),
                                  _dev_ptr(scales, "scales"), _stream(stream)), symbol)
    return packed, scales


def tl_e0m4_dequant(packed, scales, K: int, N: int, out=None, group: int = GROUP, stream=None):
    """Expand packed weights to a dense fp16 [K, N] CUDA tensor."""
    import torch

    if out is None:
        out = torch.empty((K, N), dtype=torch.float16, device=packed.device)
    _check(lib().tl_e0m4_dequant(_dev_ptr(packed, "packed"), _dev_ptr(scales, "scales"), K, N, group,
                                 _dev_ptr(out, "out"), _stream(stream)), "tl_e0m4_dequant")
    return out


def tl_e0m8_packed_sizes(K: int, N: int, group: int = GROUP):
    """(packed_bytes, scales_bytes) of a [K, N] weight in the 8-bit container."""
    a, b = _sz(0), _sz(0)
    _check(lib().tl_e0m8_packed_sizes(K, N, group, ctypes.byref(a), ctypes.byref(b)), "tl_e0m8_packed_sizes")
    return a.value, b.value


def tl_e0m8_quantize(w, packed=None, scales=None, group: int = GROUP, stream=None):
    """Quantize a CUDA weight tensor [K, N] (fp32 or fp16) to E0M8.  Returns (packed, scales) as
    uint8 CUDA tensors."""
    import torch

    K, N = w.shape
    pb, sb = tl_e0m8_packed_sizes(K, N, group)
    if packed is None:
        packed = torch.empty(pb, dtype=torch.uint8, device=w.device)
    if scales is None:
        scales = torch.empty(sb, dtype=torch.uint8, device=w.device)
    if w.dtype not in (torch.float32, torch.float16):
        raise ValueError("weights must be float32 or float16")
    dt = TL_F32 if w.dtype == torch.float32 else TL_F16
    _check(lib().tl_e0m8_quantize(_dev_ptr(w, "w"), dt, K, N, group, _dev_ptr(packed, "packed"),
                                  _dev_ptr(scales, "scales"), _stream(stream)), "tl_e0m8_quantize")
    return packed, scales


def tl_e0m8_dequant(packed, scales, K: int, N: int, out=None, group: int = GROUP, stream=None):
    """Expand E0M8 weights to a dense fp16 [K, N] CUDA tensor."""
    import torch

    if out is None:
        out = torch.empty((K, N), dtype=torch.float16, device=packed.device)
    _check(lib().tl_e0m8_dequant(_dev_ptr(packed, "packed"), _dev_ptr(scales, "scales"), K, N, group,
                                 _dev_ptr(out, "out"), _stream(stream)), "tl_e0m8_dequant")
    return out


def tl_e0m8_matmul_workspace(M: int, K: int, N: int) -> int:
    return int(lib().tl_e0m8_matmul_workspace(M, K, N))


def _matmul8(symbol, x, packed, scales, N, extra, y, y_cols, workspace, group, stream):
    import torch

    M, K = x.shape
    if x.dtype != torch.float16 or (extra is not None and extra.dtype != torch.float16):
        raise ValueError("x (and the addend or bias) must be float16")
    if y is None:
        y = torch.empty((M, y_cols), dtype=torch.float16, device=x.device)
    need = tl_e0m8_matmul_workspace(M, K, N)
    if need and workspace is None:
        workspace = tl_e0m4_workspace(need, x.device, stream=stream)
    ws_ptr = _dev_ptr(workspace, "workspace") if workspace is not None else None
    ws_bytes = workspace.numel() * workspace.element_size() if workspace is not None else 0
    args = [_dev_ptr(x, "x"), _dev_ptr(packed, "packed"), _dev_ptr(scales, "scales")]
    if extra is not None:
        args.append(_dev_ptr(extra, "addend"))
    _check(getattr(lib(), symbol)(*args, _dev_ptr(y, "y"), M, K, N, group, ws_ptr, ws_bytes, _stream(stream)), symbol)
    return y


def tl_e0m8_matmul(x, packed, scales, N: int, y=None, workspace=None, group: int = GROUP, stream=None):
    """y[M, N] = x[M, K] . W with W in packed E0M8 form (fp16 in/out, fp32 accumulation)."""
    return _matmul8("tl_e0m8_matmul", x, packed, scales, N, None, y, N, workspace, group, stream)


def tl_e0m8_matmul_add(x, packed, scales, N: int, addend, y=None, workspace=None, group: int = GROUP, stream=None):
    """y[M, N] = fp16(x . W + addend) for E0M8 weights; y defaults to writing over the addend."""
    if tuple(addend.shape) != (x.shape[0], N):
        raise ValueError("addend must be [M, N]")
    return _matmul8("tl_e0m8_matmul_add", x, packed, scales, N, addend, addend if y is None else y, N, workspace,
                    group, stream)


def tl_e0m8_matmul_bias(x, packed, scales, N: int, bias, y=None, workspace=None, group: int = GROUP, stream=None):
    """y[M, N] = fp16(x . W + bias[N]) for E0M8 weights."""
    if tuple(bias.shape) != (N,):
        raise ValueError("bias must be [N]")
    return _matmul8("tl_e0m8_matmul_bias", x, packed, scales, N, bias, y, N, workspace, group, stream)


def tl_e0m8_matmul_swiglu(x, packed, scales, N: int, y=None, workspace=None, group: int = GROUP, stream=None):
    """y[M, N / 2] = silu(gate) * up over column blocks of eight of x . W, for E0M8 weights."""
    return _matmul8("tl_e0m8_matmul_swiglu", x, packed, scales, N, None, y, N // 2, workspace, group, stream)


def tl_e0mx_packed_sizes(K: int, N: int, bits: int, group: int = GROUP):
    """(packed_bytes, scales_bytes) of a [K, N] weight in the 3-bit or 5-bit container."""
    a, b = _sz(0), _sz(0)
    _check(lib().tl_e0mx_packed_sizes(K, N, group, bits, ctypes.byref(a), ctypes.byref(b)), "tl_e0mx_packed_sizes")
    return a.value, b.value


def tl_e0mx_quantize(w, bits: int, packed=None, scales=None, group: int = GROUP, stream=None):
    """Quantize a CUDA weight tensor [K, N] (fp32 or fp16) to E0M3 or E0M5.  Returns (packed, scales)."""
    import torch

    K, N = w.shape
    pb, sb = tl_e0mx_packed_sizes(K, N, bits, group)
    if packed is None:
        packed = torch.empty(pb, dtype=torch.uint8, device=w.device)
    if scales is None:
        scales = torch.empty(sb, dtype=torch.uint8, device=w.device)
    if w.dtype not in (torch.float32, torch.float16):
        raise ValueError("weights must be float32 or float16")
    dt = TL_F32 if w.dtype == torch.float32 else TL_F16
    _check(lib().tl_e0mx_quantize(_dev_ptr(w, "w"), dt, K, N, group, bits, _dev_ptr(packed, "packed"),
                                  _dev_ptr(scales, "scales"), _stream(stream)), "tl_e0mx_quantize")
    return packed, scales


def tl_e0mx_dequant(packed, scales, K: int, N: int, bits: int, out=None, group: int = GROUP, stream=None):
    """Expand E0M3 / E0M5 weights to a dense fp16 [K, N] CUDA tensor."""
    import torch

    if out is None:
        out = torch.empty((K, N), dtype=torch.float16, device=packed.device)
    _check(lib().tl_e0mx_dequant(_dev_ptr(packed, "packed"), _dev_ptr(scales, "scales"), K, N, group, bits,
                                 _dev_ptr(out, "out"), _stream(stream)), "tl_e0mx_dequant")
    return out


def tl_e0mx_matmul(x, packed, scales, N: int, bits: int, y=None, workspace=None, group: int = GROUP, stream=None):
    """y[M, N] = x[M, K] . W with W in packed E0M3 / E0M5 form (fp16 in/out, fp32 accumulation)."""
    import torch

    M, K = x.shape
    if x.dtype != torch.float16:
        raise ValueError("x must be float16")
    if y is None:
        y = torch.empty((M, N), dtype=torch.float16, device=x.device)
    need = int(lib().tl_e0mx_matmul_workspace(M, K, N, bits))
    if need and workspace is None:
        workspace = tl_e0m4_workspace(need, x.device, stream=stream)
    ws_ptr = _dev_ptr(workspace, "workspace") if workspace is not None else None
    ws_bytes = workspace.numel() * workspace.element_size() if workspace is not None else 0
    _check(lib().tl_e0mx_matmul(_dev_ptr(x, "x"), _dev_ptr(packed, "packed"), _dev_ptr(scales, "scales"),
                                _dev_ptr(y, "y"), M, K, N, group, bits, ws_ptr, ws_bytes, _stream(stream)),
           "tl_e0mx_matmul")
    return y


def tl_kv_append(cache, new, position_ids, stream=None):
    """cache[b, h, position_ids[b] + s, :] = new[b, h, s, :] in place.  cache fp16 [B, H, L, D], new fp16
    [B, H, S, D], position_ids int32 [B], all CUDA tensors."""
    import torch

    B, H, L, D = cache.shape
    S = new.shape[2]
    if cache.dtype != torch.float16 or new.dtype != torch.float16 or position_ids.dtype != torch.int32:
        raise ValueError("cache and new must be float16, position_ids int32")
    if tuple(new.shape) != (B, H, S, D) or tuple(position_ids.shape) != (B,):
        raise ValueError("shape mismatch")
    _check(lib().tl_kv_append(_dev_ptr(cache, "cache"), _dev_ptr(new, "new"), _dev_ptr(position_ids, "position_ids"),
                              B, H, L, S, D, _stream(stream)), "tl_kv_append")
    return cache


def tl_rmsnorm(x, gamma, eps: float, residual=None, sum_out=None, y=None, stream=None):
    """Fused rms-norm of fp16 x [M, K] (CUDA); with `residual` it normalizes fp16(x + residual) and
    writes that sum to `sum_out` (allocated when `residual` is given and `sum_out` is None).
    Returns y, or (y, sum_out) with a residual."""
    import torch

    M, K = x.shape
    if y is None:
        y = torch.empty_like(x)
    if residual is not None and sum_out is None:
        sum_out = torch.empty_like(x)
    null = ctypes.c_void_p(None)
    _check(lib().tl_rmsnorm(_dev_ptr(x, "x"), _dev_ptr(residual, "residual") if residual is not None else null,
                            _dev_ptr(gamma, "gamma"), _dev_ptr(sum_out, "sum_out") if sum_out is not None else null,
                            _dev_ptr(y, "y"), M, K, float(eps), _stream(stream)), "tl_rmsnorm")
    return y if residual is None else (y, sum_out)


def tl_layernorm(x, gamma, beta, eps: float, residual=None, sum_out=None, y=None, stream=None):
    """Fused layer-norm of fp16 x [M, K] (CUDA); arguments and results as tl_rmsnorm, plus beta [K]."""
    import torch

    M, K = x.shape
    if y is None:
        y = torch.empty_like(x)
    if residual is not None and sum_out is None:
        sum_out = torch.empty_like(x)
    null = ctypes.c_void_p(None)
    _check(lib().tl_layernorm(_dev_ptr(x, "x"), _dev_ptr(residual, "residual") if residual is not None else null,
                              _dev_ptr(gamma, "gamma"), _dev_ptr(beta, "beta"),
                              _dev_ptr(sum_out, "sum_out") if sum_out is not None else null,
                              _dev_ptr(y, "y"), M, K, float(eps), _stream(stream)), "tl_layernorm")
    return y if residual is None else (y, sum_out)


def tl_e0m4_matmul_kernel(M: int, K: int, N: int) -> int:
    return lib().tl_e0m4_matmul_kernel(M, K, N)


def tl_e0m4_matmul_stage(M: int) -> int:
    return lib().tl_e0m4_matmul_stage(M)


def tl_e0m4_tuning_set(key, value: int = -1) -> None:
    """Overrides one launch heuristic process-wide (diagnostics and tests); value < 0 restores the
    library's own choice, key None restores all."""
    _check(lib().tl_e0m4_tuning_set(key.encode() if key is not None else None, int(value)), "tl_e0m4_tuning_set")


def tl_e0m4_matmul_workspace(M: int, K: int, N: int) -> int:
    return lib().tl_e0m4_matmul_workspace(M, K, N)


def tl_e0m4_workspace(nbytes: int, device, stream=None):
    """A zeroed workspace of `nbytes` bytes (allocated by torch, zeroed by the library)."""
    import torch

    ws = torch.empty(max(int(nbytes), 16), dtype=torch.uint8, device=device)
    _check(lib().tl_e0m4_workspace_init(ws.data_ptr(), ws.numel(), _stream(stream)),
           "tl_e0m4_workspace_init")
    return ws


def tl_e0m4_device_status(stream=None) -> int:
    """Status word set by a kernel whose bounded wait expired (0 = fine); synchronizes."""
    return lib().tl_e0m4_device_status(_stream(stream))


def tl_e0m4_matmul(x, packed, scales, N: int, y=None, workspace=None, group: int = GROUP,
                   stream=None):
    """y[M, N] = x[M, K] . W with W in packed E0M4 form (fp16 in/out, fp32 accumulation)."""
    import torch

    M, K = x.shape
    if x.dtype != torch.float16:
        raise ValueError("x must be float16")
    if y is None:
        y = torch.empty((M, N), dtype=torch.float16, device=x.device)
    need = tl_e0m4_matmul_workspace(M, K, N)
    if need and workspace is None:
        workspace = tl_e0m4_workspace(need, x.device, stream=stream)
    ws_ptr = _dev_ptr(workspace, "workspace") if workspace is not None else None
    ws_bytes = workspace.numel() * workspace.element_size() if workspace is not None else 0
    _check(lib().tl_e0m4_matmul(_dev_ptr(x, "x"), _dev_ptr(packed, "packed"),
                                _dev_ptr(scales, "scales"), _dev_ptr(y, "y"), M, K, N, group,
                                ws_ptr, ws_bytes, _stream(stream)), "tl_e0m4_matmul")
    return y


def tl_e0m4_matmul_add(x, packed, scales, N: int, addend, y=None, workspace=None, group: int = GROUP,
                       stream=None):
    """y[M, N] = fp16(x . W + addend): the matmul with the residual add fused in.  `addend` is a fp16
    CUDA tensor [M, N]; y defaults to writing over it."""
    import torch

    M, K = x.shape
    if x.dtype != torch.float16 or addend.dtype != torch.float16:
        raise ValueError("x and addend must be float16")
    if y is None:
        y = addend
    need = tl_e0m4_matmul_workspace(M, K, N)
    if need and workspace is None:
        workspace = tl_e0m4_workspace(need, x.device, stream=stream)
    ws_ptr = _dev_ptr(workspace, "workspace") if workspace is not None else None
    ws_bytes = workspace.numel() * workspace.element_size() if workspace is not None else 0
    _check(lib().tl_e0m4_matmul_add(_dev_ptr(x, "x"), _dev_ptr(packed, "packed"), _dev_ptr(scales, "scales"),
                                    _dev_ptr(addend, "addend"), _dev_ptr(y, "y"), M, K, N, group,
                                    ws_ptr, ws_bytes, _stream(stream)), "tl_e0m4_matmul_add")
    return y


def tl_e0m4_matmul_bias(x, packed, scales, N: int, bias, y=None, workspace=None, group: int = GROUP, stream=None):
    """y = fp16(x W + bias) with bias fp16 [N] shared by all tokens (CUDA); arguments as tl_e0m4_matmul_add."""
    import torch

    M, K = x.shape
    if y is None:
        y = torch.empty((M, N), dtype=torch.float16, device=x.device)
    ws_bytes = tl_e0m4_matmul_workspace(M, K, N)
    if workspace is None and ws_bytes:
        workspace = tl_e0m4_workspace(ws_bytes, x.device, stream)
    ws_ptr = _dev_ptr(workspace, "workspace") if workspace is not None else ctypes.c_void_p(None)
    ws_len = workspace.numel() * workspace.element_size() if workspace is not None else 0
    _check(lib().tl_e0m4_matmul_bias(_dev_ptr(x, "x"), _dev_ptr(packed, "packed"), _dev_ptr(scales, "scales"),
                                     _dev_ptr(bias, "bias"), _dev_ptr(y, "y"), M, K, N, group, ws_ptr, ws_len,
                                     _stream(stream)), "tl_e0m4_matmul_bias")
    return y


def tl_e0m4_matmul_swiglu(x, packed, scales, N: int, y=None, workspace=None, group: int = GROUP, stream=None):
    """y[M, N/2] = silu(gate) * up of x . W, where W's columns hold gate and up interleaved in blocks
    of eight (see interleave_gate_up)."""
    import torch

    M, K = x.shape
    if x.dtype != torch.float16:
        raise ValueError("x must be float16")
    if y is None:
        y = torch.empty((M, N // 2), dtype=torch.float16, device=x.device)
    need = tl_e0m4_matmul_workspace(M, K, N)
    if need and workspace is None:
        workspace = tl_e0m4_workspace(need, x.device, stream=stream)
    ws_ptr = _dev_ptr(workspace, "workspace") if workspace is not None else None
    ws_bytes = workspace.numel() * workspace.element_size() if workspace is not None else 0
    _check(lib().tl_e0m4_matmul_swiglu(_dev_ptr(x, "x"), _dev_ptr(packed, "packed"), _dev_ptr(scales, "scales"),
                                       _dev_ptr(y, "y"), M, K, N, group, ws_ptr, ws_bytes, _stream(stream)),
           "tl_e0m4_matmul_swiglu")
    return y


def interleave_gate_up(w_gate, w_up, block: int = 8):
    """[K, F] gate and up weights -> [K, 2F] with `block` gate columns, then the matching `block` up
    columns, and so on: the column order tl_e0m4_matmul_swiglu expects (argument marshalling only)."""
    import torch

    K, F = w_gate.shape
    return torch.stack((w_gate.reshape(K, F // block, block), w_up.reshape(K, F // block, block)), dim=2).reshape(K, 2 * F)


def tl_e0m4_matmul_batch_workspace() -> int:
    return lib().tl_e0m4_matmul_batch_workspace()


def make_problem_array(problems):
    """ctypes array of tl_e0m4_problem from (x, packed, scales, y) CUDA tensor tuples; y is
    [M, N] and x is [M, K]."""
    arr = (Problem * len(problems))()
    for i, (x, packed, scales, y) in enumerate(problems):
        arr[i] = Problem(_dev_ptr(x, "x"), _dev_ptr(packed, "packed"), _dev_ptr(scales, "scales"),
                         _dev_ptr(y, "y"), x.shape[1], y.shape[1])
    return arr


def tl_e0m4_matmul_batch(problems, M: int, workspace, group: int = GROUP, stream=None):
    """Runs independent problems that share M (<= 128) in one persistent launch per list chunk
    (the GEMV list kernel up to 8 tokens, the tensor-core list kernel above).
    `problems` is a list of (x, packed, scales, y) tensor tuples or an array built by
    make_problem_array()."""
    arr = problems if isinstance(problems, ctypes.Array) else make_problem_array(problems)
    _check(lib().tl_e0m4_matmul_batch(ctypes.cast(arr, _vp), len(arr), M, group,
                                      _dev_ptr(workspace, "workspace"),
                                      workspace.numel() * workspace.element_size(), _stream(stream)),
           "tl_e0m4_matmul_batch")


def tl_e0m8_matmul_batch(problems, M: int, workspace, group: int = GROUP, stream=None):
    """The same for E0M8 weights (M <= 128): one persistent tensor-core launch per 22 problems."""
    arr = problems if isinstance(problems, ctypes.Array) else make_problem_array(problems)
    _check(lib().tl_e0m8_matmul_batch(ctypes.cast(arr, _vp), len(arr), M, group,
                                      _dev_ptr(workspace, "workspace"),
                                      workspace.numel() * workspace.element_size(), _stream(stream)),
           "tl_e0m8_matmul_batch")


def tl_e0m4_matmul_batch_host(problems, M: int, x_host, x_stage, y_host, y_stage, workspace,
                              group: int = GROUP, stream=None):
    """Host-buffer variant of the batch: one copy of x_host into x_stage, the batch, one copy
    of y_stage into y_host, all on `stream`.  The problems' x/y must be views of the stages."""
    arr = problems if isinstance(problems, ctypes.Array) else make_problem_array(problems)
    _check(lib().tl_e0m4_matmul_batch_host(
        ctypes.cast(arr, _vp), len(arr), M, group, x_host.data_ptr(), _dev_ptr(x_stage, "x_stage"),
        x_stage.numel() * x_stage.element_size(), y_host.data_ptr(), _dev_ptr(y_stage, "y_stage"),
        y_stage.numel() * y_stage.element_size(), _dev_ptr(workspace, "workspace"),
        workspace.numel() * workspace.element_size(), _stream(stream)), "tl_e0m4_matmul_batch_host")


def tl_e0m4_matmul_chain_workspace() -> int:
    return lib().tl_e0m4_matmul_chain_workspace()


def make_step_array(steps):
    """ctypes array of tl_e0m4_step from dicts with the keys x, packed, scales, y (CUDA tensors) and,
    optionally, epilogue ("none", "add", "bias", "swiglu"), addend (CUDA tensor), after_previous (bool),
    rms_eps (float or None)."""
    arr = (Step * len(steps))()
    for i, st in enumerate(steps):
        x, y = st["x"], st["y"]
        epi = _EPILOGUES[st.get("epilogue", "none")]
        addend = st.get("addend")
        N = y.shape[1] * (2 if epi == TL_EPILOGUE_SWIGLU else 1)
        eps = st.get("rms_eps")
        arr[i] = Step(_dev_ptr(x, "x"), _dev_ptr(st["packed"], "packed"), _dev_ptr(st["scales"], "scales"),
                      _dev_ptr(y, "y"), _dev_ptr(addend, "addend") if addend is not None else None,
                      x.shape[1], N, epi, 1 if st.get("after_previous") else 0, 0 if eps is None else 1,
                      0.0 if eps is None else float(eps))
    return arr


def tl_e0m4_matmul_chain(steps, M: int, workspace, group: int = GROUP, stream=None):
    """Runs a list of decode steps (M <= 8), some of which consume what earlier ones produce, in one
    persistent launch per 128 steps.  `steps` is a list of dicts (see make_step_array) or an array
    built by it."""
    arr = steps if isinstance(steps, ctypes.Array) else make_step_array(steps)
    _check(lib().tl_e0m4_matmul_chain(ctypes.cast(arr, _vp), len(arr), M, group, _dev_ptr(workspace, "workspace"),
                                      workspace.numel() * workspace.element_size(), _stream(stream)),
           "tl_e0m4_matmul_chain")


def tl_e0m4_matmul_noalloc(x, packed, scales, y, group: int = GROUP, stream=None):
    """Decode matmul (M <= 16) into the caller's `y` for callers that may not allocate device
    memory: the split-K scratch is an array inside the library, nothing is allocated here or
    there.  All tensors, `y` included, must already exist.  Calls on one device must be ordered
    (they share the array); make the first call on a device outside stream capture."""
    M, K = x.shape
    N = y.shape[1]
    _check(lib().tl_e0m4_matmul_noalloc(_dev_ptr(x, "x"), _dev_ptr(packed, "packed"),
                                        _dev_ptr(scales, "scales"), _dev_ptr(y, "y"), M, K, N, group,
                                        _stream(stream)), "tl_e0m4_matmul_noalloc")
    return y


def tl_e0m4_matmul_noalloc_scratch_bytes() -> int:
    return lib().tl_e0m4_matmul_noalloc_scratch_bytes()


def tl_e0m4_matmul_host_staging(M: int, K: int, N: int) -> int:
    return lib().tl_e0m4_matmul_host_staging(M, K, N)


def tl_e0m4_matmul_host(x_host, packed, scales, N: int, y_host, staging, group: int = GROUP,
                        stream=None):
    """Host-buffer variant: x_host / y_host are CPU fp16 tensors (pinned for real overlap);
    the copies and the matmul are enqueued on `stream`; synchronize before reading y_host."""
    M, K = x_host.shape
    if x_host.is_cuda or y_host.is_cuda:
        raise ValueError("x_host and y_host must be CPU tensors")
    _check(lib().tl_e0m4_matmul_host(x_host.data_ptr(), _dev_ptr(packed, "packed"),
                                     _dev_ptr(scales, "scales"), y_host.data_ptr(), M, K, N, group,
                                     _dev_ptr(staging, "staging"),
                                     staging.numel() * staging.element_size(), _stream(stream)),
           "tl_e0m4_matmul_host")
    return y_host


def tl_e0m4_launch_count() -> int:
    return int(lib().tl_e0m4_launch_count())


def tl_status_string(status: int) -> str:
    return lib().tl_status_string(status).decode()
