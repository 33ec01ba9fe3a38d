"""CPU oracle of the fused rms-norm and layer-norm operators (Section 2.2: the small operators
that make up layer-norm and rms-norm are fused into one).  TEST INFRASTRUCTURE ONLY: imported by tests/, by smoke() and by
the benchmark's CPU legs, never by the product path.

The paper names the operator and gives no formula; the definition used is the one of the
models it runs (Llama, Gemma, Qwen, ChatGLM2):
    y[m, k] = x[m, k] / sqrt(mean_k(x[m, :]^2) + eps) * gamma[k]
computed here in double on the fp16 inputs and rounded once to fp16.  With a residual input
the operator first forms s = fp16(x + r), returns it, and normalizes s (the pair of
element-wise add and norm that closes every transformer block).

Layer-norm is the textbook definition over the last axis with the biased variance:
    y[m, k] = (x[m, k] - mean_k x[m, :]) / sqrt(var_k x[m, :] + eps) * gamma[k] + beta[k]
with the same residual form.

Parity unpinned: nothing (pins in tests/test_oracle_norm.py).
"""
import numpy as np


def rmsnorm(x_h, gamma_h, eps: float, residual_h=None):
    """x_h [M, K] fp16, gamma_h [K] fp16 -> y fp16 [M, K]  (and s fp16 [M, K] with a residual)."""
    x = np.asarray(x_h, dtype=np.float16).astype(np.float64)
    s_h = None
    if residual_h is not None:
        s_h = (x + np.asarray(residual_h, dtype=np.float16).astype(np.float64)).astype(np.float16)
        x = s_h.astype(np.float64)
    g = np.asarray(gamma_h, dtype=np.float16).astype(np.float64)
    ms = (x * x).mean(axis=1, keepdims=True)
    with np.errstate(over="ignore"):
        y = (x / np.sqrt(ms + float(eps)) * g[None, :]).astype(np.float16)
    return y if s_h is None else (y, s_h)


def rms_scale(x_h, eps: float):
    """The row factor of the rms-norm alone: r[m] = 1 / sqrt(mean_k(x[m, :]^2) + eps), double [M].
    rmsnorm(x, gamma) = x * r * gamma; with gamma folded into the weights of the matmul that
    follows, (x * r * gamma) . W = r * (x . (gamma * W)): the norm becomes a factor per output row."""
    x = np.asarray(x_h, dtype=np.float16).astype(np.float64)
    return 1.0 / np.sqrt((x * x).mean(axis=1) + float(eps))


def layernorm(x_h, gamma_h, beta_h, eps: float, residual_h=None):
    """x_h [M, K] fp16, gamma_h / beta_h [K] fp16 -> y fp16 [M, K]  (and s fp16 [M, K] with a residual)."""
    x = np.asarray(x_h, dtype=np.float16).astype(np.float64)
    s_h = None
    if residual_h is not None:
        s_h = (x + np.asarray(residual_h, dtype=np.float16).astype(np.float64)).astype(np.float16)
        x = s_h.astype(np.float64)
    g = np.asarray(gamma_h, dtype=np.float16).astype(np.float64)
    b = np.asarray(beta_h, dtype=np.float16).astype(np.float64)
    mean = x.mean(axis=1, keepdims=True)
    c = x - mean
    var = (c * c).mean(axis=1, keepdims=True)
    with np.errstate(over="ignore"):
        y = (c / np.sqrt(var + float(eps)) * g[None, :] + b[None, :]).astype(np.float16)
    return y if s_h is None else (y, s_h)
