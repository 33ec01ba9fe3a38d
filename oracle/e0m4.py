"""Plain numpy oracle of the E0M4 encoding and of the matmul that consumes it.

Test infrastructure, not a product path.  Everything here follows the paper's
Section 2.3 ("E0M4 FP4 quantization": the Quantization and Dequantization
paragraphs, the dequantization formula and Figure 2) step by step, in the
paper's notation (w0, w1, y1, y2, n, eps); the matmul is the definition
y = x . W of Section 2.2 in double precision.

Logical tensors only: codes are one uint8 per weight in [K, N] order, the two
per-group coefficients are [K/G, N].  The physical nibble layout lives in
``oracle/layout.py``.

Where the paper is silent the readings are (each repeated at its step):
  * the group runs along K for one output column, G = 128 (Section 3.1);
  * n = 1, eps = one fp16 ulp of the binade, so w1 spans [2, 4 - 2^-9];
  * the group range is widened to contain 0, so that the bias is a code;
  * the stored scale is the dequantization scale d (w0-units per w1-unit),
    rounded to fp16; the forward scale is its fp32 reciprocal;
  * Section 2.3, Quantization: the bias keeps only the fraction bits that
    become the code, i.e. it is truncated to the 4-bit grid;
  * the same paragraph wants every w1 inside the binade: w1 is clipped;
  * y1/y2 are sliced from the fp32 bit pattern of w1;
  * w1 = fl32(fl32(w0 * s) + b): two fp32 roundings, no fused multiply-add.

Other bit widths (Section 2.3 notes that the construction carries over to them): every
function takes ``bits`` (default 4), the number of fraction bits kept.  E0M8 (bits = 8)
keeps the eight highest fraction bits, so a code lands on the fp16 fraction with a shift
of 10 - 8 = 2 and the code grid has 256 points; nothing else changes.
"""

from __future__ import annotations

import numpy as np

GROUP = 128  # group size along K (the default of Section 3.1)

_F32 = np.float32


def e0m4_bits(q, n: int = 1, bits: int = 4):
    """fp16 bit pattern built by the dequantization formula of Section 2.3:
    CONST_EXP_BIN_PART | (fp4 << CONST_BIT_SHIFT_NUM).

    FP16 is 1 sign, 5 exponent (bias 15) and 10 fraction bits (Figure 2), so the
    constant exponent part of the binade [2^n, 2^(n+1)) is (15 + n) << 10 and
    the nibble lands on the four highest fraction bits with a shift of 6 (a code of `bits`
    bits on the `bits` highest ones, with a shift of 10 - bits).
    """
    if not 1 <= bits <= 9:
        raise ValueError("bits must be in 1..9")
    q = np.asarray(q).astype(np.uint16)
    return (np.uint16((15 + n) << 10) | (q << np.uint16(10 - bits))).astype(np.uint16)


def e0m4_value(q, n: int = 1, bits: int = 4):
    """as_half() of e0m4_bits: the fp16 number a code stands for inside w1."""
    return e0m4_bits(q, n, bits).view(np.float16)


def _binade(n: int):
    base = _F32(2.0 ** n)
    top = _F32(2.0 ** (n + 1) - 2.0 ** (n - 10))  # 2^(n+1) - eps, eps = fp16 ulp
    return base, top


def quantize(w0, group: int = GROUP, n: int = 1, bits: int = 4):
    """Quantize w0[K, N] (fp32 or fp16 values) group-wise to E0M4 (to E0M<bits> in general:
    read 16 as 2^bits, 15 as 2^bits - 1 and "four" as `bits` below).

    Returns (codes uint8 [K, N], d_h float16 [K/G, N], b_h float16 [K/G, N]):
    the 4-bit codes y1, the stored dequantization scale and the stored bias
    (the bias is a point of the code grid, b_h = as_half(e0m4_bits(z))).

    Steps, Section 2.3 "Quantization", all in fp32 round-to-nearest:
      1. lo = min(0, min w0), hi = max(0, max w0) over the group.
      2. d = (hi - lo) / (TOP - 2^n), TOP = 2^(n+1) - eps;  d_h = fp16(d),
         saturated to the largest finite fp16.  d_h == 0 -> all codes 0, z = 0.
      3. s = 1 / fp32(d_h)                     (the scaling coefficient)
      4. z = clamp(floor((-lo * s) * 16 / 2^n), 0, 15); b = 2^n * (1 + z/16)
         (the bias coefficient with its lower fraction bits zeroed).
      5. w1 = clip(w0 * s + b, 2^n, TOP).
      6. y1 = four highest fraction bits of w1, y2 = the next bit,
         y1 = min(y1 + y2, 15).
    """
    w0 = np.asarray(w0).astype(_F32)
    K, N = w0.shape
    if K % group:
        raise ValueError("K must be a multiple of the group size")
    ng = K // group
    wg = w0.reshape(ng, group, N)
    base, top = _binade(n)
    span = _F32(top - base)

    lo = np.minimum(_F32(0), wg.min(axis=1)).astype(_F32)
    hi = np.maximum(_F32(0), wg.max(axis=1)).astype(_F32)

    with np.errstate(over="ignore"):
        d = ((hi - lo).astype(_F32) / span).astype(_F32)
        d_h = d.astype(np.float16)
    d_h = np.where(np.isinf(d_h), np.float16(65504.0), d_h).astype(np.float16)
    dead = d_h == np.float16(0)

    d_f = d_h.astype(_F32)
    s = np.where(dead, _F32(0), _F32(1) / np.where(dead, _F32(1), d_f)).astype(_F32)

    if not 1 <= bits <= 9:
        raise ValueError("bits must be in 1..9")
    top_code = (1 << bits) - 1
    per_unit = _F32(2.0 ** bits / 2.0 ** n)  # code steps per unit of w1
    t = (((-lo).astype(_F32) * s).astype(_F32) * per_unit).astype(_F32)
    z = np.clip(np.floor(t), 0, top_code).astype(np.int32)
    z = np.where(dead, 0, z)
    b = (base + z.astype(_F32) / per_unit).astype(_F32)  # exact: `bits` fraction bits

    prod = (wg * s[:, None, :]).astype(_F32)
    w1 = (prod + b[:, None, :]).astype(_F32)
    w1 = np.minimum(np.maximum(w1, base), top).astype(_F32)

    pattern = w1.view(np.uint32)
    # the bits + 1 highest fp32 fraction bits (five of them for E0M4)
    t5 = (pattern >> np.uint32(23 - bits - 1)) & np.uint32((2 << bits) - 1)
    y1 = (t5 >> np.uint32(1)).astype(np.int32)
    y2 = (t5 & np.uint32(1)).astype(np.int32)
    y1 = np.minimum(y1 + y2, top_code)
    y1 = np.where(dead[:, None, :], 0, y1)

    codes = y1.astype(np.uint8 if bits <= 8 else np.uint16).reshape(K, N)
    b_h = e0m4_value(z.astype(np.uint16), n, bits).reshape(ng, N)
    return codes, d_h, b_h


def dequantize(codes, d_h, b_h, group: int = GROUP, n: int = 1, bits: int = 4):
    """Section 2.3 "Dequantization": w1 = as_half(EXP | (y1 << 6)), then undo the
    bias and the scale: w_hat = fp16((w1 - b) * d).  w1 - b is a multiple of the
    code step and its product with the 11-bit d is exact in fp32, so the result
    carries exactly one rounding (to fp16, subnormals kept)."""
    codes = np.asarray(codes)
    K, N = codes.shape
    ng = K // group
    w1 = e0m4_value(codes, n, bits).astype(_F32).reshape(ng, group, N)
    diff = (w1 - np.asarray(b_h, dtype=np.float16).astype(_F32)[:, None, :]).astype(_F32)
    out = (diff * np.asarray(d_h, dtype=np.float16).astype(_F32)[:, None, :]).astype(_F32)
    return out.astype(np.float16).reshape(K, N)


def matmul(x_h, w_hat_h, addend_h=None, row_scale=None):
    """Section 2.2: half-precision activation times dequantized weight,
    y[m, n] = sum_k x[m, k] * w_hat[k, n], here evaluated in double.  With `addend_h`
    (fp16 [M, N], or [N] for a bias row) the fused form of Section 2.2's operator fusion: the
    element-wise add that follows the matmul, y + addend, still in double.  With `row_scale`
    (double [M]) every row of the product is multiplied by its factor BEFORE the addend:
    y[m, n] = row_scale[m] * sum_k x[m, k] w_hat[k, n] + addend[m, n]  (the rms-norm that precedes
    a matmul, with its gain folded into the weights, is exactly such a factor: oracle.rms_scale)."""
    x = np.asarray(x_h, dtype=np.float16).astype(np.float64)
    w = np.asarray(w_hat_h, dtype=np.float16).astype(np.float64)
    y = x @ w
    if row_scale is not None:
        y = y * np.asarray(row_scale, dtype=np.float64).reshape(-1, 1)
    if addend_h is not None:
        y = y + np.asarray(addend_h, dtype=np.float16).astype(np.float64)
    return y


def swiglu_blocks(y, block: int = 8):
    """The gated activation of the MLPs the paper runs, fused after the matmul of the joined
    gate and up projections (Section 2.2, element-wise operator fused with the operator before
    it): the columns of y[M, N] alternate between `block` gate columns and `block` up columns,
        out[m, block * j + c] = silu(y[m, 2 * block * j + c]) * y[m, 2 * block * j + block + c],
    silu(g) = g / (1 + exp(-g)), in double.  Returns [M, N / 2]."""
    y = np.asarray(y, dtype=np.float64)
    M, N = y.shape
    if N % (2 * block):
        raise ValueError("N must be a multiple of twice the block")
    yb = y.reshape(M, N // (2 * block), 2, block)
    g, u = yb[:, :, 0, :], yb[:, :, 1, :]
    return (g / (1.0 + np.exp(-g)) * u).reshape(M, N // 2)


def int4_minmax_roundtrip(w0, group: int = GROUP):
    """The comparison format of Section 3.4 (Table 2): group-wise asymmetric INT4
    with step (max - min) / 15 and an integer zero point, in double.  Returns the
    dequantized weights; used only to restate the MAE ratio of Table 2."""
    w0 = np.asarray(w0, dtype=np.float64)
    K, N = w0.shape
    wg = w0.reshape(K // group, group, N)
    lo = wg.min(axis=1, keepdims=True)
    hi = wg.max(axis=1, keepdims=True)
    step = (hi - lo) / 15.0
    step = np.where(step == 0, 1.0, step)
    zp = np.clip(np.round(-lo / step), 0, 15)
    q = np.clip(np.round(wg / step) + zp, 0, 15)
    return ((q - zp) * step).reshape(K, N)
