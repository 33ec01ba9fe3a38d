"""CPU oracle of one step of a decode chain: the matmul of Section 2.2 with the element-wise
operators around it fused in (Section 2.2, operator fusions).  TEST INFRASTRUCTURE ONLY.

A step is   Y = r * (x . W_hat) + addend ,  out = Y  or  swiglu_blocks(Y) ,  all in double:
  * r is the rms-norm's row factor of the step's own input (oracle.rms_scale) when the step
    carries a norm whose gain was folded into the weights, else 1;
  * addend is a residual [M, N], a bias row [N], or nothing;
  * swiglu_blocks is the gated activation over column blocks of eight.
Every piece is one of the pinned functions of this package; this module only strings them
together in the order the operators have in a transformer block.  A chain is a sequence of such
steps, each reading fp16 tensors that earlier steps wrote (rounded to fp16 once, as stored).

Parity unpinned: nothing (pins in tests/test_oracle_chain.py).
"""
import numpy as np

from .e0m4 import matmul, swiglu_blocks
from .norm import rms_scale


def chain_step(x_h, w_hat_h, epilogue: str = "none", addend_h=None, rms_eps=None):
    """x_h fp16 [M, K], w_hat_h fp16 [K, N] (dequantized weights) -> double [M, N] ([M, N / 2] for
    "swiglu").  epilogue: "none", "add" (addend_h fp16 [M, N]), "bias" (addend_h fp16 [N]) or
    "swiglu".  rms_eps: None, or the eps of the rms-norm folded into this step."""
    if epilogue not in ("none", "add", "bias", "swiglu"):
        raise ValueError("unknown epilogue")
    if (epilogue in ("add", "bias")) != (addend_h is not None):
        raise ValueError("an addend goes with the add and bias epilogues and with no other")
    r = rms_scale(x_h, rms_eps) if rms_eps is not None else None
    y = matmul(x_h, w_hat_h, addend_h=addend_h, row_scale=r)
    return swiglu_blocks(y) if epilogue == "swiglu" else y
