"""CPU oracle for the E0M4 weight-only FP4 matmul (test infrastructure only).

This package is the slow, plain restatement of what the path computes, written
from the paper's Section 2.3 ("E0M4 FP4 quantization") and Section 2.2
("Operator optimizations").  It exists to check the CUDA library; it is not a
fallback.  Only the tests, the smoke check and the benchmark's CPU-baseline leg
may import it.  It shares no code with the CUDA path and never imports the
product package.

Parity unpinned: nothing (every function below is pinned by the CPU tests).
"""

from .e0m4 import (  # noqa: F401
    GROUP,
    e0m4_bits,
    e0m4_value,
    quantize,
    dequantize,
    matmul,
    int4_minmax_roundtrip,
    swiglu_blocks,
)
from .int4 import quantize_int4  # noqa: F401
from .kvcache import kv_append  # noqa: F401
from .norm import layernorm, rms_scale, rmsnorm  # noqa: F401
from .chain import chain_step  # noqa: F401
from .layout import pack, unpack, packed_sizes  # noqa: F401
