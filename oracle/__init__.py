"""EQuARX CPU oracle (test infrastructure, not part of the product).

Thin numpy/ctypes front end of ``equarx_oracle.c``.  Only the tests, the
smoke check and the bench's CPU legs import this package; the CUDA package
never does, and this package never imports the CUDA package.

bf16 tensors are numpy ``uint16`` arrays holding the raw bf16 words.
"""
from .binding import (  # noqa: F401
    OracleError,
    build,
    lib_path,
    quantize_blocks,
    rs_step,
    ag_dequant,
    allreduce,
    allreduce_bf16,
    allreduce_variant,
    error_bound,
)
