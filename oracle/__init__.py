"""fp64 CPU oracle for the attention forward pass -- TEST INFRASTRUCTURE ONLY.

Only the test suite, the smoke check and the benchmark's CPU-baseline leg may
import this package.  The product path (the CUDA library and its Python
binding) never does, and this package never imports the product path.
"""
from .attention import (  # noqa: F401
    attention,
    attention_prow,
    build,
    num_threads,
)
