"""fp64 CPU oracle of the L2A layer.  TEST INFRASTRUCTURE ONLY.

Only the tests, the smoke check and the benchmark's CPU-baseline leg may import this package.
It shares no code with the CUDA library and never imports it.

``l2a_oracle.c`` holds the plain definition (Eq. 2-5, masks of Section 2, textbook VJP);
``chunked.py`` evaluates the same attention as a running soft-max over arbitrary key chunks (the evaluation order of
Algorithm 1); the tests require it to equal the plain definition for any chunking.
"""
from .binding import (  # noqa: F401
    Shape,
    build,
    compact,
    route,
    forward_rows,
    forward_full,
    backward_full,
    dq_rows,
    dkv_cols,
    dgate_rows,
    num_threads,
    f64_inputs,
    router_logits,
    gate_regulariser_sum,
    router_backward,
)
