"""Float64 CPU oracle for SWAA attention.  TEST INFRASTRUCTURE, NOT PRODUCT CODE.

Only the tests, the smoke check and the benchmark's CPU-baseline leg may import
this package; the GPU library never does, and this package never imports the GPU
library.  See ``swaa_oracle.c`` for the definition it implements and the paper
passages it follows.
"""
from .swaa_oracle import (  # noqa: F401
    build,
    count_pairs,
    decode,
    decode_combine,
    decode_partial,
    decode_paged,
    layer_is_full,
    layer_is_full_mask,
    select_fa_layers,
    lazy_ratio,
    num_threads,
    prefill,
    prefill_backward,
    prefill_backward_c,
    prefill_backward_rows,
    prefill_chunked,
    prefill_cp,
    prefill_paged,
    visible,
)
