"""CPU oracle of the three-layer sparse format and its SpMM.

TEST INFRASTRUCTURE ONLY.  The product (``paper_2607_08786_b200``) never imports this package;
only the tests, the smoke check and the CPU-baseline leg of the benchmark do.
"""
from .oracle import (  # noqa: F401
    Container,
    build,
    compact_nbytes,
    compact_nbytes_all,
    decode,
    dense_fp64,
    encode,
    float_to_half,
    half_to_float,
    residual_compact,
    residual_expand,
    spmm,
    threads,
    tolerance,
    values_compact,
    values_expand,
)
