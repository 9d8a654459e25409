"""CPU oracle of the HGF linear-layer forward pass: test infrastructure, never the product path.

Only the tests, the smoke check and the benchmark's cpu-baseline leg import this package.
"""
from .hgf_oracle import (  # noqa: F401
    FLAG_NO_SILU,
    act_quant,
    backward,
    diff_attention,
    build,
    effective_bits,
    forward,
    forward_ln,
    gamma_w,
    int_gemm,
    lambda0,
    ln_quant,
    ln_stats,
    pack,
    pack_b3,
    packed_bytes,
    packed_bytes_b3,
    ternarise,
    threads,
    tmax,
    unpack,
    unpack_b3,
)
