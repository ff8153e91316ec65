"""CPU oracle of the expanded W4A4 linear layer: test infrastructure, never the product path.

Thin numpy binding over ``xq_oracle.c`` (plain C, fp64 / int64).  Only the tests, the smoke
check and the CPU-baseline leg of the benchmark import this package; the CUDA library and its
Python binding never do, and nothing here imports them.
"""
from .xq_oracle import (  # noqa: F401
    Plan,
    build,
    plan,
    hadamard_dense,
    hadamard_entry,
    bf16_to_f64,
    f64_to_bf16,
    rotate,
    rotate_dense,
    rotate_factored,
    quantize,
    quantize_asym,
    gemm_u_i64,
    epilogue_asym,
    rotate_quant_asym,
    expanded_linear_asym,
    pack_int4,
    unpack_int4,
    gemm_i64,
    epilogue,
    ref_product,
    prepare_weights,
    rotate_quant,
    expanded_linear,
    rotate_heads,
    rotate_quant_heads,
    rotate_quant_heads_asym,
    expanded_linear_heads,
    e2m1_value,
    quantize_mx,
    dequantize_mx,
    gemm_mx,
    rotate_quant_mx,
    expanded_linear_mx,
    num_threads,
)
