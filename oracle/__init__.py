"""CPU oracle for the BF16 output projection with residual — TEST INFRASTRUCTURE.

Only tests, the smoke check and the benchmark's CPU-baseline leg import this
package.  The product (the CUDA library and its Python binding) never does.
"""
from .oracle import (  # noqa: F401
    outproj, outproj_rows, element, round_bf16, widen_bf16, max_threads, rmsnorm, swiglu,
    quantize_rows, swiglu_int8, outproj_int8,
    e4m3_decode, e4m3_encode, quantize_rows_fp8, swiglu_fp8, outproj_fp8,
    e8m0_decode, quantize_rows_mx, outproj_mx, swiglu_mx,
    e2m1_decode, e2m1_encode, quantize_rows_nvfp4, outproj_nvfp4, swiglu_nvfp4,
)
