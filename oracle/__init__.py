"""CPU oracle (test infrastructure only; never imported by the product path)."""
from .t3_oracle import (  # noqa: F401
    build,
    gemm_rs,
    gemm_rs_f64,
    ring_order,
    ring_sum_f32,
    chunks,
    epilogue,
    epilogue_f32,
    threads,
    max_rel_err,
)
