"""TurboBoA float64 CPU oracle (TEST INFRASTRUCTURE, not a product path).

Only tests, the smoke check and the benchmark's CPU-baseline leg import this
package.  It never imports the CUDA package and shares no code with it.

The dense steps with a textbook definition (Hessians, inverse, Cholesky,
matrix products) use numpy float64 library routines as single steps; the
quantization loop itself (grid, column sweep, compensation, coordinate
descent) is the plain C file next to this module, loaded through ctypes.
"""
from .ref import (  # noqa: F401
    OracleDesc,
    OracleResult,
    build_oracle,
    hessian,
    cross_correlation,
    hout_from_projection,
    factor_upper,
    correction_operands,
    quantize_layer,
    grid_rows,
    sweep_rows,
    comp_matrix,
    cd_refine,
    loss_head,
    group_loop_trace,
    num_threads,
    pack_codes,
    unpack_codes,
    dequantize,
    F_ADAPTIVE_GRID,
    F_CD_REFINE,
    F_DYNAMIC_GRID,
)
