"""BAPS oracle -- TEST INFRASTRUCTURE, NOT PRODUCT CODE.

A plain double-precision CPU statement of the BAPS hot path (Algorithm 1 and Algorithm 2 of
the paper, Eq. (1) and Eq. (2), and the HiF8 format it adopts), used to check the CUDA
library.  Only the tests, the smoke check and the CPU-baseline leg of the benchmark may
import this package.  It shares no code with the CUDA path and does not import it.
"""
from .baps_oracle import (  # noqa: F401
    build,
    hif8_value_table,
    hif8_encode,
    hif8_decode,
    exp2_code_table,
    encode_scalar,
    attention,
    softmax_rows,
    softmax_rows_codes,
    all_tiles,
    num_threads,
    MODE_E2E_HIF8,
    MODE_EXACT,
    MODE_IDENTITY,
    MODE_EXP2_HIF8,
    MODE_EXP2_IDENTITY,
    MODE_EXP2_E4M3,
    MODE_EXP2_E5M2,
    MODE_EXP2_E4M3_E5M2,
    MODE_NAIVE_E2E,
    round_e4m3,
    round_e5m2,
)
