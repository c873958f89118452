"""Shared pieces of the GPU parity tests: they live beside the oracle (oracle/check.py) so that the
smoke check and the bench harness use the same tolerance and the same reference."""
from oracle.check import (ABS_COEF, ABS_FLOOR, REL_L2, assert_gemv_close, gemv_errors,  # noqa: F401
                          make_matrix, oracle_product)
