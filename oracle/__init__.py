"""CPU oracle -- TEST INFRASTRUCTURE ONLY (tests, smoke check, bench CPU-baseline leg).

Plain C loops (blas_oracle.c) with a ctypes front-end (blas_oracle.py).  Shares no code with
the CUDA library and is never imported by the product package.
"""
