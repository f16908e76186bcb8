"""CPU oracle for the paged-KV operator path -- TEST INFRASTRUCTURE, not the product.

Only the test suite, the smoke check and the CPU-baseline leg of the benchmark may
import this package.  It shares no code with the CUDA library and never calls it.

  value_model.py      the plain definition of every operator on token sequences
  kv_paged_oracle.c   the sequential paged pool (tables, refcounts, free ring, bytes)
  paged.py            ctypes wrapper around the compiled C file
"""
