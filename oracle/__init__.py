"""CPU oracle for the tensor-core-unit scan.  TEST INFRASTRUCTURE ONLY.

Two independent pieces live here, neither of which shares any code with the
CUDA library:

* ``scan_oracle``  - the prefix sum by its definition (sequential, int64/fp64),
  implemented in plain C (``scan_oracle.c``) with a thin ctypes loader;
* ``tcu_model``    - an instrumented model of the paper's matrix recursion
  (Algorithm 1, Algorithm 2 and the arbitrary-length extension of Section 2.2)
  that multiplies literal s x s matrices and counts rounds and products.

Only ``tests/``, the repository's smoke check and the benchmark's CPU-baseline
leg may import this package.  The product path never does.
"""
