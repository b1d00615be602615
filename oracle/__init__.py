"""CPU oracle for few-bit stochastic rounding.  TEST INFRASTRUCTURE ONLY.

Two independent statements of the same computation:

* ``oracle.paper_literal`` -- exact rational arithmetic, one element at a time,
  the paper's equations as printed (slow; small inputs).
* ``oracle/fbsr_oracle.c``  -- scalar C with exact integer predicates, loaded
  through ``oracle.capi`` (fast enough for millions of elements).

Nothing here is imported by the CUDA library or its Python binding, and nothing
here imports them.  Only tests, the smoke check and the benchmark's CPU-baseline
leg use this package.
"""
