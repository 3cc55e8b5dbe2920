"""CPU oracle for the LBA contraction.  TEST INFRASTRUCTURE ONLY.

Two independent statements of the same definition live here:

* ``lba_oracle`` (C++, exact dyadic carrier, threaded): GEMM, convolution, sampled points.
* ``lba_exact`` (pure Python, exact rationals): Eq. 2 and Eq. 4 written out literally,
  for small cases; it pins the C++ coding and is pinned by the same closed forms.

Only the tests, the smoke check and the benchmark's CPU-baseline leg may import this
package.  It shares no code with the CUDA library and never imports it.
"""
