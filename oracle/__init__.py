"""CPU oracle for band-wise local-operator chains.  TEST INFRASTRUCTURE ONLY.

Only the test-suite, the smoke check and the benchmark's CPU-baseline leg may import this
package; the CUDA library neither imports nor links anything in here, and nothing in here
touches the CUDA library.

  planner.py      integer band planner (band partition + halo back-propagation)
  lop_oracle.c    direct-loop conv2d / max-pool with the fused element-wise epilogue
  ops.py          ctypes access to the compiled C routines (numpy in, numpy out)
  chain.py        whole-tensor and band-wise execution of a layer list
  build.py        compiles lop_oracle.c with gcc

Parity status: every function is pinned by tests/test_oracle_*.py (closed forms, brute
force against a separately written naive loop, invariants, library special cases).
Absolute activation values of the large random workloads have no external reference and
are pinned only transitively through those per-operator checks.
"""
