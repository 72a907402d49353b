"""CPU checker for the A2CiD2 event update -- TEST INFRASTRUCTURE, not a product path.

Slow, plain, fp64. Written from the paper's definitions and pinned against closed forms by
the CPU test-suite. Only `tests/`, the smoke check and the benchmark's CPU-baseline leg may
import it; it shares no code with the CUDA library and never imports it.

  oracle.sim      OracleSim  -- sequential simulator backed by a2cid2_oracle.c (gcc)
  oracle.sim_np   NumpySim   -- the same steps in NumPy, for tiny cases
  oracle.spectral Laplacian, chi_1, chi_2 and the parameter prescription of the convergence proposition of Sec. 3.4
"""
