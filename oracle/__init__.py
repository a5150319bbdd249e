"""CPU oracle for the low-bit linear layer (test infrastructure, not product code).

Everything under this package is a plain, slow, deliberately unoptimised CPU
statement of what the quantised linear path computes.  It exists so that the
CUDA library can be checked against something that can be verified by eye.

Rules this package keeps:
  * it imports nothing from the CUDA package and shares no code, table or
    constant with it;
  * only the tests, the smoke check and the benchmark's CPU-baseline leg may
    import it; the product path never does.

Two independent writings of the same specification live here:
  * ``np_oracle``  - NumPy, vectorised only where the vectorisation is the
    definition itself (elementwise ops, ``numpy.matmul`` in fp64 / int64);
  * ``c/qil_oracle.c`` (+ ``c_oracle`` ctypes wrapper) - plain C loops, with an
    OpenMP pragma on the outermost independent loop, used for the timed CPU
    baseline and as a cross-check of the NumPy writing.

Parity pins (what fixes the oracle to something other than itself) are in
``tests/test_oracle_pins.py`` and ``tests/golden/``.  The paper prints no worked
numeric example for its quantiser (it names round-to-nearest and refers to a
figure), so beyond the closed forms, invariants, hand cases and library
reductions listed there, parity against the paper's own numbers is unpinned.
"""
