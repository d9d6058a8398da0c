"""CPU oracle for zero-value compression (ZVC).

TEST INFRASTRUCTURE: imported only by the tests, the smoke check and the
benchmark's CPU-baseline leg.  It never imports the CUDA package and the CUDA
package never imports it.

``zvc_c``     -- ctypes front end of the plain-C oracle (``zvc_oracle.c``).
``zvc_numpy`` -- an independent numpy view of the same definition (masks,
                 packed values, sizes) used to cross-check the C code.
"""
