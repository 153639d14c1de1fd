"""CPU oracle for the HPD decode step -- TEST INFRASTRUCTURE ONLY.

Only the test-suite, the smoke check and the benchmark's cpu-baseline leg may import this
package.  It shares no code with the CUDA path and does not import it.

``oracle.capi``  ctypes front-end of ``hpd_oracle.c`` (plain C, fp64 arithmetic)
``oracle.brute`` an independent full-matrix masked-softmax formulation in numpy (fp64)
``oracle.build`` compiles the C file with gcc
"""
