"""Float64 CPU oracle for Stochastic Gradient Push (test infrastructure only).

This package is a plain, slow, obviously-correct restatement of the SGP
recursion (Alg. 1), its momentum form (Alg. 3) and the fixed-delay reading of
Overlap SGP (Alg. 2 read through the delay model of the supplementary
material, Eq. 4), together with its own generator of the mixing-matrix
schedules of App. A / App. C.

It is NOT part of the product: only the tests, the smoke check and the
benchmark's CPU-baseline leg may import it.  It shares no code with the CUDA
library and never imports the package that binds it.
"""
