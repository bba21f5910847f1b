"""CPU oracle for 2-D Winograd convolution F(m x m, 3 x 3) with arbitrary points.

TEST INFRASTRUCTURE ONLY.  Nothing in the product path may import this package:
only the tests, the smoke check and the benchmark's CPU-baseline leg do.  It
shares no code with the CUDA library.

Contents (each function cites the passage of the paper it follows):
  toom_cook  - exact rational construction of A^T, G, B^T (Algorithm 3,
               Section 2.4), the exact decomposition identity, kappa_2(V)
               (Section 2.2).
  conv       - direct fp64 3x3 cross-correlation (Section 2.1, the plain
               definition), Winograd in fp64 (Section B.5 / Eq. in "Exact Zero
               with Rational Arithmetic"), exact-rational Winograd for tiny
               inputs, and the rounding emulation of the low-precision
               pipeline (Section 5.1 "FP16 Setup", Section C.3 "Setup").

Pins: every function here is pinned by tests that run without a GPU; the one
exception is the *absolute level* of the fp16 emulation error, which the paper
prints only for an unstated workload - that level is "parity unpinned" (the
emulation itself is pinned by its exact special cases).
"""
