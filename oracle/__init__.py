"""CPU oracle for 2-D Winograd convolution F(m x m, r x r), r = 3 or 5, with arbitrary points.

TEST INFRASTRUCTURE ONLY.  Nothing in the product path may import this package:
only the tests, the smoke check and the benchmark's CPU-baseline leg do.  It
shares no code with the CUDA library.

Contents (each function cites the passage of the paper it follows):
  toom_cook  - exact rational construction of A^T, G, B^T (Algorithm 3,
               Section 2.4), the exact decomposition identity, kappa_2(V)
               (Section 2.2); diagonal rescaling D_A D_G D_B = I; snap-to-rational
               (Algorithm 2); the symmetric search over the snap grid.
  conv       - direct fp64 r x r cross-correlation (Section 2.1, the plain
               definition), Winograd in fp64 (Section B.5 / Eq. in "Exact Zero
               with Rational Arithmetic"), exact-rational Winograd for tiny
               inputs, and the rounding emulation of the low-precision
               pipeline (Section 5.1 "FP16 Setup", Section C.3 "Setup"), and the
               emulation of the INT8 Winograd-domain pipeline (Section 5.1 "INT8
               Setup").

Pins: every function here is pinned by tests that run without a GPU; the
exceptions are the *absolute levels* of the fp16 and INT8 emulation errors - the
paper prints the former only for an unstated workload and the latter for a set-up
it does not fully specify - those levels are "parity unpinned" (the emulations
themselves are pinned by their exact special cases and, for INT8, by the
qualitative content of the printed table).
"""
