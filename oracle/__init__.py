"""CPU oracle for the LQER / L2QER linear layer (arXiv 2402.02446).

TEST INFRASTRUCTURE ONLY.  A plain, slow, fp64 numpy restatement of what the
layer computes, written from the paper.  It shares no code with the CUDA
library and never imports it; only the test-suite, the smoke check and the
benchmark's CPU-baseline leg may import it.  The product path never routes
through this package.

Pinned functions (each has tests that tie it to something other than itself):
  mxint.quantize / dequantize   hand-worked blocks, invariants, error bounds
  lqer.calibration_scale        closed-form example, min(s)*max(s) == 1
  lqer.jacobi_svd               orthogonality, reconstruction, textbook closed forms
  lqer.subspace_svd             agreement with jacobi_svd on mid-size matrices
  lqer.lqer_factors             full-rank identity, Eckart-Young residual closed form
  lqer.forward                  exact-rational brute force, k=0 special case, linearity
  lqer.average_weight_bits      the paper's 4.3-bit bookkeeping

Parity unpinned: the paper's perplexity / accuracy tables (they need trained
checkpoints and datasets that are not available here); they are not part of
this oracle.
"""
