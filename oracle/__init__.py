"""CPU oracle for the spectral-split NVFP4 linear layer (Metis, Sections 2.3, 3.1, 3.2, Appendix C.1).

TEST INFRASTRUCTURE ONLY.  This package is a plain, slow, float64/numpy restatement of what the
hot path computes.  It shares no code, table or constant generator with the CUDA library and is
imported only by the tests, by the smoke check and by the benchmark's CPU-baseline leg.  The
product path never calls it.

Modules
-------
philox   counter-based random bits (Philox4x32-10) and the 16-bit-per-element draw rule
nvfp4    scalar/vectorised NVFP4 encoder and decoder (E2M1 values, 16-element blocks, E4M3 block
         scales rounded up, FP32 tensor scale), round-to-nearest-even and stochastic rounding
gauss    the Gaussian test matrix of the random projection, made reproducible bit for bit
split    sparse row sampling, randomized SVD, low-rank + residual split (FULL and SAMPLED modes)
layer    forward (Eq. 2), dgrad (Eq. 3) and wgrad of the split-FP4 linear layer
metrics  spectral-fidelity and subspace-alignment measures used by the paper's figures

Parity status: every function is pinned by tests in tests/test_oracle_*.py against closed forms,
brute force, library special cases or invariants, except the end-to-end layer value itself, whose
individual terms are pinned (bilinearity, k=0 reduction, exactly representable inputs) but whose
combined number has no independent source: "parity unpinned" for that single composite figure.
"""
