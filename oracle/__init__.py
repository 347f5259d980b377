"""CPU oracle for the quantized-and-cached DiT denoising step (Q&C, arXiv 2503.02508).

TEST INFRASTRUCTURE ONLY.  This package is the slow, plain definition the CUDA
library is checked against.  Only the test-suite, the smoke check and the
benchmark's CPU-baseline leg may import it; the library itself never does, and
this package imports nothing from the library.  numpy only; floating point is
float64 except where a value decides an integer code (the quantizer's rounding),
which is taken in float32 exactly as the method's 8-bit kernels take it.

Modules
  quant    uniform quantizer (Eq. 1), its parameters (Eq. 2-3), per-channel weights
  linear   exact integer matrix product and the de-quantising affine map around it
  dit      the DiT block / network the quantized linears sit in
  sampler  cache schedule (Background, "Quantization and Cache"), guidance, DDIM
  vc       variance compensation (section "Variance Align for Exposure Bias")
  calib    activation-range collection on a calibration batch (text after Eq. 3)

Parity status: every function here is pinned by tests/test_oracle_*.py against
closed forms, brute force, invariants or an independent library composition,
except end-to-end image quality (FID etc.), which is "parity unpinned": it needs
the paper's datasets, trained weights and evaluation toolkit.
"""
