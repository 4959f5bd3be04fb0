"""CPU oracle for the DGQ hot path.  TEST INFRASTRUCTURE ONLY.

A plain, slow, fp64 / int64 restatement of what the paper's method computes,
written from the paper and used to check the CUDA library.  Nothing in the
product path imports it: only the tests, the smoke check and the benchmark's
CPU-baseline leg do.  It shares no code with the CUDA sources.

Equations are unnumbered in the paper; they are numbered here in order of
appearance:

  Eq. 1  linear quantizer / de-quantizer            (Sec. 3.1)
  Eq. 2  logarithmic quantizer / de-quantizer       (Sec. 3.1)
  Eq. 3  softmax attention score                    (Sec. 3.2)
  Eq. 4  range-variability metric D_d               (Sec. 3.3)
  Eq. 5  d* = argmax_d D_d                          (Sec. 3.3)
  Eq. 6  per-group scale s_k and zero-point z_k     (Sec. 3.3)
  Eq. 7  per-timestep parameter sets S, Z           (Sec. 3.3)
  Eq. 8  log-quantized cross-attention codes        (Sec. 3.3)
  Eq. 9  split product  A_hat V_hat                 (Sec. 3.3)

Parity unpinned (readings the paper does not fix numerically; see each
function): the K-means initialisation, the 2^b denominator of Eq. 6 taken
literally, and the per-prompt scope of the maximum in Eq. 8.
"""
from . import quantizers, calibration, linear, attention  # noqa: F401
