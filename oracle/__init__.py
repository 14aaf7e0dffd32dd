"""CPU oracle for the W4A8 quantized linear layer (Sec. 3.4, "Quantization").

TEST INFRASTRUCTURE ONLY.  Nothing under this directory is part of the product
path: it may be imported by the tests, by the smoke check and by the benchmark's
CPU-baseline leg, and by nothing else.  It shares no code, header, table or
helper with the CUDA library and never imports it.

Three independent statements of the same definition live here:

* ``oracle.exact``      - pure Python ``int`` / ``fractions.Fraction``; every
                          rounding is carried out on exact rationals.  Tiny
                          shapes only.  It pins the two below.
* ``oracle.w4a8_oracle``- numpy, int64 + fp64, group by group in the order the
                          definition is written.  Sizes up to a few 1e9 MACs.
* ``oracle/w4a8_oracle.c`` (``oracle.cfast`` loads it) - the same loops in
                          plain C with OpenMP; int32 partials, fp64 scaling.
                          Full-size shapes and the timed CPU baseline.

Parity pins (see tests): a hand-worked example, tie and clamp examples,
brute force against ``oracle.exact``, the dequantise-then-dgemm identity,
scale linearity, zero-point invariants and the a-priori quantisation bound.
No function here is "parity unpinned".
"""
