"""CPU oracle for the FP8 delayed-scaling linear layer under a split-backward schedule.

TEST INFRASTRUCTURE ONLY.  This package is the plain, slow, obviously-correct
statement of what the hot path computes.  It shares no code with the CUDA path
and must never be imported by the product package; only the tests, the smoke
entry and the benchmark's CPU-baseline leg may call it.

Modules
  fp8      OCP E4M3 / E5M2 decode and round-to-nearest-even, saturating encode
  bf16     bfloat16 bit helpers (decode, single-rounding encode from float64)
  scaling  amax history + delayed scale rule (scale = fp8_max / max(hist) / 2^margin)
  layer    the F / dI / dW state machine with tape pool, versions and arena mask

Pins (tests/test_oracle_*.py): hand-computed FP8 bytes, exhaustive decode/encode
round trip and midpoint ties, ml_dtypes agreement inside the finite range, the
closed-form scale trajectory across a history rollover, exact-rational brute
force GEMMs, split == full backward bitwise, dW leaves scale state untouched,
and the contract's fault-injection table.

Parity unpinned: byte-for-byte agreement with NVIDIA Transformer Engine (the
paper delegates its numerics to that library and prints none of them).
"""
