"""CPU oracle for the SliceMoE hot path.  TEST INFRASTRUCTURE, not product code.

Plain, slow, obviously-correct numpy implementations (float64 for floating point unless the
format fixes a precision) of what the CUDA path computes, written from the paper.  Only the
tests, the smoke check and the benchmark's CPU-baseline leg may import this package; the CUDA
path shares no code with it and never calls it.

  amat.py  - asymmetric per-group quantiser, MSB/LSB slicing, the truncation rule (Eq. in
             Section 4.2) and both dequantisation rules
  moe.py   - top-k routing with optional cache-priority bias, precision request, the
             mixed-precision expert FFN, the layer with shared experts
  dbsc.py  - the slice cache of Section 4.1 (MSB LRU, LSB lowest priority) that turns routed
             ids + gating scores into per-(token, expert) precision flags and a miss list

Parity pins: every function here is checked in tests/test_oracle_*.py against exhaustive
identities, closed forms, constructed round trips, hand-computed examples (tests/golden/) and
brute force.  Unpinned (cannot be pinned without the paper's datasets, weights and hardware
simulator): task accuracy, perplexity, energy and latency ratios - "parity unpinned", and not
computed here.
"""
