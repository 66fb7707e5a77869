"""CPU fp64 oracle for one block-diffusion denoising step (test infrastructure).

This package is test infrastructure, not product code.  It is a plain, slow,
double-precision restatement of what the decode hot path computes, written from
the paper's definitions:

* block-causal attention (Sec. 3.1, "Block-Causal Diffusion"),
* the shared-prefix fork of the KV cache (Sec. 3.4, "Shared prefix"),
* confidence-threshold parallel unmasking of the value positions of a block
  with frozen scaffold tokens (Sec. 3.2 scaffold definition, Sec. 3.3
  "Section Diffusion"),
* appending a finished block's K/V to a rollout's private cache (Sec. 3.3),
* the equal-weight mean of N rollout trajectories (Sec. 3.4, trajectory
  averaging).

Only the tests, the smoke check and the benchmark's CPU-baseline leg may import
it.  It shares no code with the CUDA library and never imports it.

Parity pins (see tests/test_oracle_*.py): every function here is pinned by
closed forms, brute force on tiny inputs, library special cases or published
known-answer values.  The jerk-minimising interpolation mentioned in Sec. 3.4
has no formula in the paper: `jmt.py` implements this repository's reading of it
and is pinned to that reading's variational definition only (parity with the
paper unpinned).
"""

MASKED = 0
COMMITTED = 1
SCAFFOLD = 2
