"""CPU oracle for the tiered decode hot path (test infrastructure, not product).

Plain, slow, fp64 / integer restatements of what the paper's method computes:
page placement (Sec. 3.1, Sec. 4.2, Sec. 4.4), per-wave statistics (Sec. 2.6),
the wave-aware KV block pool (Sec. 4.3, Sec. 4.5) and the arithmetic the decode
kernels must reproduce (GEMV / skinny GEMM, softmax attention over paged KV,
stream sum, one Llama-shaped decode step).

Rules this package keeps:
  * it imports nothing from the CUDA package and the CUDA package imports
    nothing from here; the two share no helper, table or constant generator;
  * only tests, the smoke check and the benchmark's cpu-baseline / reference
    legs may import it;
  * every function cites the passage of the paper it follows.

Pins (tests/test_oracle_*.py) tie every function to something other than
itself: values the paper prints, closed forms, invariants, brute force.
Functions whose constants the paper does not fix (RMSNorm epsilon, RoPE base
and pairing in `decode.py`) are marked "parity unpinned" in their docstrings.
"""
