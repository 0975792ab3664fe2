"""CPU oracle for the MiLoRA serving hot path.

TEST INFRASTRUCTURE ONLY.  This package is a slow, plain fp64 restatement of
what the paper's method computes (prompt-aware routing, route reuse, token
grouping, LoRA-augmented projections).  It exists so that the CUDA library can
be checked against something that was written independently of it.  It shares
no code with the CUDA path and must never be imported by it; only the tests,
the smoke check and the benchmark's CPU-baseline leg call into it.
"""
