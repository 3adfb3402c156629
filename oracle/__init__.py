"""CPU oracle for the MoE GEMM2 + GatherRS path (test infrastructure only).

Nothing in the product package imports this directory.  The only callers are the tests,
the smoke check and the benchmark's CPU-baseline leg.
"""
