"""CPU oracle for the LESS decode / prefill path (arxiv 2402.09398).

TEST INFRASTRUCTURE ONLY.  This package is a plain, slow, fp64 restatement of
the method, written from the paper's equations.  It shares no code with the
CUDA path and must never be imported by the product package: only the test
suite, the smoke check and the benchmark's CPU-baseline leg may use it.
"""
