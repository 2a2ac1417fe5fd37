"""CPU oracle for the AdaCGD hot path.

TEST INFRASTRUCTURE ONLY.  This package is a plain, slow, CPU-only restatement of
what the paper (arXiv 2211.00188) defines.  It is imported by the test-suite, by
the smoke check and by the benchmark's CPU-baseline leg, and by nothing else: the
CUDA product path never calls into it and shares no code with it.
"""
