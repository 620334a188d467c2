"""CPU oracle for the Breadcrumbs Reasoning decode hot path.

TEST INFRASTRUCTURE ONLY.  Nothing in the product package imports this; it is
used by the tests, by the smoke check and by the benchmark's CPU-baseline leg.
It shares no code with the CUDA path.
"""
