"""fp64 CPU oracle for the FLy verification step. TEST INFRASTRUCTURE ONLY.

Nothing in the product path may import this package: it exists so that tests,
the smoke check and the benchmark's CPU-baseline leg have an independent,
slow, obviously-correct statement of what the CUDA path must compute.
"""
