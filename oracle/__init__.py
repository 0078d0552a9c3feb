"""Float64 CPU oracle for the DeTAG step.

TEST INFRASTRUCTURE ONLY.  Nothing in the product path (the CUDA library, its Python
binding) imports, calls or links this package; it is used by the tests, by the smoke
check and by the benchmark's CPU-baseline leg.  It shares no code with the CUDA path.
"""
