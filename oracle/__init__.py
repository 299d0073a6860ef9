"""CPU oracle for the sparse decode hot path. TEST INFRASTRUCTURE ONLY.

Nothing in the product package may import this directory: only the tests, the
smoke check and the benchmark's CPU-baseline / reference legs do. It shares no
code with the CUDA library and never calls it.
"""
