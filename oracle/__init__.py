"""CPU oracle for the Spec-VLA tree-verification path. TEST INFRASTRUCTURE ONLY.

Nothing in the product package imports this; only tests, the smoke check and the
benchmark's CPU-baseline leg do. It shares no code with the CUDA path.
"""
