"""CPU oracle for the KAP hot path: TEST INFRASTRUCTURE ONLY.

Only the test-suite, the smoke check and the benchmark's CPU-baseline / reference leg may import
this package.  It shares no code with the CUDA library and neither imports the other.
"""
