"""CPU oracle of the group-sparse convolution path.  TEST INFRASTRUCTURE ONLY.

Only tests, the smoke check and the benchmark's CPU-baseline leg may import
this package; the CUDA library never does, and shares no code with it.
"""
