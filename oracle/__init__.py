"""TEST INFRASTRUCTURE — CPU oracle for one SpecDiff draft–verify–accept round.

Plain, slow, fp64 numpy.  Only the tests, the smoke check and the benchmark's CPU-baseline
leg may import this package; the product path (the CUDA library and its Python binding)
never does, and shares no code with it.
"""
