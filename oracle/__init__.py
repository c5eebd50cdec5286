"""CPU ORACLE -- TEST INFRASTRUCTURE ONLY.

Plain, slow, obviously-correct fp64 / integer implementations of what the CUDA library
computes, written from the paper's equations.  Only the tests, the smoke check and the
benchmark's ``cpu_baseline`` / ``--impl reference`` legs may import this package; it
shares no code with the CUDA path and never imports it.
"""
