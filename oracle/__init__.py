"""CPU oracle of the GaLore-Adam step.  TEST INFRASTRUCTURE ONLY.

Imported by the tests, by the smoke check and by the CPU-baseline leg of the
benchmark; never by the CUDA package, which in turn is never imported here.
"""
