"""CPU oracle of the RMSMP layer arithmetic -- TEST INFRASTRUCTURE, not a product path.

Only tests, the smoke check and the benchmark's CPU-baseline leg may import this package.
"""
