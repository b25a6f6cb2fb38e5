"""CPU oracle for the S2A 4-bit activation stash.  TEST INFRASTRUCTURE, NOT THE PRODUCT.

Import only from tests, the smoke check and the benchmark's CPU-baseline leg.
"""
