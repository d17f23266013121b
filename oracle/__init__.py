"""CPU oracle of the Rudra parameter-server path: test infrastructure, not product code.

Only tests, the smoke check and the benchmark's CPU-baseline leg import this package.
"""
