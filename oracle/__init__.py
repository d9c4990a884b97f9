"""CPU oracle of the CO3 gradient pipeline: test infrastructure, not the product.

Only tests, the smoke check and the benchmark's CPU-baseline leg import this package.  It never
imports the CUDA library's package, and the CUDA library never imports it.
"""
