"""Float64 CPU oracle of the CoS verification step: test infrastructure only.

Nothing in the product package imports this; tests, the smoke check and the CPU-baseline
leg of the benchmark do.
"""
