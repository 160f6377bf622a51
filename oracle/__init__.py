"""CPU oracle of the SwiftPrune pruning pass: test infrastructure only.

Nothing under this package is part of the product.  It may be imported by the
test-suite, by the smoke check and by the benchmark's CPU-baseline leg, and by
nothing else.
"""
