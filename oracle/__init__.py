"""CPU oracle for the PermuQuant quantized-linear hot path.  Test infrastructure only:
nothing on the product path may import this package."""
