"""CPU fp64 oracle for scaled-dot-product attention. TEST INFRASTRUCTURE ONLY:
tests, the smoke check and the benchmark's CPU-baseline leg may import it; the
product package never does."""
