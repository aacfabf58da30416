"""CPU checkers written from the paper.  Test infrastructure: only tests/, the smoke
check and the benchmark's CPU-baseline leg may import this package."""
