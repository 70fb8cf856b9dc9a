"""CPU oracle of the Lazy Attention decode path.  Test infrastructure: imported only by
tests/, the smoke check and the benchmark's CPU-baseline leg; never by the CUDA library."""
