"""CPU oracle of the Pacer hot path.  Test infrastructure: imported only by the
tests, the smoke check and the benchmark's cpu-baseline leg."""
