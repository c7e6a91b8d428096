"""fp64 CPU oracle of the AdaPM step.  Test infrastructure: imported only by tests/,
the smoke check and the benchmark's CPU-baseline leg; never by the CUDA package."""
