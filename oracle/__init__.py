"""fp64 CPU oracle for the composed-subkernel path.  TEST INFRASTRUCTURE ONLY:
imported by tests/, the smoke check and the benchmark's CPU-baseline leg, never
by the product package."""
