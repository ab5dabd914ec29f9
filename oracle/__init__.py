"""Float64 CPU checker for the FiCoCo reduce step.  Test infrastructure only: imported by
the tests, the smoke check and the benchmark's CPU-baseline leg, never by the product."""
