"""CPU oracle for the SDFP speculative-decode path.  TEST INFRASTRUCTURE: only
tests, the smoke check and the benchmark's CPU-baseline leg import this."""
