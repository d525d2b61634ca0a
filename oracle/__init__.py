"""Plain CPU oracle of the DART drafting step.  TEST INFRASTRUCTURE ONLY: imported by the
tests, the smoke check and the benchmark's CPU-baseline leg, never by the CUDA library or
its Python binding."""
