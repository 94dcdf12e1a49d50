"""Plain CPU oracle for the FDG module-step path.  TEST INFRASTRUCTURE ONLY:
imported by tests/, by the smoke check and by the benchmark's cpu-baseline leg,
never by the CUDA library or its binding."""
