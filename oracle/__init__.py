"""CPU oracle for the DVD-Quant quantized-linear path.  TEST INFRASTRUCTURE ONLY:
imported by tests, the smoke check and the benchmark's cpu-baseline leg; never by
the CUDA product path, with which it shares no code."""
