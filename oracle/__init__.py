"""CPU oracle (fp64) for composed-cache query prefill.  TEST INFRASTRUCTURE ONLY: nothing in the
product package imports this; tests, the smoke check and the benchmark's CPU-baseline leg do."""
