"""CPU oracle of the FSD / SD verification step.  TEST INFRASTRUCTURE: imported only by
tests, the smoke check and the benchmark's CPU-baseline leg; never by the product."""
