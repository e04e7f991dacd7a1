"""CPU fp64 oracle of the RoM layer forward.  Test infrastructure only: imported by
tests, the smoke check and the benchmark's cpu-baseline leg, never by the product path."""
