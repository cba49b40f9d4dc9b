"""CPU float64 oracle.  TEST INFRASTRUCTURE ONLY: imported by tests, the smoke check and the
CPU-baseline leg of the benchmark; never by the product.  Every function is pinned by
tests/test_oracle_pins.py against closed forms, library routines and finite differences."""
