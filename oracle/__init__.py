"""fp64 CPU oracle of the hot path.  Test infrastructure only; see oracle.py and arb_oracle.c."""
