"""CPU fp64 oracle (test infrastructure only; see monarch_oracle.py)."""
