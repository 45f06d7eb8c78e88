"""CPU oracle (test infrastructure only; see adapshot_oracle.py)."""
