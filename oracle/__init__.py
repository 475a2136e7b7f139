"""CPU oracle (test infrastructure only; see celty_oracle.py)."""
