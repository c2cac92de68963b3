"""CPU oracle (test infrastructure only; see parle_oracle.py)."""
