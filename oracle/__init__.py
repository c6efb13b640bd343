"""CPU checker (test infrastructure only; see mla_oracle.py)."""
