"""CPU oracle (test infrastructure only; see hdet_oracle.py)."""
