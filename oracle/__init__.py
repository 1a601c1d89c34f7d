"""CPU oracle package (test infrastructure only; see cowa_oracle.py)."""
