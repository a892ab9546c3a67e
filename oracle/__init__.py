"""CPU oracle (test infrastructure only; see entwine_oracle.py)."""
