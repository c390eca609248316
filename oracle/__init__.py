"""CPU oracle (test infrastructure only; see director_oracle.py)."""
