"""CPU oracle of the sparse decode step (test infrastructure; see spin_oracle.py)."""
