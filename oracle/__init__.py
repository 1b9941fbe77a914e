"""CPU oracle of the VSA2 attention path: test infrastructure only (see vsa2_oracle.py)."""
