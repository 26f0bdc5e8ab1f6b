"""CPU oracle of the Hotline hot path: test infrastructure only (see hotline_oracle.py)."""
