"""CPU oracle package: test infrastructure only (see dare_oracle.py)."""
