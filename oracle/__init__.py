"""CPU oracle package: test infrastructure only (see qwt_oracle.py)."""
