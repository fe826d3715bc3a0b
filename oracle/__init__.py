"""CPU oracle package: test infrastructure only (see marche_oracle.py)."""
