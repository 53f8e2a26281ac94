"""CPU oracle of the CSD verification step (test infrastructure only; see csd_oracle.py)."""
