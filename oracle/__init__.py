"""CPU oracle of the HEART hot path: test infrastructure only (see heart_oracle.c)."""
