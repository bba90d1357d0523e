"""CPU oracle for the Flora hot path (test infrastructure only; see flora_oracle.c)."""
