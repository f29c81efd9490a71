"""CPU oracle: test infrastructure only (see q4d_oracle.c)."""
