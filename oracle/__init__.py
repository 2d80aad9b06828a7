"""CPU oracle: test infrastructure only (see scalebits_oracle.c)."""
