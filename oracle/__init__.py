"""CPU oracle (test infrastructure only; see hat_oracle.c)."""
