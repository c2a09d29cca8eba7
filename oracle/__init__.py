"""CPU oracle (test infrastructure only; see talaria_oracle.c)."""
