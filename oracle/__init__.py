"""CPU oracle (test infrastructure only; see mxq_oracle.c)."""
