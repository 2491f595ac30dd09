"""CPU oracle (test infrastructure): see uq_oracle.c for the arithmetic and its citations."""
