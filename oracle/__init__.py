"""CPU oracle (test infrastructure only): see hma_oracle.c and oracle.py."""
