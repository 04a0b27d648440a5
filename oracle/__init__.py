"""CPU oracle (test infrastructure only): see san_oracle.c for what it computes."""
