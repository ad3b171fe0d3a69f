"""CPU oracle (test infrastructure only; see astraea_oracle.c)."""
