"""CPU oracle package (test infrastructure; see as_oracle.c)."""
