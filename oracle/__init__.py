"""CPU oracle of the G10 planning path -- test infrastructure only (see g10_oracle.c)."""
