"""CPU oracle of the CrossQuant hot path -- test infrastructure only (see cq_oracle.c)."""
