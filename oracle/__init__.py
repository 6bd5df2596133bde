"""CPU oracle of the DBA step -- test infrastructure only (see dba_oracle.c)."""
