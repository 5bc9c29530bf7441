"""CPU oracle (test infrastructure only): see fmm_oracle.c and realizations.py."""
