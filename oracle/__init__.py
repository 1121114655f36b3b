"""CPU oracle (test infrastructure): see oracle.py and wfq_oracle.c."""
