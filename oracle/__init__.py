"""CPU oracle (test infrastructure): see tkphi_oracle.py."""
