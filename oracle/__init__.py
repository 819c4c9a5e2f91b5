"""CPU oracle (test infrastructure): see skipdecode_oracle.py."""
