"""CPU oracle (test infrastructure only): see fp2_oracle.py."""
