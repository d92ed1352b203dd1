"""CPU oracle (test infrastructure). See trl_oracle.py."""
